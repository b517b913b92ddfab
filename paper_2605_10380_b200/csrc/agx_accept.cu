// Greedy acceptance: per-row vocabulary argmax fused with the draft comparison and the length
// commit, in ONE launch (Sec. 2.3, speculative decoding: the first mismatching draft and all
// drafts after it are discarded; the accepted drafts plus the target's own token continue).
//
// HBM-bound scan: rows * vocab * elem bytes, read once with 128-bit loads.  Grid = (chunks, rows);
// every block reduces its slice of one row to a packed 64-bit (ordered value, inverted index) key
// whose unsigned maximum is "largest value, lowest index on ties", and folds it into the row's key
// with one 64-bit atomic maximum (order-independent, so the result is bit-reproducible).  The last
// block to finish (ticket counter) reads the row keys back, leaves them and the ticket at zero for
// the next launch, compares drafts and writes the results, so no second launch and no host round
// trip is needed.
#include "agx_internal.cuh"
#include "agx_sm100.cuh"

namespace agx {

// Monotone map float -> uint32 with: NaN -> 0 (below everything), -0 == +0.
__device__ __forceinline__ unsigned int ordered_key(float x) {
    if (x != x) return 0u;
    unsigned int b = __float_as_uint(x);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ unsigned long long pack_key(unsigned int key, unsigned int idx) {
    return ((unsigned long long)key << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}

__device__ __forceinline__ float bf16_bits_to_float(unsigned int lo16) { return __uint_as_float(lo16 << 16); }

template <bool kBf16>
__device__ __forceinline__ void scan_vec(const uint4 v, unsigned int base, unsigned int& best_key,
                                         unsigned int& best_idx) {
    const unsigned int w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (kBf16) {
            const unsigned int k0 = ordered_key(bf16_bits_to_float(w[i] & 0xFFFFu));
            const unsigned int k1 = ordered_key(__uint_as_float(w[i] & 0xFFFF0000u));
            if (k0 > best_key) { best_key = k0; best_idx = base + 2 * i; }
            if (k1 > best_key) { best_key = k1; best_idx = base + 2 * i + 1; }
        } else {
            const unsigned int k0 = ordered_key(__uint_as_float(w[i]));
            if (k0 > best_key) { best_key = k0; best_idx = base + i; }
        }
    }
}

constexpr int kTokSmem = 2048;               // winners of up to this many rows stay in shared memory for the draft comparison

template <bool kBf16, bool kVec>
__global__ void __launch_bounds__(256)
accept_kernel(const void* __restrict__ logits, long long row_stride, int vocab, int chunk_elems,
              const int* __restrict__ drafts, const int* __restrict__ cu_q, int B, int total_q,
              int* __restrict__ accept_len, int* __restrict__ next_token, int* __restrict__ argmax,
              int* __restrict__ seq_lens, unsigned long long* row_keys, int* tokens_global, unsigned int* ticket) {
    constexpr int kVecElems = kBf16 ? 8 : 4;
    pdl_launch_dependents();
    pdl_wait();
    const int row = blockIdx.y;
    const int chunk = blockIdx.x;
    const unsigned int begin = (unsigned int)chunk * (unsigned int)chunk_elems;
    const unsigned int end = min((unsigned int)vocab, begin + (unsigned int)chunk_elems);

    unsigned long long best = 0ull;  // "no element": loses to every real element
    if (kVec) {
        const char* row_ptr = (const char*)logits + (size_t)row * row_stride * (kBf16 ? 2 : 4);
        unsigned int best_key = 0u, best_idx = 0u;
        bool any = false;
        // two independent 16-byte loads in flight per thread per trip
        unsigned int i = begin + threadIdx.x * kVecElems;
        const unsigned int stride = 256 * kVecElems;
        for (; i + stride + kVecElems <= end; i += 2 * stride) {
            const uint4 a = __ldg((const uint4*)(row_ptr + (size_t)i * (kBf16 ? 2 : 4)));
            const uint4 b = __ldg((const uint4*)(row_ptr + (size_t)(i + stride) * (kBf16 ? 2 : 4)));
            if (!any) { best_idx = i; any = true; }
            scan_vec<kBf16>(a, i, best_key, best_idx);
            scan_vec<kBf16>(b, i + stride, best_key, best_idx);
        }
        for (; i < end; i += stride) {
            if (i + kVecElems <= end) {
                const uint4 a = __ldg((const uint4*)(row_ptr + (size_t)i * (kBf16 ? 2 : 4)));
                if (!any) { best_idx = i; any = true; }
                scan_vec<kBf16>(a, i, best_key, best_idx);
            } else {
                for (unsigned int e = i; e < end; ++e) {
                    float x;
                    if (kBf16) x = bf16_bits_to_float(((const unsigned short*)row_ptr)[e]);
                    else x = ((const float*)row_ptr)[e];
                    const unsigned int k = ordered_key(x);
                    if (!any) { best_idx = e; any = true; }
                    if (k > best_key) { best_key = k; best_idx = e; }
                }
            }
        }
        if (any) best = pack_key(best_key, best_idx);
    } else {
        for (unsigned int e = begin + threadIdx.x; e < end; e += 256) {
            float x;
            if (kBf16) x = bf16_bits_to_float(((const unsigned short*)logits)[(size_t)row * row_stride + e]);
            else x = ((const float*)logits)[(size_t)row * row_stride + e];
            const unsigned long long k = pack_key(ordered_key(x), e);
            best = k > best ? k : best;
        }
    }

    // block reduce (unsigned 64-bit max)
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, best, off);
        best = o > best ? o : best;
    }
    __shared__ unsigned long long warp_best[8];
    __shared__ bool is_last;
    if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long b = warp_best[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) b = warp_best[w] > b ? warp_best[w] : b;
        if (b) atomicMax(row_keys + row, b);   // (every key of a real element is non-zero: its low word is 2^32 - 1 - index)
        __threadfence();
        const unsigned int total = gridDim.x * gridDim.y;
        const unsigned int t = atomicAdd(ticket, 1u);
        is_last = (t == total - 1);
        if (is_last) *ticket = 0u;  // leave the counter ready for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // the rows' winners: read the keys back past the L1, zero them for the next launch; up to kTokSmem winners stay in
    // shared memory for the draft comparison, more go through global memory
    __shared__ int tokens_smem[kTokSmem];
    const bool in_smem = total_q <= kTokSmem;
    int* tokens = in_smem ? tokens_smem : tokens_global;
    for (int r = threadIdx.x; r < total_q; r += 256) {
        const unsigned long long b = __ldcg(row_keys + r);
        row_keys[r] = 0ull;
        const int t = (int)(0xFFFFFFFFu - (unsigned int)(b & 0xFFFFFFFFull));
        tokens[r] = t;
        if (argmax) argmax[r] = t;
    }
    __syncthreads();
    // draft comparison and commit: one warp per sequence, 32 drafts compared at a time
    for (int s = threadIdx.x >> 5; s < B; s += 8) {
        const int lane = threadIdx.x & 31;
        const int r0 = cu_q[s];
        const int k = cu_q[s + 1] - r0 - 1;
        const int* dr = drafts + (r0 - s);
        int a = 0;
        while (a < k) {
            const bool match = (a + lane < k) ? (dr[a + lane] == (in_smem ? tokens[r0 + a + lane] : __ldcg(tokens + r0 + a + lane))) : false;
            const unsigned int m = __ballot_sync(0xFFFFFFFFu, match);
            const int run = (m == 0xFFFFFFFFu) ? 32 : __ffs(~m) - 1;   // leading matches of this group of 32
            a += run;
            if (run < 32) break;
        }
        if (lane == 0) {
            accept_len[s] = a;
            next_token[s] = in_smem ? tokens[r0 + a] : __ldcg(tokens + r0 + a);
            if (seq_lens) seq_lens[s] = seq_lens[s] + a + 1;
        }
    }
}

cudaError_t launch_accept(const void* logits, int logits_dtype, long long row_stride, int vocab, const int* drafts,
                          const int* cu_q, int B, int total_q, int* accept_len, int* next_token, int* argmax,
                          int* seq_lens, unsigned long long* row_keys, int* tokens_global, int chunks, unsigned int* ticket,
                          cudaStream_t stream) {
    const bool bf16 = logits_dtype == AGX_BF16;
    const int esz = bf16 ? 2 : 4;
    const int vec_elems = 16 / esz;
    int chunk_elems = (vocab + chunks - 1) / chunks;
    chunk_elems = (chunk_elems + vec_elems - 1) / vec_elems * vec_elems;  // chunk starts stay 16-byte aligned
    const bool vec = ((uintptr_t)logits % 16 == 0) && ((row_stride * esz) % 16 == 0);
    dim3 grid(chunks, total_q);
    cudaError_t err = cudaSuccess;
#define AGX_LAUNCH_ACCEPT(BF, VEC)                                                                              \
    err = launch_chained(accept_kernel<BF, VEC>, grid, dim3(256), 0, stream, logits, row_stride, vocab, chunk_elems,  \
                         drafts, cu_q, B, total_q, accept_len, next_token, argmax, seq_lens, row_keys, tokens_global, \
                         ticket)
    if (bf16) { if (vec) AGX_LAUNCH_ACCEPT(true, true); else AGX_LAUNCH_ACCEPT(true, false); }
    else      { if (vec) AGX_LAUNCH_ACCEPT(false, true); else AGX_LAUNCH_ACCEPT(false, false); }
#undef AGX_LAUNCH_ACCEPT
    return err;
}

}  // namespace agx

// --------------------------------------------------------------------------------------------
// Allocation-free variant of the accept step.
//
// Some callers cannot allocate device memory at the point where they verify drafts: code running
// inside a pre-sized serving arena or an embedded runtime whose memory is fixed at start-up, and
// code that must not disturb a caching allocator owned by someone else (a cudaMalloc there can
// synchronise the device or fail outright).  agx_accept_greedy needs a caller-provided workspace
// and a handle whose creation allocates; the entry point below needs neither.  Its scratch (the
// rows' argmax keys and the ticket counter) lives in a fixed array that is part of the loaded
// module, so every GPU that loads the library carries these 16 KB until the process exits.
#include <atomic>
#include <mutex>

namespace agx {
namespace {
constexpr int kStaticMaxRows = 2048;    // logits rows per call (their winners fit the kernel's shared memory)
constexpr int kStaticDevices = 64;
// layout: [0, 256) ticket counter | one 64-bit key per row
constexpr size_t kStaticBytes = 256 + (size_t)kStaticMaxRows * 8;
static_assert(kStaticMaxRows <= kTokSmem, "the allocation-free variant has no global buffer for the rows' winners");
static __device__ __align__(256) unsigned char g_accept_scratch[kStaticBytes];

struct StaticDeviceState {
    std::atomic<void*> scratch{nullptr};  // device address of g_accept_scratch on that device (NULL until resolved)
    int sm_count = 0;                     // written before `scratch` is published
};
StaticDeviceState g_static_state[kStaticDevices];
std::mutex g_static_init;                 // serialises the one-time set-up (several host threads may make the first call)

inline bool aligned_to(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }
}  // namespace
}  // namespace agx

extern "C" AGX_API agx_status agx_accept_greedy_static(const void* logits, int32_t logits_dtype, int64_t row_stride,
                                                       int32_t vocab, const int32_t* drafts, const int32_t* cu_q,
                                                       int32_t B, int32_t total_q, int32_t* accept_len,
                                                       int32_t* next_token, int32_t* argmax, int32_t* seq_lens,
                                                       void* stream) {
    using namespace agx;
    if (B < 0 || total_q < 0) return AGX_E_INVAL;
    if (B == 0) return AGX_OK;
    if (total_q < B) return AGX_E_INVAL;
    if (logits_dtype != AGX_BF16 && logits_dtype != AGX_F32) return AGX_E_UNSUPPORTED;
    if (vocab < 1 || row_stride < vocab) return AGX_E_RANGE;
    if (!logits || !cu_q || !accept_len || !next_token || (!drafts && total_q > B)) return AGX_E_INVAL;
    // the same alignment rules as the workspace variant: a misaligned pointer is an argument error, not a device fault
    if (!aligned_to(logits, logits_dtype == AGX_BF16 ? 2 : 4) || !aligned_to(drafts, 4) || !aligned_to(cu_q, 4) ||
        !aligned_to(accept_len, 4) || !aligned_to(next_token, 4) || !aligned_to(argmax, 4) || !aligned_to(seq_lens, 4))
        return AGX_E_INVAL;
    if (total_q > kStaticMaxRows) return AGX_E_RANGE;  // beyond the fixed scratch: use agx_accept_greedy

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kStaticDevices) return AGX_E_CUDA;
    StaticDeviceState& st = g_static_state[device];
    void* scratch = st.scratch.load(std::memory_order_acquire);
    if (!scratch) {
        // One-time set-up for this device, with it current.  In host code the array's name is only a
        // stand-in for the symbol; the address kernels can use has to be asked for.
        std::lock_guard<std::mutex> lock(g_static_init);
        scratch = st.scratch.load(std::memory_order_relaxed);
        if (!scratch) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_accept_scratch) != cudaSuccess || !ptr) return AGX_E_CUDA;
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) return AGX_E_CUDA;
            st.sm_count = sms;
            st.scratch.store(ptr, std::memory_order_release);
            scratch = ptr;
        }
    }
    // Chunks per row: enough CTAs that every thread needs a single trip of two 16-byte loads (8 per SM, as the workspace
    // variant aims for).
    const int vec = logits_dtype == AGX_BF16 ? 8 : 4;
    int want = (8 * st.sm_count + total_q - 1) / total_q;
    const int max_chunks = (vocab + 256 * vec * 2 - 1) / (256 * vec * 2);   // >= 2 vectors per thread
    if (want > max_chunks) want = max_chunks;
    if (want < 1) want = 1;
    int chunk_elems = (vocab + want - 1) / want;
    chunk_elems = (chunk_elems + vec - 1) / vec * vec;
    const int chunks = (vocab + chunk_elems - 1) / chunk_elems;   // <= want

    unsigned char* base = (unsigned char*)scratch;
    // the array keeps whatever the previous call left: the ticket counter and the rows' keys must start at zero (the
    // kernel leaves them at zero itself; the clear makes the call independent of how an earlier one ended)
    if (cudaMemsetAsync(base, 0, 256 + (size_t)total_q * 8, (cudaStream_t)stream) != cudaSuccess) return AGX_E_CUDA;
    cudaError_t e = launch_accept(logits, logits_dtype, row_stride, vocab, drafts, cu_q, B, total_q, accept_len,
                                  next_token, argmax, seq_lens, (unsigned long long*)(base + 256), nullptr, chunks,
                                  (unsigned int*)base, (cudaStream_t)stream);
    return e == cudaSuccess ? AGX_OK : AGX_E_CUDA;
}
