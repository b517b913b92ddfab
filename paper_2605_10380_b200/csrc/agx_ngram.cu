// n-gram draft source of example-based speculative decoding (Sec. 4.3): a lookup table built from one
// token stream (key = n-1 consecutive tokens, value = the successor seen most often after them), and
// draft generation by chaining lookups on the most recent n-1 tokens, with the selective fallback (no
// drafts at all when the first lookup misses).  Everything stays on the GPU so that a verify loop never
// has to visit the host.
//
// Build, two passes over open-addressing hash tables (linear probing, capacities are powers of two at
// least twice the number of windows, so a probe always ends):
//   1. every window (t_1 .. t_n) is counted: find-or-insert its packed key with atomicCAS, atomicAdd;
//   2. every counted window offers (count, successor) to the entry of its prefix with a 64-bit
//      atomicMin of (~count << 32 | successor): most frequent successor, lowest token id on equal counts
//      (free slots are all ones, so one memset prepares keys and values alike).
// The result does not depend on thread order (where an entry sits in the table does; lookups do not).
#include "agx_internal.cuh"

namespace agx {

namespace {

constexpr int kTokenBits = 21;                       // token ids < 2^21 (2 M): three tokens fit 63 bits
constexpr unsigned long long kEmpty = ~0ull;         // no packed key has all 64 bits set

struct LutHeader {        // first 64 bytes of the table
    unsigned int capacity;  // slots, power of two
    int n;
    unsigned int entries;   // filled slots (diagnostic)
    unsigned int pad[13];
};
struct LutSlot {
    unsigned long long key;   // packed prefix, kEmpty when free
    unsigned long long best;  // (0xFFFFFFFF - count) << 32 | successor; all ones when free
};

__device__ __forceinline__ unsigned int hash64(unsigned long long k) {
    k ^= k >> 33; k *= 0xff51afd7ed558ccdull; k ^= k >> 33; k *= 0xc4ceb9fe1a85ec53ull; k ^= k >> 33;
    return (unsigned int)k;
}
__device__ __forceinline__ bool token_ok(int t) { return t >= 0 && t < (1 << kTokenBits); }

// find-or-insert `key` in keys[capacity]; returns the slot
__device__ __forceinline__ unsigned int claim(unsigned long long* keys, unsigned int stride_words, unsigned int capacity,
                                              unsigned long long key) {
    unsigned int s = hash64(key) & (capacity - 1);
    for (unsigned int probe = 0; probe < capacity; ++probe) {
        unsigned long long* slot = keys + (size_t)s * stride_words;
        const unsigned long long seen = atomicCAS(slot, kEmpty, key);
        if (seen == kEmpty || seen == key) return s;
        s = (s + 1) & (capacity - 1);
    }
    return capacity;  // cannot happen: the table is never more than half full
}

__global__ void ngram_count_kernel(const int* __restrict__ stream, int num_tokens, int n, unsigned long long* win_keys,
                                   unsigned int* win_counts, unsigned int win_capacity, int* status) {
    const int windows = num_tokens - n + 1;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < windows; i += gridDim.x * blockDim.x) {
        unsigned long long key = 0;
        bool ok = true;
        for (int j = 0; j < n; ++j) {
            const int t = stream[i + j];
            ok = ok && token_ok(t);
            key = (key << kTokenBits) | (unsigned long long)(unsigned int)(t & ((1 << kTokenBits) - 1));
        }
        if (!ok) { atomicOr(status, AGX_DEV_BAD_TOKEN); continue; }   // a window with a token outside [0, 2^21) is skipped
        const unsigned int s = claim(win_keys, 1, win_capacity, key);
        if (s < win_capacity) atomicAdd(win_counts + s, 1u);
    }
}

__global__ void ngram_select_kernel(const unsigned long long* __restrict__ win_keys, const unsigned int* __restrict__ win_counts,
                                    unsigned int win_capacity, LutSlot* lut, unsigned int lut_capacity) {
    for (unsigned int s = blockIdx.x * blockDim.x + threadIdx.x; s < win_capacity; s += gridDim.x * blockDim.x) {
        const unsigned long long key = win_keys[s];
        if (key == kEmpty) continue;
        const unsigned long long prefix = key >> kTokenBits;
        const unsigned int succ = (unsigned int)(key & ((1ull << kTokenBits) - 1));
        const unsigned int slot = claim(&lut[0].key, 2, lut_capacity, prefix);
        if (slot < lut_capacity)
            atomicMin(&lut[slot].best, ((unsigned long long)(0xFFFFFFFFu - win_counts[s]) << 32) | (unsigned long long)succ);
    }
}

__device__ __forceinline__ bool lut_find(const LutSlot* lut, unsigned int capacity, unsigned long long prefix, int& token) {
    unsigned int s = hash64(prefix) & (capacity - 1);
    for (unsigned int probe = 0; probe < capacity; ++probe) {
        const unsigned long long k = lut[s].key;
        if (k == prefix) { token = (int)(unsigned int)(lut[s].best & 0xFFFFFFFFull); return true; }
        if (k == kEmpty) return false;
        s = (s + 1) & (capacity - 1);
    }
    return false;
}

// One thread per sequence: k chained lookups on the last n-1 tokens.
__global__ void ngram_draft_kernel(const unsigned char* __restrict__ lut_mem, const int* __restrict__ context,
                                   const int* __restrict__ fill, int B, int k, int* __restrict__ drafts,
                                   int* __restrict__ has_draft) {
    const LutHeader* hdr = (const LutHeader*)lut_mem;
    const LutSlot* lut = (const LutSlot*)(lut_mem + sizeof(LutHeader));
    const unsigned int capacity = hdr->capacity;
    const int m = hdr->n - 1;   // tokens in a key: 1 or 2
    for (int s = blockIdx.x * blockDim.x + threadIdx.x; s < B; s += gridDim.x * blockDim.x) {
        int c0 = m == 2 ? context[s * 2] : 0, c1 = context[s * m + (m - 1)];
        bool first = true, hit_first = false;
        for (int i = 0; i < k; ++i) {
            int tok = 0;
            const bool ctx_ok = token_ok(c1) && (m == 1 || token_ok(c0));
            const unsigned long long prefix = m == 2 ? (((unsigned long long)(unsigned int)c0 << kTokenBits) | (unsigned int)c1)
                                                     : (unsigned long long)(unsigned int)c1;
            const bool hit = ctx_ok && capacity != 0 && lut_find(lut, capacity, prefix, tok);
            if (first) { hit_first = hit; first = false; }
            if (!hit) tok = fill[(size_t)s * k + i];   // the caller's guess for a context the table does not know
            drafts[(size_t)s * k + i] = tok;
            c0 = c1; c1 = tok;
        }
        has_draft[s] = (k > 0 && hit_first) ? 1 : 0;   // 0: fall back to a plain one-token step
        if (k == 0) {
            int tok;
            const bool ctx_ok = token_ok(c1) && (m == 1 || token_ok(c0));
            const unsigned long long prefix = m == 2 ? (((unsigned long long)(unsigned int)c0 << kTokenBits) | (unsigned int)c1)
                                                     : (unsigned long long)(unsigned int)c1;
            has_draft[s] = (ctx_ok && capacity != 0 && lut_find(lut, capacity, prefix, tok)) ? 1 : 0;
        }
    }
}

__global__ void ngram_header_kernel(LutHeader* hdr, unsigned int capacity, int n) {
    hdr->capacity = capacity; hdr->n = n; hdr->entries = 0;
}

unsigned int pow2_at_least(long long v) {
    unsigned int c = 16;
    while ((long long)c < v) c <<= 1;
    return c;
}

}  // namespace

long long ngram_lut_bytes(int max_stream_tokens) {
    return (long long)sizeof(LutHeader) + (long long)pow2_at_least(2ll * max_stream_tokens) * (long long)sizeof(LutSlot);
}
long long ngram_workspace_bytes(int stream_tokens) {
    return (long long)pow2_at_least(2ll * stream_tokens) * 12ll + 256;
}

cudaError_t launch_ngram_build(const int* stream_tokens, int num_tokens, int n, void* lut, void* workspace, int* status,
                               cudaStream_t stream) {
    const unsigned int cap = pow2_at_least(2ll * num_tokens);
    LutHeader* hdr = (LutHeader*)lut;
    LutSlot* slots = (LutSlot*)((unsigned char*)lut + sizeof(LutHeader));
    unsigned long long* win_keys = (unsigned long long*)workspace;
    unsigned int* win_counts = (unsigned int*)((unsigned char*)workspace + (size_t)cap * 8);
    // free slots are all ones (keys and values alike); counts start at zero
    cudaError_t e = cudaMemsetAsync(win_keys, 0xFF, (size_t)cap * 8, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(win_counts, 0, (size_t)cap * 4, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(slots, 0xFF, (size_t)cap * sizeof(LutSlot), stream);
    if (e != cudaSuccess) return e;
    ngram_header_kernel<<<1, 1, 0, stream>>>(hdr, cap, n);
    const int windows = num_tokens - n + 1;
    if (windows > 0) {
        const int blocks = (windows + 255) / 256 < 1184 ? (windows + 255) / 256 : 1184;
        ngram_count_kernel<<<blocks, 256, 0, stream>>>(stream_tokens, num_tokens, n, win_keys, win_counts, cap, status);
        const int blocks2 = (int)((cap + 255) / 256 < 1184 ? (cap + 255) / 256 : 1184);
        ngram_select_kernel<<<blocks2, 256, 0, stream>>>(win_keys, win_counts, cap, slots, cap);
    }
    return cudaGetLastError();
}

cudaError_t launch_ngram_draft(const void* lut, const int* context, const int* fill, int B, int k, int* drafts,
                               int* has_draft, cudaStream_t stream) {
    if (B == 0) return cudaSuccess;
    ngram_draft_kernel<<<(B + 127) / 128, 128, 0, stream>>>((const unsigned char*)lut, context, fill, B, k, drafts, has_draft);
    return cudaGetLastError();
}

}  // namespace agx
