// KV append: scatter the block's K/V rows into the sequences' pages (Sec. 2.3: prefill fills the
// KV cache; with prefix caching only the uncached suffix is written, behind the cached prefix).
//
// HBM-bound copy: 2 * 2 * rows * Hkv * d * elem bytes (read + write, K and V).  One thread moves
// 16 bytes of K and 16 bytes of V; a (token, kv head) row is `vec_per_row` consecutive threads, so
// loads and stores are fully coalesced 128-bit accesses.
#include <stdlib.h>

#include <algorithm>

#include "agx_internal.cuh"
#include "agx_sm100.cuh"

namespace agx {

__global__ void __launch_bounds__(256)
kv_append_kernel(uint4* __restrict__ k_pool, uint4* __restrict__ v_pool, long long num_pages,
                 const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                 const int* __restrict__ page_table, int pt_stride, const int* __restrict__ prefix_len,
                 const int* __restrict__ cu_q, int B, int total_q, int hkv, int vec_per_row, int* status) {
    pdl_launch_dependents();
    pdl_wait();
    const long long n_vec = (long long)total_q * hkv * vec_per_row;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n_vec;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % vec_per_row);
        const long long row = idx / vec_per_row;  // (token, kv head)
        const int g = (int)(row % hkv);
        const int r = (int)(row / hkv);           // row of k_new
        // sequence of row r: last s with cu_q[s] <= r
        int lo = 0, hi = B;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(cu_q + mid) <= r) lo = mid; else hi = mid;
        }
        const int s = lo;
        const int tok = __ldg(prefix_len + s) + (r - __ldg(cu_q + s));
        const int page_slot = tok / kPage;
        long long page = -1;
        if (tok >= 0 && page_slot < pt_stride) page = __ldg(page_table + (long long)s * pt_stride + page_slot);
        if (page < 0 || page >= num_pages) {
            if (c == 0 && g == 0) atomicOr(status, AGX_DEV_BAD_PAGE);
            continue;
        }
        const long long dst = (((page * hkv + g) * kPage) + (tok % kPage)) * vec_per_row + c;
        k_pool[dst] = k_new[idx];
        v_pool[dst] = v_new[idx];
    }
}

cudaError_t launch_kv_append(int dtype, void* k_pool, void* v_pool, long long num_pages, const void* k_new,
                             const void* v_new, const int* page_table, int pt_stride, const int* prefix_len,
                             const int* cu_q, int B, int total_q, int hkv, int head_dim, int* status,
                             cudaStream_t stream) {
    const int esz = dtype == AGX_BF16 ? 2 : 4;
    const int vec_per_row = head_dim * esz / 16;
    const long long n_vec = (long long)total_q * hkv * vec_per_row;
    if (n_vec == 0) return cudaSuccess;
    long long blocks = (n_vec + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    return launch_chained(kv_append_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, (uint4*)k_pool, (uint4*)v_pool, num_pages,
                          (const uint4*)k_new, (const uint4*)v_new, page_table, pt_stride, prefix_len, cu_q, B, total_q, hkv,
                          vec_per_row, status);
}

// The same scatter for the sequences of one attention launch, lengths and row offsets taken from the launch's plans.
__global__ void __launch_bounds__(256)
kv_append_plan_kernel(const __grid_constant__ AttnParams p, int vec_per_row, int total_rows) {
    pdl_launch_dependents();
    pdl_wait();
    const long long n_vec = (long long)total_rows * p.hkv * vec_per_row;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n_vec; idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % vec_per_row);
        const long long row = idx / vec_per_row;
        const int g = (int)(row % p.hkv);
        int lr = (int)(row / p.hkv);   // row within the launch: sequences back to back
        int si = 0;
        while (si + 1 < p.num_seqs && lr >= p.seq[si].q_len) { lr -= p.seq[si].q_len; ++si; }
        const SeqPlan& sp = p.seq[si];
        const int tok = sp.prefix_len + lr;
        const long long page = (tok >> 4) < p.pt_stride ? __ldg(p.page_table + (long long)sp.seq_index * p.pt_stride + (tok >> 4)) : -1;
        if (page < 0 || page >= p.num_pages) { if (c == 0 && g == 0) atomicOr(p.status, AGX_DEV_BAD_PAGE); continue; }
        const long long src = ((long long)(sp.q_row0 + lr) * p.hkv + g) * vec_per_row + c;
        const long long dst = ((page * p.hkv + g) * kPage + (tok & 15)) * vec_per_row + c;
        ((uint4*)p.k_pool)[dst] = ((const uint4*)p.k_new)[src];
        ((uint4*)p.v_pool)[dst] = ((const uint4*)p.v_new)[src];
    }
}

cudaError_t launch_kv_append_plan(const AttnParams& p, int dtype, int total_rows, cudaStream_t stream) {
    const int vec_per_row = p.head_dim * (dtype == AGX_BF16 ? 2 : 4) / 16;
    const long long n_vec = (long long)total_rows * p.hkv * vec_per_row;
    if (n_vec == 0) return cudaSuccess;
    long long blocks = (n_vec + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    return launch_chained(kv_append_plan_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, p, vec_per_row, total_rows);
}

// Lengths of a small batch travel as kernel arguments instead of three pageable host-to-device copies (each
// of which would first synchronise the stream): prefix_len, the committed lengths and the row offsets.
__global__ void write_meta_kernel(const __grid_constant__ StepMeta m, int* prefix, int* seq_lens, int* cu_q) {
    pdl_launch_dependents();
    pdl_wait();
    const int i = threadIdx.x;
    if (i < m.B) { prefix[i] = m.prefix[i]; seq_lens[i] = m.prefix[i]; }
    if (i <= m.B) cu_q[i] = m.cu[i];
}

cudaError_t launch_write_meta(const StepMeta& m, int* prefix, int* seq_lens, int* cu_q, cudaStream_t stream) {
    return launch_chained(write_meta_kernel, dim3(1), dim3(64), 0, stream, m, prefix, seq_lens, cu_q);
}

__global__ void __launch_bounds__(256) stage_in_kernel(const StageCopies c) {
    pdl_launch_dependents();
    pdl_wait();   // the launch before this one may still read the destination
    const unsigned n0 = c.units[0], n1 = n0 + c.units[1], n2 = n1 + c.units[2];
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < n2; i += gridDim.x * blockDim.x) {
        const int k = i < n0 ? 0 : i < n1 ? 1 : 2;
        const unsigned j = i - (k == 0 ? 0u : k == 1 ? n0 : n1);
        c.dst[k][j] = c.src[k][j];
    }
}

cudaError_t launch_stage_in(const StageCopies& c, cudaStream_t stream) {
    const unsigned n = c.units[0] + c.units[1] + c.units[2];
    if (n == 0) return cudaSuccess;
    const unsigned blocks = std::min(1024u, (n + 255u) / 256u);
    return launch_chained(stage_in_kernel, dim3(blocks), dim3(256), 0, stream, c);
}

bool pdl_enabled() {
    static const bool on = [] { const char* e = getenv("AGX_NO_PDL"); return !(e && atoi(e) != 0); }();
    return on;
}

}  // namespace agx
