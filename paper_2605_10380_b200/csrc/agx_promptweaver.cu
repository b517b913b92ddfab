// The prompt-rewriting half of the method as far as it touches the KV cache (Sec. 4.2):
//   * Algorithm 1 - which cluster combinations to precompute under a budget (host code: a few thousand
//     short sequences, run once offline);
//   * the online lookup - the stored combination that shares the longest run of leading clusters with a
//     request, the mismatched tail of the stored one being cut off;
//   * bringing stored KV pages from host memory into the pool (two large copies into a staging area, one
//     scatter kernel), on whatever stream the caller chooses so that it overlaps attention elsewhere;
//   * the page copy a cut needs: a reused prefix that ends inside a page shares the full pages before it
//     and gets a private copy of that last page, so that the new sequence can append behind the cut.
#include <algorithm>
#include <map>
#include <vector>

#include "agx_internal.cuh"
#include "agx_sm100.cuh"

namespace agx {

// One CTA per (page pair, K or V): 16-byte loads and stores over the whole page (all KV heads).
__global__ void __launch_bounds__(256)
copy_pages_kernel(uint4* __restrict__ k_pool, uint4* __restrict__ v_pool, long long num_pages, const int* __restrict__ src,
                  const int* __restrict__ dst, long long vec_per_page, int* status) {
    pdl_launch_dependents();
    pdl_wait();
    const int pair = blockIdx.x >> 1;
    uint4* pool = (blockIdx.x & 1) ? v_pool : k_pool;
    const long long s = src[pair], d = dst[pair];
    if (s < 0 || s >= num_pages || d < 0 || d >= num_pages) {
        if (threadIdx.x == 0) atomicOr(status, AGX_DEV_BAD_PAGE);
        return;
    }
    if (s == d) return;
    for (long long i = threadIdx.x; i < vec_per_page; i += blockDim.x) pool[d * vec_per_page + i] = pool[s * vec_per_page + i];
}

// Scatter pages from a packed staging area (page i of the import) to pool pages dst[i]: one CTA per (page, K or V).
__global__ void __launch_bounds__(256)
scatter_pages_kernel(uint4* __restrict__ k_pool, uint4* __restrict__ v_pool, long long num_pages, const uint4* __restrict__ k_stage,
                     const uint4* __restrict__ v_stage, const int* __restrict__ dst, long long vec_per_page, int* status) {
    pdl_launch_dependents();
    pdl_wait();
    const int i = blockIdx.x >> 1;
    const bool is_v = blockIdx.x & 1;
    const long long d = dst[i];
    if (d < 0 || d >= num_pages) {
        if (threadIdx.x == 0) atomicOr(status, AGX_DEV_BAD_PAGE);
        return;
    }
    uint4* pool = is_v ? v_pool : k_pool;
    const uint4* stage = is_v ? v_stage : k_stage;
    for (long long j = threadIdx.x; j < vec_per_page; j += blockDim.x) pool[d * vec_per_page + j] = stage[(long long)i * vec_per_page + j];
}

cudaError_t launch_scatter_pages(int dtype, void* k_pool, void* v_pool, long long num_pages, const void* k_stage,
                                 const void* v_stage, const int* dst, int count, int hkv, int head_dim, int* status,
                                 cudaStream_t stream) {
    if (count == 0) return cudaSuccess;
    const long long vec_per_page = (long long)hkv * kPage * head_dim * (dtype == AGX_BF16 ? 2 : 4) / 16;
    return launch_chained(scatter_pages_kernel, dim3(2 * count), dim3(256), 0, stream, (uint4*)k_pool, (uint4*)v_pool, num_pages,
                          (const uint4*)k_stage, (const uint4*)v_stage, dst, vec_per_page, status);
}

cudaError_t launch_copy_pages(int dtype, void* k_pool, void* v_pool, long long num_pages, const int* src, const int* dst,
                              int count, int hkv, int head_dim, int* status, cudaStream_t stream) {
    if (count == 0) return cudaSuccess;
    const long long vec_per_page = (long long)hkv * kPage * head_dim * (dtype == AGX_BF16 ? 2 : 4) / 16;
    return launch_chained(copy_pages_kernel, dim3(2 * count), dim3(256), 0, stream, (uint4*)k_pool, (uint4*)v_pool, num_pages,
                          src, dst, vec_per_page, status);
}

}  // namespace agx

extern "C" {

AGX_API agx_status agx_pw_select_combinations(const int32_t* samples, int32_t num_samples, int32_t max_len, int32_t budget,
                                              int32_t* selected, int32_t* selected_len, int32_t* gains,
                                              int32_t* num_selected) {
    if (!num_selected || num_samples < 0 || max_len < 1 || budget < 0) return AGX_E_INVAL;
    *num_selected = 0;
    if (num_samples == 0 || budget == 0) return AGX_OK;
    if (!samples || !selected || !selected_len) return AGX_E_INVAL;
    typedef std::vector<int32_t> Seq;
    std::map<Seq, int32_t> count;   // every prefix of every sample -> number of samples that start with it
    for (int s = 0; s < num_samples; ++s) {
        Seq p;
        for (int i = 0; i < max_len; ++i) {
            const int32_t c = samples[(size_t)s * max_len + i];
            if (c < 0) break;
            p.push_back(c);
            ++count[p];
        }
    }
    // The cached set stays prefix-closed, so adding a candidate p (a single cluster, or a cached sequence plus one
    // cluster) raises the coverage by exactly the number of samples that start with p.
    std::map<Seq, bool> cached;
    for (int step = 0; step < budget; ++step) {
        const Seq* best = nullptr;
        int32_t best_gain = -1;
        for (const auto& kv : count) {
            const Seq& p = kv.first;
            if (cached.count(p)) continue;
            if (p.size() > 1 && !cached.count(Seq(p.begin(), p.end() - 1))) continue;
            // equal gains: the shorter candidate, then the lexicographically smaller one
            const bool better = kv.second > best_gain ||
                                (kv.second == best_gain && (p.size() < best->size() || (p.size() == best->size() && p < *best)));
            if (better) { best = &p; best_gain = kv.second; }
        }
        if (!best) break;
        cached[*best] = true;
        int32_t* out = selected + (size_t)step * max_len;
        for (int i = 0; i < max_len; ++i) out[i] = i < (int)best->size() ? (*best)[i] : -1;
        selected_len[step] = (int32_t)best->size();
        if (gains) gains[step] = best_gain;
        *num_selected = step + 1;
    }
    return AGX_OK;
}

AGX_API agx_status agx_pw_longest_prefix(const int32_t* stored, const int32_t* stored_len, int32_t num_stored, int32_t max_len,
                                         const int32_t* query, int32_t query_len, int32_t* index, int32_t* length) {
    if (!index || !length || num_stored < 0 || max_len < 1 || query_len < 0) return AGX_E_INVAL;
    *index = -1; *length = 0;
    if (num_stored == 0 || query_len == 0) return AGX_OK;
    if (!stored || !stored_len || !query) return AGX_E_INVAL;
    for (int i = 0; i < num_stored; ++i) {
        const int n_max = std::min(std::min(stored_len[i], max_len), query_len);
        int n = 0;
        while (n < n_max && stored[(size_t)i * max_len + n] == query[n]) ++n;
        if (n > *length) { *index = i; *length = n; }
    }
    return AGX_OK;
}

}  // extern "C"
