// Internal declarations shared by the agx CUDA sources (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "agx.h"

namespace agx {

constexpr int kPage = 16;          // tokens per KV page
constexpr int kMaxSeqs = 48;       // sequences per attention launch (plans travel as kernel arguments)
constexpr int kSmallRowsMax = 64;  // q_len * G above this goes to the tile kernel
constexpr long long kWaitLimitCycles = 4000000000ll;  // ~2 s at 1.9 GHz: default limit of every in-kernel wait

// 2-D TMA view of a KV pool: [num_pages * Hkv * 16 rows][128 dims] bf16, box = 16 rows x 64 dims, SWIZZLE_128B.
bool make_pool_map(CUtensorMap* map, const void* pool, long long num_pages, int hkv);

// Per-sequence launch plan, built on the host from the host lengths.
struct SeqPlan {
    int prefix_len;    // P
    int q_len;         // q
    int q_row0;        // first row of the sequence in q_block / out
    int seq_index;     // row of the page table
    int nsplit;        // KV splits
    int row_chunks;    // query-row chunks per KV head (1 for verify blocks)
    int split_tokens;  // tokens per split (multiple of the kernel's KV tile)
    int item0;         // first work item of this sequence in the launch
    int part_base;     // first partial entry; entry = part_base + (i*Hq + h)*nsplit + split
};

struct AttnParams {
    const void* q;
    const void* k_pool;
    const void* v_pool;
    const int* page_table;
    void* out;
    float* lse;
    float* part_o;   // [entries][head_dim] fp32, un-normalised, relative to part_ml.x; or, with part_half, rows NORMALISED by their
                     // own sum and stored as fp16 in the first 256 bytes of the same 512-byte slots
    float2* part_ml; // [entries] (running max in log2 units, sum)
    int* status;
    unsigned long long row_div_magic;   // ceil(2^32 / G), G = hq / hkv: (row * magic) >> 32 == row / G for rows < 2^22
    int part_half;       // != 0: split partials of this launch are normalised fp16 rows (256-row tensor-core schedule)
    int cluster_size;    // > 1: the launch's CTAs form clusters of this size = the KV splits of one (sequence, KV head), merged in-kernel
    const void* k_new;   // fused append (agx_attn_prefixed_append): the block's K/V rows [total_q][hkv][d], or NULL
    const void* v_new;
    long long num_pages;
    int pt_stride;
    int hq, hkv, head_dim;
    int num_seqs;
    int num_items;
    float scale_log2;  // scale * log2(e)
    long long wait_limit_cycles;   // every in-kernel wait gives up after this many clock64 ticks (agx_set_option)
    int early_prefix;    // != 0: page ids and K/V tiles that lie wholly inside the cached prefix may be fetched before the
                         // dependency wait (the caller vouches that no launch still in flight writes them)
    int drop_stage;      // test hook: the producer leaves this K/V stage (tile) out, so its consumers' waits run out; -1 = none
    SeqPlan seq[kMaxSeqs];
};

// Launch with programmatic stream serialisation: the kernel may start while the launch before it in the
// stream is still draining, so its launch latency and set-up overlap that kernel's tail.  Every kernel
// launched this way calls pdl_wait() before its first global-memory access.  AGX_NO_PDL=1 turns it off.
bool pdl_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// The same with thread-block clusters of `cluster` CTAs along x (grid.x a multiple of it).
template <typename... KArgs, typename... Args>
cudaError_t launch_chained_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster,
                                   cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Lengths of a batch of at most kMaxSeqs sequences, passed to write_meta_kernel by value.
struct StepMeta {
    int B;
    int prefix[kMaxSeqs];
    int cu[kMaxSeqs + 1];
};
cudaError_t launch_write_meta(const StepMeta& m, int* prefix, int* seq_lens, int* cu_q, cudaStream_t stream);

// Up to three copies of 16-byte units by one kernel (sources may be pinned host memory mapped into the device's
// address space: a few hundred KB cross faster this way than as separate copy-engine transfers).
struct StageCopies {
    const uint4* src[3];
    uint4* dst[3];
    unsigned units[3];
};
cudaError_t launch_stage_in(const StageCopies& c, cudaStream_t stream);

// Append of the launch's sequences with the plans taken from the kernel arguments (no device-side lengths needed).
cudaError_t launch_kv_append_plan(const AttnParams& p, int dtype, int total_rows, cudaStream_t stream);

// Launchers (each returns the cudaError_t of its launch).
cudaError_t launch_kv_append(int dtype, void* k_pool, void* v_pool, long long num_pages, const void* k_new,
                             const void* v_new, const int* page_table, int pt_stride, const int* prefix_len,
                             const int* cu_q, int B, int total_q, int hkv, int head_dim, int* status,
                             cudaStream_t stream);

// Small-q split-KV kernel (bf16, d = 128, tensor-core mma.sync); mt = m-tiles of 16 rows (1, 2, 4), kw = KV groups
// (4 or 8 pages per pipeline stage; 8 only with mt <= 2): CTA = 32 * mt * kw threads.
// Clusters of `cluster` CTAs of the small-q kernel <mt, kw> that can be resident at once on the current device
// (0 when such a cluster cannot be launched); cached per device.
int attn_small_max_clusters(int mt, int kw, int cluster);
cudaError_t launch_attn_small_bf16(const AttnParams& p, int mt, int kw, const CUtensorMap& map_k, const CUtensorMap& map_v,
                                   cudaStream_t stream);
// Scalar fp32-math kernel for AGX_F32 pools (any q, d in {64, 128}) and for AGX_BF16 pools with d = 64.
cudaError_t launch_attn_simt(const AttnParams& p, int dtype, cudaStream_t stream);
// Merge of split partials into out / lse.
cudaError_t launch_attn_combine(const AttnParams& p, int dtype, int total_rows, cudaStream_t stream);   // honours p.part_half

// Tensor-core tile kernel (bf16, d = 128, tcgen05 + TMEM + TMA).  streams = false: 256 query rows per CTA
// (two Q tiles); streams = true: 128 rows per CTA whose KV tiles alternate between two softmax warpgroups
// (verify blocks and short suffixes over long contexts).
cudaError_t launch_attn_tile_bf16(const AttnParams& p, bool streams, const CUtensorMap& map_k, const CUtensorMap& map_v,
                                  cudaStream_t stream);

cudaError_t launch_accept(const void* logits, int logits_dtype, long long row_stride, int vocab, const int* drafts,
                          const int* cu_q, int B, int total_q, int* accept_len, int* next_token, int* argmax,
                          int* seq_lens, unsigned long long* row_keys, int* tokens_global, int chunks, unsigned int* ticket,
                          cudaStream_t stream);

// Private copies of KV pages (a reused prefix that is cut inside a page, Sec. 4.2).
cudaError_t launch_copy_pages(int dtype, void* k_pool, void* v_pool, long long num_pages, const int* src, const int* dst,
                              int count, int hkv, int head_dim, int* status, cudaStream_t stream);

cudaError_t launch_scatter_pages(int dtype, void* k_pool, void* v_pool, long long num_pages, const void* k_stage,
                                 const void* v_stage, const int* dst, int count, int hkv, int head_dim, int* status,
                                 cudaStream_t stream);

// n-gram draft table (Sec. 4.3): sizes, build (three memsets + three small kernels) and chained lookups.
long long ngram_lut_bytes(int max_stream_tokens);
long long ngram_workspace_bytes(int stream_tokens);
cudaError_t launch_ngram_build(const int* stream_tokens, int num_tokens, int n, void* lut, void* workspace, int* status,
                               cudaStream_t stream);
cudaError_t launch_ngram_draft(const void* lut, const int* context, const int* fill, int B, int k, int* drafts,
                               int* has_draft, cudaStream_t stream);

}  // namespace agx
