// C ABI of the agx library: argument checks, launch planning, dispatch.  No kernel lives here.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <unordered_map>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "agx_internal.cuh"

namespace {
// An NVTX range around every call that enqueues work: a timeline tool shows the library's calls by name; with no tool
// attached a range costs a few nanoseconds.
struct CallRange {
    explicit CallRange(const char* name) { nvtxRangePushA(name); }
    ~CallRange() { nvtxRangePop(); }
};
struct Plan;
// TMA view of one KV pool, kept per pool address: encoding a tensor map costs about as much host time as a launch.
struct PoolMap {
    alignas(64) CUtensorMap map;
    long long num_pages;
    int hkv;
};
}  // namespace

struct agx_handle {
    agx_config cfg;
    float scale;
    int device;
    int sm_count;
    int* d_status;          // device status word
    unsigned int* d_ticket; // ticket counter of the accept kernel (self-resetting)
    unsigned long long* d_row_keys;   // one argmax key per logits row of the accept kernel (all zero between launches)
    int last_launches;
    int small_min_split;    // tokens; tuning knob (env AGX_SMALL_MIN_SPLIT)
    int force_mma_sync;     // route large q through the mma.sync kernel (env AGX_FORCE_MMA_SYNC)
    int debug_plan;         // print launch plans to stderr (env AGX_DEBUG_PLAN)
    int small_kw;           // pages per pipeline stage of the warp-MMA kernel: 4, 8, or 0 = chosen per batch (env AGX_SMALL_KW)
    int batch_stream_tokens; // total tokens of a batch's small blocks from which they all take the stream schedule (env AGX_BATCH_STREAM_TOKENS)
    bool longest_first;     // sequences of a launch ordered by decreasing context length (env AGX_LONGEST_FIRST=0: batch order)
    bool merge_sms;         // one-wave small-q launches leave SMs free for their merge kernel (env AGX_MERGE_SMS=0 turns it off)
    bool cluster_merge;     // KV splits of the small-q kernel merged inside thread-block clusters where the batch allows (env AGX_CLUSTER_MERGE=0 turns it off)
    int zero_copy;          // host steps: bit 0 = kernels read small pinned inputs, bit 1 = kernels write `out` into a pinned buffer (env AGX_ZERO_COPY, default 3)
    int stream_max_rows;    // blocks of up to this many rows per KV head may take the one-Q-tile schedule in 128-row chunks (env AGX_STREAM_MAX_ROWS)
    int stream_min_tokens;  // context length from which blocks of <= 32 rows take the tensor-core stream schedule (env AGX_STREAM_MIN_TOKENS; -1 = by block height)
    long long wait_limit_cycles;   // AGX_OPT_WAIT_LIMIT_CYCLES
    int early_prefix;       // AGX_OPT_EARLY_PREFIX_LOADS
    int drop_stage;         // AGX_OPT_TEST_DROP_STAGE (-1 = none)
    std::unordered_map<const void*, PoolMap> pool_maps;
    std::vector<int32_t> cu_host;  // staging for agx_verify_step_host (lives until its final sync)
    // Large attention-only host steps run as a pipeline of row chunks: uploads on one stream of the handle's own, the
    // attention calls on the caller's stream, downloads on a third (env AGX_HOST_PIPELINE_ROWS: rows per chunk, 0 = off).
    int pipe_rows;
    cudaStream_t pipe_in, pipe_out;
    std::vector<cudaEvent_t> pipe_events;
    // the launch plan of the last batch seen: the layers of a model step all ask for the same one
    Plan* plan_cache;
    std::vector<int32_t> plan_P, plan_Q;
    char err[512];
};

namespace {

using namespace agx;

agx_status fail(agx_handle* h, agx_status code, const char* fmt, ...) {
    if (h) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(h->err, sizeof h->err, fmt, ap);
        va_end(ap);
    }
    return code;
}

agx_status cuda_fail(agx_handle* h, cudaError_t e, const char* what) {
    return fail(h, AGX_E_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

// The handle's tensor map of a pool (encoded on first use of that address with that geometry).
const CUtensorMap* pool_map(agx_handle* h, const void* pool, long long num_pages, int hkv) {
    auto it = h->pool_maps.find(pool);
    if (it != h->pool_maps.end() && it->second.num_pages == num_pages && it->second.hkv == hkv) return &it->second.map;
    if (h->pool_maps.size() >= 4096) h->pool_maps.clear();
    PoolMap& pm = h->pool_maps[pool];
    pm.num_pages = -1;
    if (!make_pool_map(&pm.map, pool, num_pages, hkv)) { h->pool_maps.erase(pool); return nullptr; }
    pm.num_pages = num_pages;
    pm.hkv = hkv;
    return &pm.map;
}
inline int round_up(long long v, int m) { return (int)((v + m - 1) / m * m); }
inline int elem_size(int dtype) { return dtype == AGX_BF16 ? 2 : 4; }

enum Kind { KIND_SMALL1 = 0, KIND_SMALL2, KIND_SMALL4, KIND_STREAM, KIND_TILE, KIND_SIMT, KIND_COUNT };

struct Launch {
    Kind kind;
    int total_rows;  // sum of q_len over the launch's sequences
    int num_items;
    int kw;          // small-q kernel: pages per pipeline stage (KV groups), 4 or 8
    int cluster;     // > 1: CTAs per cluster = KV splits of every sequence of the launch, merged in-kernel (no partials)
    bool lean_merge; // small-q kernel or one-Q-tile schedule: fp16 partials, merged by the two-warp merge kernel on SMs left out of the attention grid
    std::vector<SeqPlan> seqs;
};

struct Plan {
    std::vector<Launch> launches;
    long long part_entries = 0;  // (row, head, split) partial slots
    bool any_split = false;
};

// Decide kernel kind, KV splits and partial slots for every sequence (host lengths only).
agx_status build_plan(agx_handle* h, int B, const int32_t* P, const int32_t* Q, int pt_stride, Plan& plan) {
    const agx_config& c = h->cfg;
    const int G = c.num_q_heads / c.num_kv_heads;
    std::vector<int> row0(B + 1, 0);
    for (int s = 0; s < B; ++s) {
        if (Q[s] < 1) return fail(h, AGX_E_INVAL, "q_len[%d] = %d < 1", s, Q[s]);
        if (P[s] < 0) return fail(h, AGX_E_INVAL, "prefix_len[%d] = %d < 0", s, P[s]);
        if (pt_stride >= 0 && (long long)P[s] + Q[s] > (long long)pt_stride * kPage)
            return fail(h, AGX_E_RANGE, "sequence %d: %d + %d tokens exceed the page table (%d pages)", s, P[s], Q[s], pt_stride);
        if ((long long)row0[s] + Q[s] > (1 << 30)) return fail(h, AGX_E_RANGE, "too many rows");
        row0[s + 1] = row0[s] + Q[s];
    }
    // Blocks of at most 32 rows: measured on B200 (GQA 32/8, equal sequences), what decides is the batch's total
    // context, not each sequence's: from ~24k tokens in all (two sequences or more) the tensor-core stream schedule
    // wins whatever the single lengths; below that the warp-MMA kernel, with 4-page stages and two CTAs per SM from
    // ~8k tokens in all, with 8-page stages (one 16-warp CTA per SM) for less.  A single sequence keeps its own
    // cross-over (stream_min_tokens).
    long long small_tokens = 0;
    int small_seqs = 0;
    const bool scalar_path = c.dtype == AGX_F32 || c.head_dim != 128;   // fp32 pools, and bf16 with head_dim 64
    if (!scalar_path)
        for (int s = 0; s < B; ++s)
            if (Q[s] * G <= 32) { small_tokens += P[s] + Q[s]; ++small_seqs; }
    small_tokens = small_tokens * c.num_kv_heads / 8;   // the thresholds were measured with 8 KV heads: scale to the same bytes
    const bool batch_streams = small_seqs >= 2 && small_tokens >= h->batch_stream_tokens;
    long long warp_mma_tokens = 0;
    int warp_mma_seqs = 0;
    std::vector<int> groups[KIND_COUNT];
    for (int s = 0; s < B; ++s) {
        Kind k;
        if (scalar_path) k = KIND_SIMT;
        else {
            const int rows = Q[s] * G;
            const bool tile_ok = !h->force_mma_sync;
            // up to 128 rows: one Q tile per CTA, KV tiles alternating between two softmax warpgroups (HBM-bound
            // streaming on the tcgen05 pipe); blocks of at most 32 rows over short contexts stay with the warp-MMA
            // kernel, whose fixed costs are lower (none above 32 rows)
            // cross-over of a single sequence (GQA 32/8): q = 8 near 7k tokens, q = 1 near 10k
            const int cross = h->stream_min_tokens >= 0 ? h->stream_min_tokens : (rows > 8 ? 7168 : 10240);
            if (tile_ok && rows <= h->stream_max_rows && (rows > 32 || batch_streams || P[s] + Q[s] >= cross)) k = KIND_STREAM;
            else if (rows <= 16) k = KIND_SMALL1;
            else if (rows <= 32) k = KIND_SMALL2;
            else if (rows <= kSmallRowsMax || h->force_mma_sync) k = KIND_SMALL4;
            else k = KIND_TILE;
            if (k == KIND_SMALL1 || k == KIND_SMALL2) { warp_mma_tokens += P[s] + Q[s]; ++warp_mma_seqs; }
        }
        groups[k].push_back(s);
    }
    const int small_kw = h->small_kw ? h->small_kw : (warp_mma_seqs >= 2 && warp_mma_tokens * c.num_kv_heads / 8 >= 8192) ? 4 : 8;
    // Work items are handed to the SMs in launch order: the sequences with the longest contexts go first, so that the
    // longest items of a ragged batch are not the ones left over for the last wave (env AGX_LONGEST_FIRST=0 keeps the batch order).
    if (h->longest_first)
        for (int k : {(int)KIND_TILE, (int)KIND_STREAM})
            std::stable_sort(groups[k].begin(), groups[k].end(), [&](int a, int b) { return P[a] + Q[a] > P[b] + Q[b]; });
    for (int k = 0; k < KIND_COUNT; ++k) {
        const std::vector<int>& seqs = groups[k];
        if (seqs.empty()) continue;
        // ---- choose the split length C (tokens) so that one wave of CTAs covers the group
        int unit, min_split, target;
        long long base_items = 0;  // items per split, summed over sequences
        std::vector<long long> per_seq_items(seqs.size());
        if (k == KIND_SIMT) { unit = 64; min_split = 256; target = h->sm_count * 16; }
        else if (k == KIND_TILE || k == KIND_STREAM) { unit = 128; min_split = k == KIND_TILE ? 128 : 256; target = h->sm_count; }
        else { unit = 16; min_split = h->small_min_split; target = h->sm_count * ((k == KIND_SMALL4 || small_kw == 8) ? 1 : 2); }
        const int rows_per_chunk = (k == KIND_SMALL1) ? 16 : (k == KIND_SMALL2) ? 32 : (k == KIND_SMALL4) ? 64 : (k == KIND_STREAM) ? 128 : 256;
        long long work = 0;
        for (size_t n = 0; n < seqs.size(); ++n) {
            const int s = seqs[n];
            long long items;
            if (k == KIND_SIMT) items = (long long)Q[s] * c.num_q_heads;
            else items = (long long)c.num_kv_heads * ((Q[s] * G + rows_per_chunk - 1) / rows_per_chunk);
            per_seq_items[n] = items;
            base_items += items;
            work += items * (P[s] + Q[s]);
        }
        int C = std::max(min_split, round_up((work + target - 1) / target, unit));
        // small-q kernel: when one wave of CTAs needs splits only a little shorter than the minimum, take them (the
        // headline decode-verify shape then fills 144 SMs with 18 splits of 240 tokens instead of 136 with 17 of 256)
        if (k != KIND_SIMT && k != KIND_TILE && k != KIND_STREAM && C == min_split &&
            round_up((work + target - 1) / target, unit) * 20 >= min_split * 17)
            C = round_up((work + target - 1) / target, unit);
        auto count_items = [&](int c_tokens) {
            long long items = 0;
            for (size_t n = 0; n < seqs.size(); ++n) {
                const int L = P[seqs[n]] + Q[seqs[n]];
                items += per_seq_items[n] * ((L + c_tokens - 1) / c_tokens);
            }
            return items;
        };
        if (k == KIND_TILE || k == KIND_STREAM) {
            // several waves are fine here: pick the split length with the smallest estimated makespan, in units of one KV
            // tile's time (~1.6 us): waves * (tiles per item + fixed per-CTA cost of ~3 tiles), plus what the split costs
            // afterwards: the merge launch (~2 units) and the partial rows written and read back (~0.3 units per MB beyond the
            // first 16 MB, which stay in L2; measured on a ragged batch of eight suffix prefills: 95 MB of partials cost 60 us
            // more than 22 MB, while 9 MB in one-tile splits of a 128-token suffix over 1000 tokens cost nothing)
            int max_len = 0;
            for (int s : seqs) max_len = std::max(max_len, P[s] + Q[s]);
            const long long row_bytes = k == KIND_TILE ? 256 : 520;   // fp16 row | fp32 row + (m, l)
            long long best_cost = -1;
            for (int c_tokens = min_split; c_tokens < max_len + unit; c_tokens += unit) {
                const long long waves = (count_items(c_tokens) + h->sm_count - 1) / h->sm_count;
                long long part_bytes = 0;
                for (int s : seqs) {
                    const long long ns = (P[s] + Q[s] + c_tokens - 1) / c_tokens;
                    if (ns > 1) part_bytes += (long long)Q[s] * c.num_q_heads * ns * row_bytes;
                }
                const long long cost = 16 * waves * (std::min(c_tokens, round_up(max_len, unit)) / unit + 3) +
                                       (part_bytes ? 32 + 5 * std::max<long long>(0, (part_bytes >> 20) - 16) : 0);
                if (best_cost < 0 || cost < best_cost) { best_cost = cost; C = c_tokens; }
            }
            if (const char* force = getenv("AGX_TILE_SPLIT_TOKENS")) { if (atoi(force) >= unit) C = atoi(force) / unit * unit; }
            if (h->debug_plan)
                fprintf(stderr, "agx plan: tile kernel, %lld row chunks, longest sequence %d tokens -> KV splits of %d tokens, %lld CTAs\n",
                        base_items, max_len, C, count_items(C));
        } else {
            while (count_items(C) > std::max<long long>(target, base_items)) C += unit;
        }
        // ---- small-q kernel: when every sequence has one row chunk and the same number of KV splits (2..16), the
        //      splits of a (sequence, KV head) form a thread-block cluster and are merged through distributed shared
        //      memory: no partials in global memory, no combine launch.  17..20 splits are squeezed into 16.
        int cluster = 0;
        if ((k == KIND_SMALL1 || k == KIND_SMALL2 || k == KIND_SMALL4) && h->cluster_merge && seqs.size() <= (size_t)kMaxSeqs) {
            int common = -1;
            bool ok = true;
            for (size_t n = 0; n < seqs.size() && ok; ++n) {
                const int L = P[seqs[n]] + Q[seqs[n]];
                int ns = (L + C - 1) / C;
                ns = (L + round_up((L + ns - 1) / ns, unit) - 1) / round_up((L + ns - 1) / ns, unit);
                if (ns > 16 && ns <= 20) ns = 16;
                ok = per_seq_items[n] == c.num_kv_heads && (common < 0 || ns == common);
                common = ns;
            }
            if (ok && common >= 2 && common <= 16) {
                const int mt = k == KIND_SMALL1 ? 1 : k == KIND_SMALL2 ? 2 : 4;
                const int fit = attn_small_max_clusters(mt, mt == 4 ? 4 : small_kw, common);
                if (fit >= base_items) cluster = common;
                if (h->debug_plan) fprintf(stderr, "agx plan: clusters of %d: %d fit the device, %lld needed\n", common, fit, base_items);
            }
        }
        // ---- small-q kernel, one wave of one CTA per SM, splits merged by the merge kernel: leave that kernel SMs of its own.
        //      An attention CTA takes a whole SM, so merge CTAs that find no free SM sit on SMs the next call's attention CTAs
        //      need, and those CTAs then start (and fetch their K/V) only after the merge instead of under it.  With a few SMs
        //      left out of the attention grid the merge CTAs are resident there from the start and the next call's grid
        //      follows this one without a gap.  A two-warp merge CTA handles two (row, head) pairs; 12 (up to 20 splits) or 8
        //      of them fit an SM.
        bool lean_merge = false;   // fp16 partials and the two-warp merge kernel (slower than fp32 partials and the four-warp
                                   // one where the attention grid fills every SM twice over, e.g. four verify blocks of 4096)
        const bool small_one_per_sm = (k == KIND_SMALL1 || k == KIND_SMALL2 || k == KIND_SMALL4) && (k == KIND_SMALL4 || small_kw == 8);
        // (the one-Q-tile tensor-core schedule as well: a single long sequence is one wave of whole-SM CTAs too)
        if (!cluster && (small_one_per_sm || k == KIND_STREAM) && seqs.size() <= (size_t)kMaxSeqs && h->merge_sms) {
            long long pairs = 0;
            for (int s : seqs) pairs += (long long)Q[s] * c.num_q_heads;
            for (;;) {
                const long long items = count_items(C);
                int ns_max = 1;
                for (int s : seqs) ns_max = std::max(ns_max, (P[s] + Q[s] + C - 1) / C);
                if (ns_max == 1 || items > h->sm_count) break;   // no merge, or more than one wave anyway
                const long long reserve = (pairs + (ns_max <= 20 ? 24 : 16) - 1) / (ns_max <= 20 ? 24 : 16);
                if (reserve > h->sm_count / 8) break;   // a merge that large needs the whole device anyway
                lean_merge = true;
                if (items <= h->sm_count - reserve || items <= base_items) break;
                C += unit;
            }
        }
        // ---- emit launches of at most kMaxSeqs sequences
        for (size_t a = 0; a < seqs.size(); a += kMaxSeqs) {
            Launch ln;
            ln.kind = (Kind)k;
            ln.total_rows = 0;
            ln.num_items = 0;
            ln.cluster = cluster;
            ln.lean_merge = lean_merge;
            ln.kw = (k == KIND_SMALL4) ? 4 : small_kw;
            for (size_t n = a; n < std::min(seqs.size(), a + kMaxSeqs); ++n) {
                const int s = seqs[n];
                const int L = P[s] + Q[s];
                SeqPlan sp;
                sp.prefix_len = P[s];
                sp.q_len = Q[s];
                sp.q_row0 = row0[s];
                sp.seq_index = s;
                sp.nsplit = (L + C - 1) / C;
                sp.split_tokens = round_up((L + sp.nsplit - 1) / sp.nsplit, unit);
                sp.nsplit = (L + sp.split_tokens - 1) / sp.split_tokens;
                if (cluster) { sp.nsplit = cluster; sp.split_tokens = round_up((L + cluster - 1) / cluster, kPage); }
                sp.row_chunks = (k == KIND_SIMT) ? 1 : (Q[s] * G + rows_per_chunk - 1) / rows_per_chunk;
                sp.item0 = ln.num_items;
                sp.part_base = 0;
                if (sp.nsplit > 1 && !cluster) {
                    if (plan.part_entries + (long long)Q[s] * c.num_q_heads * sp.nsplit > 0x7FFFFFFFll)
                        return fail(h, AGX_E_RANGE, "split partials exceed 2^31 entries");
                    sp.part_base = (int)plan.part_entries;
                    plan.part_entries += (long long)Q[s] * c.num_q_heads * sp.nsplit;
                    plan.any_split = true;
                }
                const long long items = per_seq_items[n] * sp.nsplit;
                if (ln.num_items + items > 0x7FFFFFFFll) return fail(h, AGX_E_RANGE, "too many work items");
                ln.num_items += (int)items;
                ln.total_rows += Q[s];
                ln.seqs.push_back(sp);
            }
            if (h->debug_plan && k != KIND_TILE && k != KIND_STREAM)
                fprintf(stderr, "agx plan: kind %d (stages of %d pages), %zu sequences, %d CTAs, first sequence %d splits of %d tokens%s\n", k,
                        ln.kw, ln.seqs.size(), ln.num_items, ln.seqs[0].nsplit, ln.seqs[0].split_tokens,
                        cluster ? ", merged in clusters" : "");
            plan.launches.push_back(std::move(ln));
        }
    }
    return AGX_OK;
}

// The plan for this batch: the cached one when the lengths are those of the last call on the handle.
agx_status make_plan(agx_handle* h, int B, const int32_t* P, const int32_t* Q, int pt_stride, const Plan*& out) {
    if (h->plan_cache && (int)h->plan_P.size() == B && memcmp(h->plan_P.data(), P, sizeof(int32_t) * B) == 0 &&
        memcmp(h->plan_Q.data(), Q, sizeof(int32_t) * B) == 0) {
        if (pt_stride >= 0)
            for (int s = 0; s < B; ++s)
                if ((long long)P[s] + Q[s] > (long long)pt_stride * kPage)
                    return fail(h, AGX_E_RANGE, "sequence %d: %d + %d tokens exceed the page table (%d pages)", s, P[s], Q[s], pt_stride);
        out = h->plan_cache;
        return AGX_OK;
    }
    if (!h->plan_cache) h->plan_cache = new (std::nothrow) Plan;
    if (!h->plan_cache) return fail(h, AGX_E_NOMEM, "out of host memory");
    h->plan_P.clear();   // (invalid while it is rebuilt)
    *h->plan_cache = Plan();
    agx_status st = build_plan(h, B, P, Q, pt_stride, *h->plan_cache);
    if (st != AGX_OK) return st;
    h->plan_P.assign(P, P + B);
    h->plan_Q.assign(Q, Q + B);
    out = h->plan_cache;
    return AGX_OK;
}

inline size_t part_ml_bytes(long long entries) { return (size_t)((entries * sizeof(float2) + 255) / 256 * 256); }

}  // namespace

extern "C" {

const char* agx_status_string(agx_status s) {
    switch (s) {
        case AGX_OK: return "ok";
        case AGX_E_INVAL: return "invalid argument";
        case AGX_E_RANGE: return "argument out of range";
        case AGX_E_UNSUPPORTED: return "unsupported configuration";
        case AGX_E_CUDA: return "CUDA error";
        case AGX_E_DEVICE: return "device status word set";
        case AGX_E_NOMEM: return "out of memory";
        default: return "unknown status";
    }
}

const char* agx_last_error(const agx_handle* h) { return h ? h->err : "null handle"; }

agx_status agx_create(const agx_config* cfg, agx_handle** out) {
    if (!cfg || !out) return AGX_E_INVAL;
    *out = nullptr;
    if (cfg->num_q_heads < 1 || cfg->num_kv_heads < 1 || cfg->num_q_heads % cfg->num_kv_heads != 0) return AGX_E_INVAL;
    if (cfg->page_size != kPage) return AGX_E_UNSUPPORTED;
    if (cfg->dtype != AGX_BF16 && cfg->dtype != AGX_F32) return AGX_E_UNSUPPORTED;
    if (cfg->dtype == AGX_BF16 && cfg->head_dim != 128 && cfg->head_dim != 64) return AGX_E_UNSUPPORTED;
    if (cfg->dtype == AGX_F32 && cfg->head_dim != 64 && cfg->head_dim != 128) return AGX_E_UNSUPPORTED;
    if (!(cfg->scale >= 0.f)) return AGX_E_INVAL;
    agx_handle* h = new (std::nothrow) agx_handle();
    if (!h) return AGX_E_NOMEM;
    h->cfg = *cfg;
    h->scale = cfg->scale > 0.f ? cfg->scale : 1.0f / sqrtf((float)cfg->head_dim);
    h->err[0] = 0;
    h->last_launches = 0;
    const char* env = getenv("AGX_SMALL_MIN_SPLIT");
    h->small_min_split = env ? std::max(64, atoi(env) / 64 * 64) : 256;
    env = getenv("AGX_FORCE_MMA_SYNC");
    h->force_mma_sync = env ? atoi(env) : 0;
    env = getenv("AGX_STREAM_MIN_TOKENS");
    h->stream_min_tokens = env ? atoi(env) : -1;   // -1: the measured cross-over, by block height
    env = getenv("AGX_STREAM_MAX_ROWS");
    h->stream_max_rows = env ? atoi(env) : 384;
    env = getenv("AGX_CLUSTER_MERGE");
    h->cluster_merge = !(env && atoi(env) == 0);
    env = getenv("AGX_HOST_PIPELINE_ROWS");
    h->pipe_rows = env ? std::max(0, atoi(env)) : 384;   // measured on the long-context step: 256 / 384 / 512 / 768 / 1024 rows -> 1.54 / 1.43 / 1.57 / 1.56 / 1.72 ms
    h->pipe_in = h->pipe_out = nullptr;
    env = getenv("AGX_LONGEST_FIRST");
    h->longest_first = !(env && atoi(env) == 0);
    env = getenv("AGX_MERGE_SMS");
    h->merge_sms = !(env && atoi(env) == 0);
    env = getenv("AGX_ZERO_COPY");
    h->zero_copy = env ? atoi(env) : 3;
    env = getenv("AGX_SMALL_KW");
    h->small_kw = (env && (atoi(env) == 4 || atoi(env) == 8)) ? atoi(env) : 0;
    env = getenv("AGX_BATCH_STREAM_TOKENS");   // (forcing the per-sequence cross-over also switches the batch rule off)
    h->batch_stream_tokens = env ? atoi(env) : getenv("AGX_STREAM_MIN_TOKENS") ? 0x7FFFFFFF : 24576;
    env = getenv("AGX_DEBUG_PLAN");
    h->debug_plan = env ? atoi(env) : 0;
    h->wait_limit_cycles = kWaitLimitCycles;
    env = getenv("AGX_EARLY_PREFIX");
    h->early_prefix = env ? atoi(env) : 0;
    h->drop_stage = -1;
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    int major = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, h->device);
    if (e == cudaSuccess && major != 10) { delete h; return AGX_E_UNSUPPORTED; }
    constexpr size_t kStateBytes = 256 + 65536 * 8;   // status word and accept ticket | one key per logits row (at most 65535)
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_status, kStateBytes);
    if (e != cudaSuccess) { delete h; return e == cudaErrorMemoryAllocation ? AGX_E_NOMEM : AGX_E_CUDA; }
    e = cudaMemset(h->d_status, 0, kStateBytes);
    if (e != cudaSuccess) { cudaFree(h->d_status); delete h; return AGX_E_CUDA; }
    h->d_ticket = (unsigned int*)(h->d_status + 16);
    h->d_row_keys = (unsigned long long*)(h->d_status + 64);
    *out = h;
    return AGX_OK;
}

agx_status agx_destroy(agx_handle* h) {
    if (!h) return AGX_E_INVAL;
    cudaFree(h->d_status);
    if (h->pipe_in) cudaStreamDestroy(h->pipe_in);
    if (h->pipe_out) cudaStreamDestroy(h->pipe_out);
    for (cudaEvent_t ev : h->pipe_events) cudaEventDestroy(ev);
    delete h->plan_cache;
    delete h;
    return AGX_OK;
}

agx_status agx_kv_append(agx_handle* h, void* k_pool, void* v_pool, int64_t num_pages, const void* k_new,
                         const void* v_new, const int32_t* page_table, int32_t pt_stride, const int32_t* prefix_len,
                         const int32_t* cu_q, int32_t B, int32_t total_q, void* stream) {
    CallRange range_("agx_kv_append");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (B < 0 || total_q < 0) return fail(h, AGX_E_INVAL, "negative B or total_q");
    if (B == 0 || total_q == 0) return AGX_OK;
    if (!k_pool || !v_pool || !k_new || !v_new || !page_table || !prefix_len || !cu_q)
        return fail(h, AGX_E_INVAL, "null pointer");
    if (!aligned(k_pool, 16) || !aligned(v_pool, 16) || !aligned(k_new, 16) || !aligned(v_new, 16))
        return fail(h, AGX_E_INVAL, "K/V buffers must be 16-byte aligned");
    if (num_pages < 1 || pt_stride < 1) return fail(h, AGX_E_INVAL, "num_pages and page_table_stride must be >= 1");
    cudaError_t e = launch_kv_append(h->cfg.dtype, k_pool, v_pool, num_pages, k_new, v_new, page_table, pt_stride,
                                     prefix_len, cu_q, B, total_q, h->cfg.num_kv_heads, h->cfg.head_dim, h->d_status,
                                     (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "kv_append launch");
    h->last_launches = 1;
    return AGX_OK;
}

int64_t agx_attn_workspace_bytes(agx_handle* h, int32_t B, const int32_t* P, const int32_t* Q) {
    if (!h) return AGX_E_INVAL;
    if (B < 0) return fail(h, AGX_E_INVAL, "negative B");
    if (B == 0) return 0;
    if (!P || !Q) return fail(h, AGX_E_INVAL, "null pointer");
    const Plan* plan_ptr = nullptr;
    agx_status st = make_plan(h, B, P, Q, -1, plan_ptr);
    if (st != AGX_OK) return st;
    const Plan& plan = *plan_ptr;
    if (plan.part_entries == 0) return 0;
    return (int64_t)(part_ml_bytes(plan.part_entries) + (size_t)plan.part_entries * h->cfg.head_dim * sizeof(float));
}

// Attention, optionally preceded by the append of the block's own K/V rows (k_new != NULL).  Launches whose
// sequences all fit one row chunk write those rows in the attention kernel's prologue (each CTA the rows of its own
// KV split and head); the others (blocks of more than 256 rows, fp32 handles) get a separate append launch in front.
static agx_status attn_impl(agx_handle* h, const void* q_block, const void* k_new, const void* v_new, const void* k_pool,
                            const void* v_pool, int64_t num_pages, const int32_t* page_table, int32_t pt_stride,
                            const int32_t* P, const int32_t* Q, int32_t B, void* out, float* lse, void* workspace,
                            size_t workspace_bytes, void* stream_v) {
    CallRange range_("agx_attn_prefixed");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (B < 0) return fail(h, AGX_E_INVAL, "negative B");
    if (B == 0) return AGX_OK;
    if (!q_block || !k_pool || !v_pool || !page_table || !P || !Q || !out) return fail(h, AGX_E_INVAL, "null pointer");
    if (k_new && (!v_new || !aligned(k_new, 16) || !aligned(v_new, 16)))
        return fail(h, AGX_E_INVAL, "k_new/v_new must both be given and 16-byte aligned");
    if (!aligned(q_block, 16) || !aligned(out, 16) || !aligned(k_pool, 256) || !aligned(v_pool, 256))
        return fail(h, AGX_E_INVAL, "q_block/out must be 16-byte and pools 256-byte aligned");
    if (num_pages < 1 || pt_stride < 1) return fail(h, AGX_E_INVAL, "num_pages and page_table_stride must be >= 1");
    const Plan* plan_ptr = nullptr;
    agx_status st = make_plan(h, B, P, Q, pt_stride, plan_ptr);
    if (st != AGX_OK) return st;
    const Plan& plan = *plan_ptr;
    const size_t need = plan.part_entries == 0 ? 0
        : part_ml_bytes(plan.part_entries) + (size_t)plan.part_entries * h->cfg.head_dim * sizeof(float);
    if (need > 0) {
        if (!workspace || !aligned(workspace, 256)) return fail(h, AGX_E_INVAL, "workspace missing or not 256-byte aligned");
        if (workspace_bytes < need) return fail(h, AGX_E_INVAL, "workspace too small: %zu < %zu", workspace_bytes, need);
    }
    cudaStream_t stream = (cudaStream_t)stream_v;
    AttnParams p;
    memset(&p, 0, sizeof p);
    p.q = q_block; p.k_pool = k_pool; p.v_pool = v_pool; p.page_table = page_table;
    p.out = out; p.lse = lse;
    p.part_ml = (float2*)workspace;
    p.part_o = need ? (float*)((char*)workspace + part_ml_bytes(plan.part_entries)) : nullptr;
    p.status = h->d_status;
    p.num_pages = num_pages;
    p.pt_stride = pt_stride;
    p.hq = h->cfg.num_q_heads; p.hkv = h->cfg.num_kv_heads; p.head_dim = h->cfg.head_dim;
    p.scale_log2 = h->scale * 1.4426950408889634f;
    p.row_div_magic = (0x100000000ull + (unsigned)(p.hq / p.hkv) - 1) / (unsigned)(p.hq / p.hkv);
    p.wait_limit_cycles = h->wait_limit_cycles;
    p.early_prefix = h->early_prefix;
    p.drop_stage = h->drop_stage;
    const CUtensorMap *map_k = nullptr, *map_v = nullptr;
    if (h->cfg.dtype == AGX_BF16 && h->cfg.head_dim == 128) {
        if ((long long)num_pages * p.hkv * kPage > 0x7FFFFFFFll) return fail(h, AGX_E_RANGE, "pool too large for one tensor map");
        map_k = pool_map(h, k_pool, num_pages, p.hkv);
        map_v = pool_map(h, v_pool, num_pages, p.hkv);
        if (!map_k || !map_v) return fail(h, AGX_E_CUDA, "cuTensorMapEncodeTiled failed");
    }
    for (const Launch& ln : plan.launches) {
        p.num_seqs = (int)ln.seqs.size();
        p.num_items = ln.num_items;
        bool split = false;
        bool one_chunk = true;
        for (int i = 0; i < p.num_seqs; ++i) {
            p.seq[i] = ln.seqs[i];
            split |= ln.seqs[i].nsplit > 1 && !ln.cluster;
            one_chunk &= ln.seqs[i].row_chunks == 1;
        }
        cudaError_t e;
        p.cluster_size = ln.cluster;
        p.part_half = ln.kind == KIND_TILE || ln.lean_merge;
        p.k_new = p.v_new = nullptr;
        if (k_new) {
            p.k_new = k_new; p.v_new = v_new;
            if (ln.kind == KIND_SIMT || !one_chunk) {
                e = launch_kv_append_plan(p, h->cfg.dtype, ln.total_rows, stream);
                if (e != cudaSuccess) return cuda_fail(h, e, "append launch");
                h->last_launches++;
                p.k_new = p.v_new = nullptr;
            }
        }
        switch (ln.kind) {
            case KIND_SMALL1: e = launch_attn_small_bf16(p, 1, ln.kw, *map_k, *map_v, stream); break;
            case KIND_SMALL2: e = launch_attn_small_bf16(p, 2, ln.kw, *map_k, *map_v, stream); break;
            case KIND_SMALL4: e = launch_attn_small_bf16(p, 4, 4, *map_k, *map_v, stream); break;
            case KIND_SIMT: e = launch_attn_simt(p, h->cfg.dtype, stream); break;
            case KIND_TILE: e = launch_attn_tile_bf16(p, false, *map_k, *map_v, stream); break;
            case KIND_STREAM: e = launch_attn_tile_bf16(p, true, *map_k, *map_v, stream); break;
            default: return fail(h, AGX_E_UNSUPPORTED, "unknown kernel kind");
        }
        if (e != cudaSuccess) return cuda_fail(h, e, "attention launch");
        h->last_launches++;
        if (split) {
            e = launch_attn_combine(p, h->cfg.dtype, ln.total_rows, stream);
            if (e != cudaSuccess) return cuda_fail(h, e, "combine launch");
            h->last_launches++;
        }
    }
    return AGX_OK;
}

agx_status agx_attn_prefixed(agx_handle* h, const void* q_block, const void* k_pool, const void* v_pool,
                             int64_t num_pages, const int32_t* page_table, int32_t pt_stride, const int32_t* P,
                             const int32_t* Q, int32_t B, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, void* stream) {
    return attn_impl(h, q_block, nullptr, nullptr, k_pool, v_pool, num_pages, page_table, pt_stride, P, Q, B, out, lse,
                     workspace, workspace_bytes, stream);
}

agx_status agx_attn_prefixed_append(agx_handle* h, const void* q_block, const void* k_new, const void* v_new, void* k_pool,
                                    void* v_pool, int64_t num_pages, const int32_t* page_table, int32_t pt_stride,
                                    const int32_t* P, const int32_t* Q, int32_t B, void* out, float* lse,
                                    void* workspace, size_t workspace_bytes, void* stream) {
    if (h && B > 0 && (!k_new || !v_new)) return fail(h, AGX_E_INVAL, "null pointer");
    return attn_impl(h, q_block, k_new, v_new, k_pool, v_pool, num_pages, page_table, pt_stride, P, Q, B, out, lse,
                     workspace, workspace_bytes, stream);
}

static int accept_chunks(const agx_handle* h, int total_q, int vocab, int dtype) {
    const int vec = 16 / elem_size(dtype);
    const int target = 8 * h->sm_count;   // enough CTAs that every thread needs a single trip of two 16-byte loads
    int want = std::max(1, (target + total_q - 1) / total_q);
    const int max_chunks = std::max(1, (vocab + 256 * vec * 2 - 1) / (256 * vec * 2));  // >= 2 vectors per thread
    want = std::min(want, max_chunks);
    int chunk_elems = (vocab + want - 1) / want;
    chunk_elems = (chunk_elems + vec - 1) / vec * vec;
    return (vocab + chunk_elems - 1) / chunk_elems;
}

int64_t agx_accept_workspace_bytes(agx_handle* h, int32_t total_q, int32_t vocab) {
    if (!h) return AGX_E_INVAL;
    if (total_q < 0 || vocab < 1) return fail(h, AGX_E_RANGE, "total_q < 0 or vocab < 1");
    // the rows' winners when they do not fit the kernel's shared memory (more than 2048 rows); the rows' keys live in the handle
    return (int64_t)total_q * 4 + 256;
}

agx_status agx_accept_greedy(agx_handle* h, const void* logits, int32_t logits_dtype, int64_t row_stride,
                             int32_t vocab, const int32_t* drafts, const int32_t* cu_q, int32_t B, int32_t total_q,
                             int32_t* accept_len, int32_t* next_token, int32_t* argmax, int32_t* seq_lens,
                             void* workspace, size_t workspace_bytes, void* stream) {
    CallRange range_("agx_accept_greedy");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (B < 0 || total_q < 0) return fail(h, AGX_E_INVAL, "negative B or total_q");
    if (B == 0) return AGX_OK;
    if (total_q < B) return fail(h, AGX_E_INVAL, "total_q < B (every sequence has at least one row)");
    if (logits_dtype != AGX_BF16 && logits_dtype != AGX_F32) return fail(h, AGX_E_UNSUPPORTED, "logits dtype");
    if (vocab < 1 || row_stride < vocab) return fail(h, AGX_E_RANGE, "vocab < 1 or row_stride < vocab");
    if (total_q > 65535) return fail(h, AGX_E_RANGE, "more than 65535 logits rows in one call");
    if (!logits || !cu_q || !accept_len || !next_token || (!drafts && total_q > B)) return fail(h, AGX_E_INVAL, "null pointer");
    if (!aligned(logits, elem_size(logits_dtype))) return fail(h, AGX_E_INVAL, "logits misaligned");
    const int64_t need = agx_accept_workspace_bytes(h, total_q, vocab);
    if (!workspace || !aligned(workspace, 8) || (int64_t)workspace_bytes < need)
        return fail(h, AGX_E_INVAL, "accept workspace missing, misaligned or too small (%lld needed)", (long long)need);
    const int chunks = accept_chunks(h, total_q, vocab, logits_dtype);
    cudaError_t e = launch_accept(logits, logits_dtype, row_stride, vocab, drafts, cu_q, B, total_q, accept_len,
                                  next_token, argmax, seq_lens, h->d_row_keys, (int*)workspace, chunks, h->d_ticket,
                                  (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "accept launch");
    h->last_launches = 1;
    return AGX_OK;
}

agx_status agx_get_status(agx_handle* h, void* stream, int32_t* device_status) {
    if (!h || !device_status) return AGX_E_INVAL;
    int v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, h->d_status, sizeof v, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "status read");
    *device_status = v;
    if (v != 0) {
        e = cudaMemsetAsync(h->d_status, 0, sizeof(int), (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(h, e, "status clear");
        return fail(h, AGX_E_DEVICE, "device status 0x%x", v);
    }
    return AGX_OK;
}

int32_t agx_last_launch_count(const agx_handle* h) { return h ? h->last_launches : 0; }

agx_status agx_set_option(agx_handle* h, int32_t option, int64_t value) {
    if (!h) return AGX_E_INVAL;
    switch (option) {
        case AGX_OPT_EARLY_PREFIX_LOADS:
            h->early_prefix = value != 0;
            return AGX_OK;
        case AGX_OPT_WAIT_LIMIT_CYCLES:
            if (value < 1000) return fail(h, AGX_E_RANGE, "wait limit below 1000 cycles");
            h->wait_limit_cycles = value;
            return AGX_OK;
        case AGX_OPT_ZERO_COPY:
            if (value < 0 || value > 3) return fail(h, AGX_E_RANGE, "zero-copy bits");
            h->zero_copy = (int)value;
            return AGX_OK;
        case AGX_OPT_TEST_DROP_STAGE:
            if (value < -1 || value > 0x7FFFFFFF) return fail(h, AGX_E_RANGE, "stage index");
            h->drop_stage = (int)value;
            return AGX_OK;
        default:
            return fail(h, AGX_E_INVAL, "unknown option %d", option);
    }
}

}  // extern "C"

namespace {
constexpr size_t kZeroCopyMaxBytes = 1u << 20;

// Device-side address of a 16-byte-aligned host buffer that is pinned and mapped (cudaHostAlloc / cudaHostRegister
// under unified addressing), else NULL.
void* mapped_alias(const void* host) {
    if (!host || ((uintptr_t)host & 15)) return nullptr;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// Attention-only host steps that move a few megabytes or more are cut into row chunks whose transfers overlap the
// attention calls of the other chunks (chunked prefill: rows [r0, r1) of a block are a block of their own behind a prefix
// longer by r0, since the chunks before them have appended their K/V by then).
bool host_step_pipelined(const agx_handle* h, int B, const int32_t* Q, int vocab) {
    if (vocab > 0 || h->pipe_rows <= 0) return false;
    long long tq = 0;
    for (int s = 0; s < B; ++s) tq += Q[s];
    const long long in_bytes = tq * (h->cfg.num_q_heads + 2 * h->cfg.num_kv_heads) * h->cfg.head_dim * elem_size(h->cfg.dtype);
    return in_bytes >= (4ll << 20) && tq > h->pipe_rows;
}

// The attention calls of a pipelined host step: runs of whole blocks that together have about a thousand rows, and
// blocks longer than that in row chunks of pipe_rows rows.
struct HostChunk {
    int s0, nseq;      // sequences [s0, s0 + nseq)
    int r0, rows;      // nseq == 1: rows [r0, r0 + rows) of the block; otherwise r0 = 0 and rows = all rows of the run
    size_t row_begin;  // first row of the chunk in the step's row order
};
void host_step_chunks(const agx_handle* h, int B, const int32_t* Q, std::vector<HostChunk>& out) {
    // Runs of whole blocks of about a thousand rows (measured on the ragged prefill blocks of c4, runs of 384 / 512 / 768 / 1024 rows:
    // 1.94 / 1.97 / 1.81 / 1.77 ms per step).  When that gives fewer than three calls there is nothing to overlap: blocks on their
    // own are then cut into row chunks (the 512-row block of c3 as one call 1.68 ms per 8 layers, as 384 + 128 rows 1.54 ms; with
    // many runs the cut only adds calls: c4 1.93 ms).
    const int run_rows = std::max(1024, 2 * h->pipe_rows);
    std::vector<HostChunk> runs;
    size_t row = 0;
    int s = 0;
    while (s < B) {
        HostChunk c = {s, 0, 0, 0, row};
        while (s < B && c.nseq < kMaxSeqs && (c.nseq == 0 || c.rows + Q[s] <= run_rows)) {
            c.rows += Q[s]; row += Q[s]; ++c.nseq; ++s;
        }
        runs.push_back(c);
    }
    out.clear();
    for (const HostChunk& c : runs) {
        if (runs.size() < 3 && c.nseq == 1 && c.rows > h->pipe_rows) {
            for (int r0 = 0; r0 < c.rows; r0 += h->pipe_rows)
                out.push_back({c.s0, 1, r0, std::min(h->pipe_rows, c.rows - r0), c.row_begin + (size_t)r0});
        } else {
            out.push_back(c);
        }
    }
}

struct HostStepLayout {
    size_t q, k, v, out, logits, drafts, prefix, cu, acc, next, seqlen, attn_ws, accept_ws, total;
    size_t q_bytes, kv_bytes, logits_bytes, attn_ws_bytes, accept_ws_bytes;
    int total_q;
};
agx_status host_step_layout(agx_handle* h, int B, const int32_t* P, const int32_t* Q, int logits_dtype,
                            int64_t row_stride, int vocab, HostStepLayout& L) {
    if (B < 1 || !P || !Q) return fail(h, AGX_E_INVAL, "B < 1 or null lengths");
    const bool with_accept = vocab > 0;  // vocab == 0: attention only
    if (with_accept) {
        if (logits_dtype != AGX_BF16 && logits_dtype != AGX_F32) return fail(h, AGX_E_UNSUPPORTED, "logits dtype");
        if (row_stride < vocab) return fail(h, AGX_E_RANGE, "row_stride < vocab");
    } else if (vocab < 0) {
        return fail(h, AGX_E_RANGE, "vocab < 0");
    }
    long long tq = 0;
    for (int s = 0; s < B; ++s) {
        if (Q[s] < 1) return fail(h, AGX_E_INVAL, "q_len[%d] = %d < 1", s, Q[s]);
        tq += Q[s];
    }
    if (tq > 65535) return fail(h, AGX_E_RANGE, "more than 65535 rows in one host step");
    int64_t aws = 0;
    if (host_step_pipelined(h, B, Q, vocab)) {
        // one attention call per chunk, one after the other on the caller's stream: the largest workspace of them
        std::vector<HostChunk> chunks;
        host_step_chunks(h, B, Q, chunks);
        for (const HostChunk& c : chunks) {
            const int32_t pc = P[c.s0] + c.r0, qc = c.rows;
            const int64_t w = c.nseq == 1 ? agx_attn_workspace_bytes(h, 1, &pc, &qc) : agx_attn_workspace_bytes(h, c.nseq, P + c.s0, Q + c.s0);
            if (w < 0) return (agx_status)w;
            aws = std::max(aws, w);
        }
    } else {
        aws = agx_attn_workspace_bytes(h, B, P, Q);
        if (aws < 0) return (agx_status)aws;
    }
    const int64_t cws = with_accept ? agx_accept_workspace_bytes(h, (int)tq, vocab) : 0;
    if (cws < 0) return (agx_status)cws;
    const size_t es = elem_size(h->cfg.dtype);
    L.total_q = (int)tq;
    L.q_bytes = (size_t)tq * h->cfg.num_q_heads * h->cfg.head_dim * es;
    L.kv_bytes = (size_t)tq * h->cfg.num_kv_heads * h->cfg.head_dim * es;
    L.logits_bytes = with_accept ? (size_t)tq * row_stride * elem_size(logits_dtype) : 0;
    L.attn_ws_bytes = (size_t)aws;
    L.accept_ws_bytes = (size_t)cws;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
    L.q = take(L.q_bytes); L.k = take(L.kv_bytes); L.v = take(L.kv_bytes); L.out = take(L.q_bytes);
    L.logits = take(L.logits_bytes); L.drafts = take((size_t)(tq - B) * 4 + 4);
    L.prefix = take((size_t)B * 4); L.cu = take((size_t)(B + 1) * 4);
    L.acc = take((size_t)B * 4); L.next = take((size_t)B * 4); L.seqlen = take((size_t)B * 4);
    L.attn_ws = take(L.attn_ws_bytes); L.accept_ws = take(L.accept_ws_bytes);
    L.total = off;
    return AGX_OK;
}
}  // namespace

extern "C" {

int64_t agx_verify_step_host_workspace_bytes(agx_handle* h, int32_t B, const int32_t* P, const int32_t* Q,
                                             int32_t logits_dtype, int64_t row_stride, int32_t vocab) {
    if (!h) return AGX_E_INVAL;
    HostStepLayout L;
    agx_status st = host_step_layout(h, B, P, Q, logits_dtype, row_stride, vocab, L);
    return st != AGX_OK ? (int64_t)st : (int64_t)L.total;
}

static agx_status verify_step_host_impl(agx_handle* h, void* k_pool, void* v_pool, int64_t num_pages,
                                const int32_t* page_table, int32_t pt_stride, const int32_t* P, const int32_t* Q,
                                int32_t B, const void* h_q, const void* h_k, const void* h_v, const void* h_logits,
                                int32_t logits_dtype, int64_t row_stride, int32_t vocab, const int32_t* h_drafts,
                                void* h_out, int32_t* h_accept, int32_t* h_next, int32_t* h_seq_lens, void* workspace,
                                size_t workspace_bytes, void* stream_v, bool sync) {
    CallRange range_("agx_verify_step_host");
    if (!h) return AGX_E_INVAL;
    HostStepLayout L;
    agx_status st = host_step_layout(h, B, P, Q, logits_dtype, row_stride, vocab, L);
    if (st != AGX_OK) return st;
    const bool with_accept = vocab > 0;
    if (!k_pool || !v_pool || !page_table || !h_q || !h_k || !h_v || !h_out) return fail(h, AGX_E_INVAL, "null pointer");
    if (with_accept && (!h_logits || !h_accept || !h_next || !h_seq_lens || (!h_drafts && L.total_q > B)))
        return fail(h, AGX_E_INVAL, "null pointer (accept arguments)");
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < L.total)
        return fail(h, AGX_E_INVAL, "host-step workspace missing, misaligned or too small (%zu needed)", L.total);
    cudaStream_t stream = (cudaStream_t)stream_v;
    char* ws = (char*)workspace;
    if (host_step_pipelined(h, B, Q, vocab)) {
        cudaError_t pe = cudaSuccess;
        if (!h->pipe_in) pe = cudaStreamCreateWithFlags(&h->pipe_in, cudaStreamNonBlocking);
        if (pe == cudaSuccess && !h->pipe_out) pe = cudaStreamCreateWithFlags(&h->pipe_out, cudaStreamNonBlocking);
        std::vector<HostChunk> list;
        host_step_chunks(h, B, Q, list);
        const size_t chunks = list.size();
        while (pe == cudaSuccess && h->pipe_events.size() < 2 * chunks + 2) {
            cudaEvent_t ev;
            pe = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            if (pe == cudaSuccess) h->pipe_events.push_back(ev);
        }
        if (pe != cudaSuccess) return cuda_fail(h, pe, "host step: pipeline set-up");
        const size_t es = elem_size(h->cfg.dtype);
        const size_t q_row = (size_t)h->cfg.num_q_heads * h->cfg.head_dim * es, kv_row = (size_t)h->cfg.num_kv_heads * h->cfg.head_dim * es;
        cudaEvent_t fork = h->pipe_events[2 * chunks], join = h->pipe_events[2 * chunks + 1];
        // the side streams start behind whatever the caller has already put on its stream ...
        pe = cudaEventRecord(fork, stream);
        if (pe == cudaSuccess) pe = cudaStreamWaitEvent(h->pipe_in, fork, 0);
        if (pe == cudaSuccess) pe = cudaStreamWaitEvent(h->pipe_out, fork, 0);
        int launches = 0;
        for (size_t i = 0; i < chunks && pe == cudaSuccess; ++i) {
            const HostChunk& c = list[i];
            const int32_t pc = P[c.s0] + c.r0, qc = c.rows;
            const size_t r = c.row_begin, n = (size_t)c.rows;
            cudaEvent_t in_done = h->pipe_events[2 * i], out_ready = h->pipe_events[2 * i + 1];
            pe = cudaMemcpyAsync(ws + L.q + r * q_row, (const char*)h_q + r * q_row, n * q_row, cudaMemcpyHostToDevice, h->pipe_in);
            if (pe == cudaSuccess) pe = cudaMemcpyAsync(ws + L.k + r * kv_row, (const char*)h_k + r * kv_row, n * kv_row, cudaMemcpyHostToDevice, h->pipe_in);
            if (pe == cudaSuccess) pe = cudaMemcpyAsync(ws + L.v + r * kv_row, (const char*)h_v + r * kv_row, n * kv_row, cudaMemcpyHostToDevice, h->pipe_in);
            if (pe == cudaSuccess) pe = cudaEventRecord(in_done, h->pipe_in);
            if (pe == cudaSuccess) pe = cudaStreamWaitEvent(stream, in_done, 0);
            if (pe != cudaSuccess) break;
            st = agx_attn_prefixed_append(h, ws + L.q + r * q_row, ws + L.k + r * kv_row, ws + L.v + r * kv_row, k_pool, v_pool, num_pages,
                                          page_table + (size_t)c.s0 * pt_stride, pt_stride, c.nseq == 1 ? &pc : P + c.s0,
                                          c.nseq == 1 ? &qc : Q + c.s0, c.nseq, ws + L.out + r * q_row, nullptr,
                                          L.attn_ws_bytes ? ws + L.attn_ws : nullptr, L.attn_ws_bytes, stream);
            if (st != AGX_OK) break;
            launches += h->last_launches;
            pe = cudaEventRecord(out_ready, stream);
            if (pe == cudaSuccess) pe = cudaStreamWaitEvent(h->pipe_out, out_ready, 0);
            if (pe == cudaSuccess) pe = cudaMemcpyAsync((char*)h_out + r * q_row, ws + L.out + r * q_row, n * q_row, cudaMemcpyDeviceToHost, h->pipe_out);
        }
        // ... and the caller's stream ends behind the last download (also when a call in the middle failed: the join still
        // has to bring the side streams back, or a stream capture of the caller's would be left forked)
        cudaError_t je = cudaEventRecord(join, h->pipe_out);
        if (je == cudaSuccess) je = cudaStreamWaitEvent(stream, join, 0);
        if (st != AGX_OK) return st;
        if (pe == cudaSuccess) pe = je;
        if (pe == cudaSuccess && sync) pe = cudaStreamSynchronize(stream);
        if (pe != cudaSuccess) return cuda_fail(h, pe, "host step: pipelined transfers");
        h->last_launches = launches;
        return AGX_OK;
    }
    std::vector<int32_t>& cu = h->cu_host;  // outlives the asynchronous copy (the call ends with a sync)
    cu.assign(B + 1, 0);
    for (int s = 0; s < B; ++s) cu[s + 1] = cu[s] + Q[s];
    cudaError_t e = cudaSuccess;
    int launches = 0;
    auto h2d = [&](size_t off, const void* src, size_t bytes) {
        if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(ws + off, src, bytes, cudaMemcpyHostToDevice, stream);
    };
    // Small blocks in pinned, device-mapped host memory cross by one kernel that reads the host buffers and, on the
    // way back, by the attention kernels writing `out` straight into the host buffer: each copy-engine transfer on
    // the stream costs several microseconds whatever its size.  Anything else goes through cudaMemcpyAsync.
    const size_t in_bytes = L.q_bytes + 2 * L.kv_bytes;
    const void* mq = (h->zero_copy & 1) && in_bytes <= kZeroCopyMaxBytes ? mapped_alias(h_q) : nullptr;
    const void* mk = mq ? mapped_alias(h_k) : nullptr;
    const void* mv = mk ? mapped_alias(h_v) : nullptr;
    void* out_dev = ws + L.out;
    if ((h->zero_copy & 2) && L.q_bytes <= kZeroCopyMaxBytes)
        if (void* mo = mapped_alias(h_out)) out_dev = mo;
    if (mv) {
        StageCopies sc;
        sc.src[0] = (const uint4*)mq; sc.src[1] = (const uint4*)mk; sc.src[2] = (const uint4*)mv;
        sc.dst[0] = (uint4*)(ws + L.q); sc.dst[1] = (uint4*)(ws + L.k); sc.dst[2] = (uint4*)(ws + L.v);
        sc.units[0] = (unsigned)(L.q_bytes / 16); sc.units[1] = sc.units[2] = (unsigned)(L.kv_bytes / 16);
        e = launch_stage_in(sc, stream);
        if (e == cudaSuccess) ++launches;
    } else {
        h2d(L.q, h_q, L.q_bytes); h2d(L.k, h_k, L.kv_bytes); h2d(L.v, h_v, L.kv_bytes);
    }
    // The logits are needed by the accept step only: a megabyte or more of them crosses on a stream of the handle's own,
    // beside the attention kernels, and the caller's stream waits for that copy just before the accept launch.
    cudaEvent_t logits_done = nullptr;
    if (with_accept && L.logits_bytes >= (1u << 20) && h->pipe_rows > 0 && e == cudaSuccess) {
        if (!h->pipe_in) e = cudaStreamCreateWithFlags(&h->pipe_in, cudaStreamNonBlocking);
        while (e == cudaSuccess && h->pipe_events.size() < 2) {
            cudaEvent_t ev;
            e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            if (e == cudaSuccess) h->pipe_events.push_back(ev);
        }
        if (e == cudaSuccess) e = cudaEventRecord(h->pipe_events[0], stream);   // behind whatever last used the workspace
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->pipe_in, h->pipe_events[0], 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ws + L.logits, h_logits, L.logits_bytes, cudaMemcpyHostToDevice, h->pipe_in);
        if (e == cudaSuccess && L.total_q > B)
            e = cudaMemcpyAsync(ws + L.drafts, h_drafts, (size_t)(L.total_q - B) * 4, cudaMemcpyHostToDevice, h->pipe_in);
        if (e == cudaSuccess) e = cudaEventRecord(h->pipe_events[1], h->pipe_in);
        if (e == cudaSuccess) logits_done = h->pipe_events[1];
    } else if (with_accept) {
        h2d(L.logits, h_logits, L.logits_bytes);
        h2d(L.drafts, h_drafts, (size_t)(L.total_q - B) * 4);
    }
    if (!with_accept) {
        // lengths are needed on the device by the accept step only
    } else if (B <= kMaxSeqs) {   // as kernel arguments: no pageable copies, which would each synchronise the stream first
        StepMeta meta;
        meta.B = B;
        for (int s = 0; s < B; ++s) { meta.prefix[s] = P[s]; meta.cu[s] = cu[s]; }
        meta.cu[B] = cu[B];
        if (e == cudaSuccess)
            e = launch_write_meta(meta, (int*)(ws + L.prefix), (int*)(ws + L.seqlen), (int*)(ws + L.cu), stream);
        if (e == cudaSuccess) ++launches;
    } else {
        h2d(L.prefix, P, (size_t)B * 4);
        h2d(L.seqlen, P, (size_t)B * 4);
        h2d(L.cu, cu.data(), (size_t)(B + 1) * 4);
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "host step: upload");
    st = agx_attn_prefixed_append(h, ws + L.q, ws + L.k, ws + L.v, k_pool, v_pool, num_pages, page_table, pt_stride, P, Q,
                                  B, out_dev, nullptr, L.attn_ws_bytes ? ws + L.attn_ws : nullptr, L.attn_ws_bytes,
                                  stream);
    if (st == AGX_OK) launches += h->last_launches;
    if (logits_done) {   // (also when the attention call failed: the side stream is brought back before the call returns)
        e = cudaStreamWaitEvent(stream, logits_done, 0);
        if (e != cudaSuccess) return cuda_fail(h, e, "host step: logits upload");
    }
    if (st != AGX_OK) return st;
    if (with_accept) {
        st = agx_accept_greedy(h, ws + L.logits, logits_dtype, row_stride, vocab, (const int32_t*)(ws + L.drafts),
                               (const int32_t*)(ws + L.cu), B, L.total_q, (int32_t*)(ws + L.acc),
                               (int32_t*)(ws + L.next), nullptr, (int32_t*)(ws + L.seqlen), ws + L.accept_ws,
                               L.accept_ws_bytes, stream);
        if (st != AGX_OK) return st;
        launches += h->last_launches;
    }
    auto d2h = [&](void* dst, size_t off, size_t bytes) {
        if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, ws + off, bytes, cudaMemcpyDeviceToHost, stream);
    };
    if (out_dev == ws + L.out) d2h(h_out, L.out, L.q_bytes);
    if (with_accept) {
        d2h(h_accept, L.acc, (size_t)B * 4); d2h(h_next, L.next, (size_t)B * 4); d2h(h_seq_lens, L.seqlen, (size_t)B * 4);
    }
    if (e == cudaSuccess && sync) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "host step: download");
    h->last_launches = launches;
    return AGX_OK;
}

agx_status agx_verify_step_host(agx_handle* h, void* k_pool, void* v_pool, int64_t num_pages,
                                const int32_t* page_table, int32_t pt_stride, const int32_t* P, const int32_t* Q,
                                int32_t B, const void* h_q, const void* h_k, const void* h_v, const void* h_logits,
                                int32_t logits_dtype, int64_t row_stride, int32_t vocab, const int32_t* h_drafts,
                                void* h_out, int32_t* h_accept, int32_t* h_next, int32_t* h_seq_lens, void* workspace,
                                size_t workspace_bytes, void* stream) {
    return verify_step_host_impl(h, k_pool, v_pool, num_pages, page_table, pt_stride, P, Q, B, h_q, h_k, h_v, h_logits,
                                 logits_dtype, row_stride, vocab, h_drafts, h_out, h_accept, h_next, h_seq_lens, workspace,
                                 workspace_bytes, stream, true);
}

agx_status agx_verify_step_host_enqueue(agx_handle* h, void* k_pool, void* v_pool, int64_t num_pages,
                                        const int32_t* page_table, int32_t pt_stride, const int32_t* P, const int32_t* Q,
                                        int32_t B, const void* h_q, const void* h_k, const void* h_v,
                                        const void* h_logits, int32_t logits_dtype, int64_t row_stride, int32_t vocab,
                                        const int32_t* h_drafts, void* h_out, int32_t* h_accept, int32_t* h_next,
                                        int32_t* h_seq_lens, void* workspace, size_t workspace_bytes, void* stream) {
    return verify_step_host_impl(h, k_pool, v_pool, num_pages, page_table, pt_stride, P, Q, B, h_q, h_k, h_v, h_logits,
                                 logits_dtype, row_stride, vocab, h_drafts, h_out, h_accept, h_next, h_seq_lens, workspace,
                                 workspace_bytes, stream, false);
}

int64_t agx_ngram_lut_bytes(int32_t max_stream_tokens) {
    if (max_stream_tokens < 0 || max_stream_tokens > (1 << 24)) return AGX_E_RANGE;
    return (int64_t)ngram_lut_bytes(max_stream_tokens);
}

int64_t agx_ngram_workspace_bytes(int32_t stream_tokens) {
    if (stream_tokens < 0 || stream_tokens > (1 << 24)) return AGX_E_RANGE;
    return (int64_t)ngram_workspace_bytes(stream_tokens);
}

agx_status agx_ngram_build(agx_handle* h, const int32_t* stream_tokens, int32_t num_tokens, int32_t n, void* lut,
                           size_t lut_bytes, void* workspace, size_t workspace_bytes, void* stream) {
    CallRange range_("agx_ngram_build");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (n != 2 && n != 3) return fail(h, AGX_E_UNSUPPORTED, "n-gram order %d (2 and 3 are built)", n);
    if (num_tokens < 0) return fail(h, AGX_E_INVAL, "negative num_tokens");
    if (num_tokens > (1 << 24)) return fail(h, AGX_E_RANGE, "more than 2^24 stream tokens");
    if (!lut || !workspace || (!stream_tokens && num_tokens > 0)) return fail(h, AGX_E_INVAL, "null pointer");
    if (!aligned(lut, 16) || !aligned(workspace, 16)) return fail(h, AGX_E_INVAL, "lut/workspace must be 16-byte aligned");
    if ((long long)lut_bytes < ngram_lut_bytes(num_tokens) || (long long)workspace_bytes < ngram_workspace_bytes(num_tokens))
        return fail(h, AGX_E_INVAL, "lut (%lld needed) or workspace (%lld needed) too small", ngram_lut_bytes(num_tokens),
                    ngram_workspace_bytes(num_tokens));
    cudaError_t e = launch_ngram_build(stream_tokens, num_tokens, n, lut, workspace, h->d_status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "n-gram build");
    h->last_launches = num_tokens >= n ? 3 : 1;
    return AGX_OK;
}

agx_status agx_ngram_draft(agx_handle* h, const void* lut, const int32_t* context, const int32_t* fill, int32_t B, int32_t k,
                           int32_t* drafts, int32_t* has_draft, void* stream) {
    CallRange range_("agx_ngram_draft");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (B < 0 || k < 0) return fail(h, AGX_E_INVAL, "negative B or k");
    if (B == 0) return AGX_OK;
    if (!lut || !context || !has_draft || (k > 0 && (!fill || !drafts))) return fail(h, AGX_E_INVAL, "null pointer");
    cudaError_t e = launch_ngram_draft(lut, context, fill, B, k, drafts, has_draft, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "n-gram draft");
    h->last_launches = 1;
    return AGX_OK;
}

agx_status agx_kv_copy_pages(agx_handle* h, void* k_pool, void* v_pool, int64_t num_pages, const int32_t* src,
                             const int32_t* dst, int32_t count, void* stream) {
    CallRange range_("agx_kv_copy_pages");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (count < 0) return fail(h, AGX_E_INVAL, "negative count");
    if (count == 0) return AGX_OK;
    if (!k_pool || !v_pool || !src || !dst || num_pages < 1) return fail(h, AGX_E_INVAL, "null pointer or no pages");
    if (!aligned(k_pool, 16) || !aligned(v_pool, 16)) return fail(h, AGX_E_INVAL, "pools must be 16-byte aligned");
    cudaError_t e = launch_copy_pages(h->cfg.dtype, k_pool, v_pool, num_pages, src, dst, count, h->cfg.num_kv_heads,
                                      h->cfg.head_dim, h->d_status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "page copy");
    h->last_launches = 1;
    return AGX_OK;
}

int64_t agx_kv_import_staging_bytes(const agx_handle* h, int32_t count) {
    if (!h || count < 0) return AGX_E_INVAL;
    return 2ll * count * h->cfg.num_kv_heads * kPage * h->cfg.head_dim * elem_size(h->cfg.dtype);
}

agx_status agx_kv_import_pages(agx_handle* h, void* k_pool, void* v_pool, int64_t num_pages, const void* h_k, const void* h_v,
                               const int32_t* dst_pages, int32_t count, void* staging, size_t staging_bytes, void* stream_v) {
    CallRange range_("agx_kv_import_pages");
    if (!h) return AGX_E_INVAL;
    h->last_launches = 0;
    if (count < 0) return fail(h, AGX_E_INVAL, "negative count");
    if (count == 0) return AGX_OK;
    if (!k_pool || !v_pool || !h_k || !h_v || !dst_pages || !staging || num_pages < 1) return fail(h, AGX_E_INVAL, "null pointer or no pages");
    if (!aligned(k_pool, 16) || !aligned(v_pool, 16) || !aligned(staging, 16)) return fail(h, AGX_E_INVAL, "pools and staging must be 16-byte aligned");
    const size_t half = (size_t)agx_kv_import_staging_bytes(h, count) / 2;
    if (staging_bytes < 2 * half) return fail(h, AGX_E_INVAL, "staging too small: %zu < %zu", staging_bytes, 2 * half);
    cudaStream_t stream = (cudaStream_t)stream_v;
    char* st = (char*)staging;
    // Stored pages in pinned, device-mapped host memory are read across the bus by the scatter kernel itself (one pass,
    // no staging); anything else is copied into the staging area first.
    const void* mk = (h->zero_copy & 1) ? mapped_alias(h_k) : nullptr;
    const void* mv = mk ? mapped_alias(h_v) : nullptr;
    cudaError_t e = cudaSuccess;
    if (mv) {
        e = launch_scatter_pages(h->cfg.dtype, k_pool, v_pool, num_pages, mk, mv, dst_pages, count, h->cfg.num_kv_heads,
                                 h->cfg.head_dim, h->d_status, stream);
    } else {
        e = cudaMemcpyAsync(st, h_k, half, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(st + half, h_v, half, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess)
            e = launch_scatter_pages(h->cfg.dtype, k_pool, v_pool, num_pages, st, st + half, dst_pages, count, h->cfg.num_kv_heads,
                                     h->cfg.head_dim, h->d_status, stream);
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "page import");
    h->last_launches = 1;
    return AGX_OK;
}

}  // extern "C"
