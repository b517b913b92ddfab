// Small-q attention over a paged KV cache: the verify block of speculative decoding (q = N + 1
// rows, Sec. 2.3) and plain decode (q = 1, the selective fallback of Sec. 4.3).
//
// The step is HBM-bound: every K and V byte of the sequence is read once and meets only q * G
// query rows (G = Hq / Hkv), i.e. q * G flop per KV byte.  That is above what the fp32 FMA pipes
// sustain at HBM speed once q * G > ~8, so the q * G rows of one KV head are packed into the M
// dimension of warp-level bf16 tensor-core MMAs (m16n8k16, fp32 accumulate): the kernel stays
// bandwidth-bound and verifying 8 tokens costs the same bytes as decoding 1.
//
// Work item = (sequence, KV head, KV split).  A CTA of KW * MT warps (KW = 4 or 8 KV groups): warp (mt, kg)
// owns query rows [16 mt, 16 mt + 16) and, in every stage of KW pages, page kg.  K/V pages stream through a
// 3-stage ring filled by TMA (per page two [16 tokens][64 dims] boxes for K and for V, SWIZZLE_128B so
// ldmatrix is conflict-free; page ids come from the page table, prefetched 32 at a time) and handed over
// with full/empty mbarriers, so no thread spends instructions on addresses.  Per stage the KV groups of an
// m-tile meet twice at a named barrier: once to agree on the rows' running maximum (page maxima through
// shared memory), once to hand round the pages' P (as MMA A fragments, 512 bytes per page).  Each warp
// then accumulates O over all pages of the stage, but only for the 128 / KW output columns it owns, so
// the accumulators never have to be merged: at the end only the row sums are added up.  KW = 8 (16 warps
// for a 32-row verify block, one CTA per SM) halves the number of page steps per warp.  Splits write
// fp32 (m, l, O) partials; a combine kernel merges them in fixed order, so results are bit-reproducible
// run to run.
#include <cuda_fp16.h>
#include <math.h>

#include "agx_internal.cuh"
#include "agx_sm100.cuh"

namespace agx {

namespace {

constexpr int kD = 128;                    // head dim of the bf16 kernels
constexpr int kRowBytes = kD * 2;          // one (token, head) row
// KW = KV groups = pages per pipeline stage (4 or 8): stage = KW * 16 tokens, K + V = KW * 8 KB



__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// byte offset of 16-byte chunk `ch` (0..15) of row `r` in a [rows][256 B] tile, XOR-swizzled
__device__ __forceinline__ uint32_t swz(int r, int ch) { return (uint32_t)(r * kRowBytes + ((ch ^ (r & 7)) << 4)); }

// Loads the compiler keeps where they are written (and that go to L2: the data was just written by other SMs).
__device__ __forceinline__ uint2 ld_volatile_u2(const void* p) {
    uint2 v;
    asm volatile("ld.volatile.global.v2.u32 {%0, %1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float4 ld_volatile_f4(const void* p) {
    float4 v;
    asm volatile("ld.volatile.global.v4.f32 {%0, %1, %2, %3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float2 ld_volatile_f2(const void* p) {
    float2 v;
    asm volatile("ld.volatile.global.v2.f32 {%0, %1}, [%2];\n" : "=f"(v.x), "=f"(v.y) : "l"(p) : "memory");
    return v;
}

// Locate the work item: sequence plan + (kv head, split).
__device__ __forceinline__ int find_seq(const AttnParams& p, int item) {
    int s = 0;
#pragma unroll 1
    for (int i = 1; i < p.num_seqs; ++i)
        if (p.seq[i].item0 <= item) s = i;
    return s;
}

}  // namespace

// MW = m-tiles per warp: with MW = 2 a warp scores its page against both 16-row tiles of a 32-row block and accumulates
// both tiles' output columns, so every K and V fragment is read from shared memory once instead of twice.
template <int MT, int KW, int NS, int MW>
__global__ void __launch_bounds__(32 * (MT / MW) * KW, ((MT / MW) * KW <= 8 && MW == 1) ? 2 : 1)
attn_small_bf16_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ unsigned char smem_raw[];
    constexpr int kKW = KW;
    constexpr int kStageTokens = kKW * kPage;
    constexpr int kStageBytes = 2 * kStageTokens * kRowBytes;
    constexpr int kThreads = 32 * (MT / MW) * KW;
    constexpr int kWarps = (MT / MW) * KW;
    constexpr int kRingBytes = NS * kStageBytes;
    constexpr int kClusterBytes = MT * 16 * (kD * 4 + 8);   // this CTA's (O, m, l) rows, read by the cluster's other CTAs (in the dead ring)
    constexpr int kRegion = kRingBytes > kClusterBytes ? kRingBytes : kClusterBytes;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* ring = smem_raw + (smem_base - smem_u32(smem_raw));   // 1024-aligned: TMA swizzle atoms
    unsigned char* q_smem = ring + kRegion;
    const uint32_t bar_base = smem_base + kRegion + MT * 16 * kRowBytes;  // full[NS], empty[NS]
    volatile int* abort_flag = (volatile int*)(q_smem + MT * 16 * kRowBytes + 2 * NS * 8);
    // exchange area of the KV groups: per-page row maxima, per-group row sums, P fragments of the stage's pages
    float* x_max = (float*)(q_smem + MT * 16 * kRowBytes + 2 * NS * 8 + 16);   // [MT][16][KW]
    float* x_l = x_max + MT * 16 * KW;                                          // [MT][16][KW]
    uint4* x_p = (uint4*)(x_l + MT * 16 * KW);                                  // [MT][KW][32]
    auto full_bar = [&](int i) { return bar_base + 8u * i; };
    auto empty_bar = [&](int i) { return bar_base + 8u * (NS + i); };

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int mt0 = (warp % (MT / MW)) * MW;   // first of this warp's MW m-tiles
    const int kg = warp / (MT / MW);

    const int si = find_seq(p, blockIdx.x);
    const SeqPlan sp = p.seq[si];
    int local = blockIdx.x - sp.item0;  // ((g * row_chunks) + rc) * nsplit + split
    const int split = local % sp.nsplit;
    local /= sp.nsplit;
    const int rc = local % sp.row_chunks;
    const int g = local / sp.row_chunks;
    const int G = p.hq / p.hkv;
    const int P = sp.prefix_len;
    const int q = sp.q_len;
    const int L = P + q;
    const int rows = q * G;          // query rows of this KV head, r = i * G + (h % G)
    const int row0 = rc * 16 * MT;   // first row of this CTA's chunk
    // the chunk's last row sees tokens 0 .. P + i_last
    const int vis_end = P + min(q - 1, (row0 + 16 * MT - 1) / G) + 1;
    const int tok_begin = split * sp.split_tokens;
    const int tok_end = min(vis_end, tok_begin + sp.split_tokens);
    const int n_stages = max(0, (tok_end - tok_begin + kStageTokens - 1) / kStageTokens);

    if (tid == 0) {
        for (int i = 0; i < NS; ++i) { mbar_init(full_bar(i), 1); mbar_init(empty_bar(i), kWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&map_v) : "memory");
    }
    pdl_launch_dependents();
    const int* pt_row = p.page_table + (long long)sp.seq_index * p.pt_stride;
    const int page0 = tok_begin / kPage;
    const int n_pages = (tok_end - tok_begin + kPage - 1) / kPage;
    // A CTA whose KV split holds block rows stores them itself first (fused append) and keeps its copies back until
    // they are in place.  Any other CTA may, with p.early_prefix (the caller vouches that the page table and the pages
    // below the cached-prefix length are not written by a launch still in flight), fetch page ids and K/V stages that
    // lie wholly inside the cached prefix before the dependency wait, i.e. while the launch in front drains.
    const bool own_rows = p.k_new && tok_begin < L && tok_begin + sp.split_tokens > P;
    const bool pre = p.early_prefix && !own_rows;
    if (!(warp == 0 && pre)) pdl_wait();   // from here on global memory written by the launch before this one is read
    // ---- producer state (warp 0; lane 0 issues the TMA copies).  Page ids are fetched 32 at a time,
    //      one group ahead, so the page-table latency never sits in front of a copy.
    int ids_cur = 0, ids_next = 0, group_cur = 0;
    auto fetch_ids = [&](int group) {
        const int pi = group * 32 + lane;
        long long id = 0;
        if (pi < n_pages) {
            id = __ldg(pt_row + page0 + pi);
            if (id < 0 || id >= p.num_pages) { id = 0; atomicOr(p.status, AGX_DEV_BAD_PAGE); }
        }
        return (int)id;
    };
    bool alive = true;
    int last_armed = -1;              // last stage whose copies were armed (lane 0 of warp 0)
    auto produce = [&](int stage) {   // called by all lanes of warp 0
        if (stage >= n_stages || !alive) return;
        const int slot = stage % NS;
        alive = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(slot), ((stage / NS) & 1) ^ 1, abort_flag, p.status, p.wait_limit_cycles));
        if (!alive) return;   // (the same answer in every lane: the lanes stay together for the shuffles and copies below)
        const int pi0 = stage * kKW;
        if ((pi0 >> 5) != group_cur) { ids_cur = ids_next; group_cur = pi0 >> 5; ids_next = fetch_ids(group_cur + 1); }
        const int npg = min(kKW, n_pages - pi0);
        const int my_id = __shfl_sync(0xFFFFFFFFu, ids_cur, (pi0 + lane) & 31);   // lane pg < npg: the id of the stage's page pg
        if (stage == p.drop_stage) return;   // test hook: this stage never arrives, its consumers' waits run out
        if (lane == 0) {
            mbar_arrive_expect_tx(full_bar(slot), npg * 8192u);
            last_armed = stage;
        }
        __syncwarp();   // the barrier is armed before any lane's copies can complete on it
        // lane pg copies page pg: one lane issuing a stage's 32 boxes of 2 KB takes ~60 ns per box, eight lanes ~40 (measured)
        if (lane < npg) {
            const int y = (my_id * p.hkv + g) * kPage;
            const uint32_t dk = smem_base + slot * kStageBytes + lane * 4096, dv = dk + kStageTokens * kRowBytes;
            tma_load_2d(dk, &map_k, 0, y, full_bar(slot));
            tma_load_2d(dk + 2048, &map_k, 64, y, full_bar(slot));
            tma_load_2d(dv, &map_v, 0, y, full_bar(slot));
            tma_load_2d(dv + 2048, &map_v, 64, y, full_bar(slot));
        }
    };
    // A CTA with block rows of its own stores them first (fused append, one row chunk per sequence); its producer warp
    // waits on a named barrier until every thread's rows are in the pages, the other warps only arrive there and go on.
    if (own_rows) {
        append_rows_bf16(p, sp, g, tok_begin, tok_begin + sp.split_tokens, tid, kThreads);
        if (warp != 0) asm volatile("bar.arrive 8, %0;\n" ::"n"(kThreads) : "memory");
    }
    // The producer lane set the barriers up itself, so it needs nothing else from the other warps: it fetches the page
    // ids and issues the first copies at once, while the others bring the Q tile in.
    if (warp == 0) {
        __syncwarp();   // lane 0's barrier initialisation, before the other lanes poll those barriers
        ids_cur = fetch_ids(0);
        ids_next = fetch_ids(1);
        bool waited = !pre;
        if (own_rows) asm volatile("bar.sync 8, %0;\n" ::"n"(kThreads) : "memory");
        const int stable_end = P & ~(kPage - 1);   // tokens below this sit in pages no append of this block touches
#pragma unroll 1
        for (int s = 0; s < NS - 1; ++s) {
            if (!waited && tok_begin + (s + 1) * kStageTokens > stable_end) { pdl_wait(); waited = true; }
            produce(s);
        }
        if (!waited) pdl_wait();
    }
    // ---- Q tile -> shared (rows beyond q*G are zero), by the warps other than the producer's
    //      (a thread's loads are all issued before its first store: one trip to memory, not one per 16-byte unit)
    if (tid >= 32) {
        constexpr int kUnits = MT * 16 * 16, kLoaders = kThreads - 32, kPer = (kUnits + kLoaders - 1) / kLoaders;
        uint4 v[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int c = tid - 32 + j * kLoaders, r = c >> 4, ch = c & 15;
            v[j] = make_uint4(0, 0, 0, 0);
            if (c < kUnits && row0 + r < rows) {
                const int i = (row0 + r) / G, hg = (row0 + r) - i * G;
                const long long off = ((long long)(sp.q_row0 + i) * p.hq + g * G + hg) * kRowBytes + ch * 16;
                v[j] = __ldg((const uint4*)((const unsigned char*)p.q + off));
            }
        }
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int c = tid - 32 + j * kLoaders;
            if (c < kUnits) *(uint4*)(q_smem + swz(c >> 4, c & 15)) = v[j];
        }
    }
    __syncthreads();  // barriers initialised, Q tile visible

    uint32_t qa[MW][8][4];
#pragma unroll
    for (int w = 0; w < MW; ++w) {
        const int r = (mt0 + w) * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const int ch = ks * 2 + (lane >> 4);
            ldmatrix_x4(qa[w][ks][0], qa[w][ks][1], qa[w][ks][2], qa[w][ks][3], smem_u32(q_smem) + swz(r, ch));
        }
    }

    // Warp (mt, kg) scores page kg of every stage against its 16 rows (per m-tile), but accumulates O only for the kCG * 16
    // output columns it owns, over ALL pages of the stage: the P fragments of the stage's pages travel through shared
    // memory and the KV groups of an m-tile share one running maximum, so nothing has to be merged at the end.
    constexpr int kCG = 8 / KW;                    // 16-column groups of O per warp
    float o[MW][2 * kCG][4];
    float m_run[MW][2], l_run[MW][2];              // running maximum of rows g and g + 8 (log2 units) | this lane's share of the row sums
    int limit[MW][2];                              // last visible token of the two rows this thread holds
#pragma unroll
    for (int w = 0; w < MW; ++w) {
#pragma unroll
        for (int n = 0; n < 2 * kCG; ++n) { o[w][n][0] = o[w][n][1] = o[w][n][2] = o[w][n][3] = 0.f; }
        m_run[w][0] = m_run[w][1] = -INFINITY;
        l_run[w][0] = l_run[w][1] = 0.f;
        const int rA = row0 + (mt0 + w) * 16 + (lane >> 2);
        limit[w][0] = P + min(rA / G, q - 1);
        limit[w][1] = P + min((rA + 8) / G, q - 1);
    }
    // Per-lane ldmatrix offsets inside one page of the TMA layout [half 2][16 rows][128 B], where the
    // 16-byte unit u of row r sits at ((u ^ (r & 7)) << 4).  K (x4): row = nt*8 + lane%8, unit = (kp&1)*4 + lane/8.
    // V (x4.trans): row = lane%8 + 8*((lane/8)&1), unit = (cp&3)*2 + lane/16.
    const uint32_t k_x = ((lane >> 3) ^ (lane & 7));
    const uint32_t k_off[2] = {(uint32_t)((lane & 7) * 128 + (k_x << 4)), (uint32_t)((lane & 7) * 128 + ((k_x ^ 4u) << 4))};
    const uint32_t v_row = (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t v_x = (lane >> 4) ^ (lane & 7);
    uint32_t v_off[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v_off[j] = v_row * 128 + ((v_x ^ (uint32_t)(j << 1)) << 4);

    const int rg = lane >> 2;                      // this lane's rows in an m-tile: rg and rg + 8
    float* my_max = x_max + (mt0 * 16 + rg) * KW;  // x_max[mt][row][kg]; m-tile mt0 + w: + w * 16 * KW
    uint4* my_p = x_p + (mt0 * KW) * 32 + lane;    // x_p[mt][kg][lane]: page kg's P as the lanes' MMA A fragments; + w * KW * 32
    auto group_sync = [&]() { asm volatile("bar.sync %0, %1;\n" ::"r"(1 + mt0 / MW), "n"(32 * KW) : "memory"); };

    bool live = true;   // a warp whose wait gave up keeps meeting the others at the group barriers
#pragma unroll 1
    for (int stage = 0; stage < n_stages; ++stage) {
        const int slot = stage % NS;
        if (warp == 0) produce(stage + NS - 1);
        if (live) live = mbar_wait(full_bar(slot), (stage / NS) & 1, abort_flag, p.status, p.wait_limit_cycles);

        const int stage_tok0 = tok_begin + stage * kStageTokens;
        const int npg = live ? min(kKW, (tok_end - stage_tok0 + kPage - 1) / kPage) : 0;   // pages of this stage
        const int tok0 = stage_tok0 + kg * kPage;
        const bool has_page = kg < npg;
        const uint32_t stage_base = smem_base + slot * kStageBytes;
        float s[MW][2][4];
        float mx[MW][2];
#pragma unroll
        for (int w = 0; w < MW; ++w) mx[w][0] = mx[w][1] = -INFINITY;
        if (has_page) {
            const uint32_t k_base = stage_base + kg * 4096;
            const uint32_t v_base = k_base + kStageTokens * kRowBytes;
            // slots past the end of the sequence may hold anything: zero those V rows (P is 0 there,
            // but 0 * NaN is not).  Every warp that scores the page writes the same zeros.
            if (tok0 + kPage > L) {
                const int valid_rows = L - tok0;
                for (int idx = lane; idx < (kPage - valid_rows) * 16; idx += 32) {
                    const int r = valid_rows + (idx >> 4), ch = idx & 15;
                    *(uint4*)(ring + (v_base - smem_base) + (ch >> 3) * 2048 + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = make_uint4(0, 0, 0, 0);
                }
                __syncwarp();
            }
            // S = Q K^T for 16 tokens: two n-tiles of 8 tokens, as four accumulation chains of four MMAs each per m-tile
            // (even and odd k-steps of both n-tiles): a dependent mma.sync is slow to issue.  A K fragment serves every m-tile.
            float s_odd[MW][2][4];
#pragma unroll
            for (int w = 0; w < MW; ++w) {
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    s[w][nt][0] = s[w][nt][1] = s[w][nt][2] = s[w][nt][3] = 0.f;
                    s_odd[w][nt][0] = s_odd[w][nt][1] = s_odd[w][nt][2] = s_odd[w][nt][3] = 0.f;
                }
            }
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(b0, b1, b2, b3, k_base + (kp >> 1) * 2048 + nt * 1024 + k_off[kp & 1]);
#pragma unroll
                    for (int w = 0; w < MW; ++w) {
                        mma_bf16(s[w][nt], qa[w][2 * kp], b0, b1);
                        mma_bf16(s_odd[w][nt], qa[w][2 * kp + 1], b2, b3);
                    }
                }
            }
#pragma unroll
            for (int w = 0; w < MW; ++w) {
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) s[w][nt][e] += s_odd[w][nt][e];
                }
                // mask the causal edge / the end of the split (raw scores; the scale is folded into the exp)
                if ((tok0 + kPage - 1 > P) || (tok0 + kPage > tok_end)) {
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int tok = tok0 + nt * 8 + 2 * (lane & 3) + (e & 1);
                            if (tok > limit[w][e >> 1] || tok >= tok_end) s[w][nt][e] = -INFINITY;
                        }
                    }
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float v = fmaxf(fmaxf(s[w][0][2 * h], s[w][0][2 * h + 1]), fmaxf(s[w][1][2 * h], s[w][1][2 * h + 1]));
                    v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, 1));
                    v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, 2));
                    mx[w][h] = v * p.scale_log2;
                }
            }
        }
        if ((lane & 3) == 0) {
#pragma unroll
            for (int w = 0; w < MW; ++w) { my_max[w * 16 * KW + kg] = mx[w][0]; my_max[w * 16 * KW + 8 * KW + kg] = mx[w][1]; }
        }
        group_sync();   // the stage's page maxima of this warp's m-tiles are in place

        // one running maximum per row for a whole m-tile; P of this warp's page against it
#pragma unroll
        for (int w = 0; w < MW; ++w) {
            float corr[2];
            uint32_t pa[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float m_new = m_run[w][h];
#pragma unroll
                for (int k4 = 0; k4 < KW; k4 += 4) {
                    const float4 v = *(const float4*)(my_max + w * 16 * KW + h * 8 * KW + k4);
                    m_new = fmaxf(fmaxf(m_new, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
                }
                const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
                corr[h] = ex2(m_run[w][h] - m_ref);
                m_run[w][h] = m_new;
                float sum = 0.f;
                if (has_page) {
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        s[w][nt][2 * h] = ex2(fmaf(s[w][nt][2 * h], p.scale_log2, -m_ref));
                        s[w][nt][2 * h + 1] = ex2(fmaf(s[w][nt][2 * h + 1], p.scale_log2, -m_ref));
                        sum += s[w][nt][2 * h] + s[w][nt][2 * h + 1];
                    }
                }
                l_run[w][h] = l_run[w][h] * corr[h] + sum;
            }
            if (has_page) {
                pa[0] = pack_bf16(s[w][0][0], s[w][0][1]);
                pa[1] = pack_bf16(s[w][0][2], s[w][0][3]);
                pa[2] = pack_bf16(s[w][1][0], s[w][1][1]);
                pa[3] = pack_bf16(s[w][1][2], s[w][1][3]);
            }
            my_p[(w * KW + kg) * 32] = make_uint4(pa[0], pa[1], pa[2], pa[3]);
            if (__any_sync(0xFFFFFFFFu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
                for (int n = 0; n < 2 * kCG; ++n) {
                    o[w][n][0] *= corr[0]; o[w][n][1] *= corr[0];
                    o[w][n][2] *= corr[1]; o[w][n][3] *= corr[1];
                }
            }
        }
        group_sync();   // every page's P fragments (and zeroed V rows) are in place

        // O[:, this warp's columns] += P V over the stage's pages (a V fragment serves every m-tile)
#pragma unroll
        for (int k = 0; k < kKW; ++k) {
            if (k < npg) {
                uint4 pk[MW];
#pragma unroll
                for (int w = 0; w < MW; ++w) pk[w] = my_p[(w * KW + k) * 32];
                const uint32_t v_base = stage_base + kStageTokens * kRowBytes + k * 4096;
#pragma unroll
                for (int c = 0; c < kCG; ++c) {
                    const int cp = kg * kCG + c;
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b0, b1, b2, b3, v_base + (cp >> 2) * 2048 + v_off[cp & 3]);
#pragma unroll
                    for (int w = 0; w < MW; ++w) {
                        const uint32_t a[4] = {pk[w].x, pk[w].y, pk[w].z, pk[w].w};
                        mma_bf16(o[w][2 * c], a, b0, b1);
                        mma_bf16(o[w][2 * c + 1], a, b2, b3);
                    }
                }
            }
        }
        __syncwarp();
        if (live && lane == 0) mbar_arrive(empty_bar(slot));
    }

    // ---- row sums of the m-tile: each KV group's share through shared memory
#pragma unroll
    for (int w = 0; w < MW; ++w) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            l_run[w][h] += __shfl_xor_sync(0xFFFFFFFFu, l_run[w][h], 1);
            l_run[w][h] += __shfl_xor_sync(0xFFFFFFFFu, l_run[w][h], 2);
        }
        if ((lane & 3) == 0) {
            x_l[((mt0 + w) * 16 + rg) * KW + kg] = l_run[w][0];
            x_l[((mt0 + w) * 16 + rg + 8) * KW + kg] = l_run[w][1];
        }
    }
    // After a wait gave up, copies armed by the producer lane may still be on their way into the ring: it waits for
    // them (bounded by the clock alone) before the CTA reuses or releases that shared memory.
    if (tid == 0 && *abort_flag) {
        for (int s = max(0, last_armed - NS + 1); s <= last_armed; ++s)
            if (s != p.drop_stage) mbar_drain(full_bar(s % NS), (s / NS) & 1, p.wait_limit_cycles);
    }
    __syncthreads();  // all row sums in place; every armed stage has been consumed: the ring is dead

    // With clusters, the KV splits of this (sequence, KV head) are the cluster's CTAs (rank = split): the split
    // results stay in shared memory and are merged across the cluster below instead of going through global memory.
    const bool in_cluster = p.cluster_size > 1;
    float* cl_o = (float*)ring;                              // [MT*16][kD]
    float2* cl_ml = (float2*)(ring + MT * 16 * kD * 4);      // [MT*16]
#pragma unroll
    for (int wh = 0; wh < 2 * MW; ++wh) {
        const int w = wh >> 1, h = wh & 1;
        const int r = (mt0 + w) * 16 + rg + 8 * h;           // row of the CTA's chunk
        const unsigned int row_lanes = __ballot_sync(0xFFFFFFFFu, row0 + r < rows);   // (the four lanes of a row go together)
        if (row0 + r >= rows) continue;
        float l_all = 0.f;
#pragma unroll
        for (int k4 = 0; k4 < KW; k4 += 4) {
            const float4 v = *(const float4*)(x_l + r * KW + k4);
            l_all += (v.x + v.y) + (v.z + v.w);
        }
        const float m_all = m_run[w][h];
        const int i = (row0 + r) / G, hg = (row0 + r) - i * G;
        const int hd = g * G + hg;
        const bool first = kg == 0 && (lane & 3) == 0;       // one lane per row writes the row's (m, l)
        if (sp.nsplit == 1) {
            const float inv = 1.f / l_all;
            __nv_bfloat16* orow = (__nv_bfloat16*)p.out + ((long long)(sp.q_row0 + i) * p.hq + hd) * kD;
#pragma unroll
            for (int n = 0; n < 2 * kCG; ++n)
                *(uint32_t*)(orow + (kg * kCG * 2 + n) * 8 + 2 * (lane & 3)) = pack_bf16(o[w][n][2 * h] * inv, o[w][n][2 * h + 1] * inv);
            if (p.lse && first) p.lse[(long long)(sp.q_row0 + i) * p.hq + hd] = (m_all + log2f(l_all)) * 0.6931471805599453f;
        } else {
            if (in_cluster) {
                float* orow = cl_o + r * kD;
                if (first) cl_ml[r] = make_float2(m_all, l_all);
#pragma unroll
                for (int n = 0; n < 2 * kCG; ++n)
                    *(float2*)(orow + (kg * kCG * 2 + n) * 8 + 2 * (lane & 3)) = make_float2(o[w][n][2 * h], o[w][n][2 * h + 1]);
            } else {
                // split partial for the merge kernel, written past the L1 (read next by other SMs)
                const long long e = (long long)sp.part_base + ((long long)i * p.hq + hd) * sp.nsplit + split;
                if (first) p.part_ml[e] = make_float2(m_all, l_all);
                if (p.part_half) {
                    // the row divided by its own sum, as fp16 in the first 256 bytes of the entry's 512-byte slot (the merge
                    // weighs split k by l_k 2^(m_k - m)).  A lane holds two columns of each of two neighbouring 8-column
                    // tiles: lane pairs swap one pair each, so that every lane stores four consecutive columns (8 bytes) and
                    // the four lanes of a row write a whole 32-byte sector
                    const float inv = (l_all > 0.f) ? 1.f / l_all : 0.f;
                    unsigned char* orow = (unsigned char*)p.part_o + e * 512;
#pragma unroll
                    for (int c = 0; c < kCG; ++c) {
                        const __half2 lo = __floats2half2_rn(o[w][2 * c][2 * h] * inv, o[w][2 * c][2 * h + 1] * inv);
                        const __half2 hi = __floats2half2_rn(o[w][2 * c + 1][2 * h] * inv, o[w][2 * c + 1][2 * h + 1] * inv);
                        const unsigned int mine_lo = *reinterpret_cast<const unsigned int*>(&lo);
                        const unsigned int mine_hi = *reinterpret_cast<const unsigned int*>(&hi);
                        const bool odd = lane & 1;
                        const unsigned int got = __shfl_xor_sync(row_lanes, odd ? mine_lo : mine_hi, 1);
                        // even lane: its own columns of the first tile, then its partner's; odd lane: the same in the second tile
                        const uint2 pk = odd ? make_uint2(got, mine_hi) : make_uint2(mine_lo, got);
                        const int col = (kg * kCG + c) * 16 + (odd ? 8 : 0) + 4 * ((lane & 3) >> 1);
                        __stcg((uint2*)(orow + col * 2), pk);
                    }
                } else {   // the un-normalised fp32 row
                    float* orow = p.part_o + e * kD;
#pragma unroll
                    for (int n = 0; n < 2 * kCG; ++n)
                        __stcg((float2*)(orow + (kg * kCG * 2 + n) * 8 + 2 * (lane & 3)), make_float2(o[w][n][2 * h], o[w][n][2 * h + 1]));
                }
            }
        }
    }
    if (in_cluster && sp.nsplit > 1) {   // (uniform over the cluster: all its CTAs belong to one sequence)
        cluster_sync();   // every split's rows are in place
        const int cs = sp.nsplit;
        const int n_rows = min(rows - row0, MT * 16);
        // rows are dealt round-robin to the cluster's CTAs; one warp merges one row, lane k < cs holding split k's
        // (m, l), every lane four columns of each split's O row (all loads in flight at once)
        for (int r = split + warp * cs; r < n_rows; r += kWarps * cs) {
            float2 ml = make_float2(-INFINITY, 0.f);
            if (lane < cs) ml = ld_cluster_f2(cluster_map(smem_u32(cl_ml + r), lane));
            float m_all = ml.x;
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xFFFFFFFFu, m_all, d));
            const float w = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - m_all);
            float l_all = ml.y * w;
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) l_all += __shfl_xor_sync(0xFFFFFFFFu, l_all, d);
            const uint32_t row_addr = smem_u32(cl_o + r * kD + lane * 4);
            float4 v[16];
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if (k < cs) v[k] = ld_cluster_f4(cluster_map(row_addr, k));
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float wk = __shfl_sync(0xFFFFFFFFu, w, k);
                if (k < cs && wk != 0.f) { acc.x += v[k].x * wk; acc.y += v[k].y * wk; acc.z += v[k].z * wk; acc.w += v[k].w * wk; }
            }
            const int i = (row0 + r) / G, hg = (row0 + r) - i * G;
            const int h = g * G + hg;
            const float inv = 1.f / l_all;
            uint2 packed;
            packed.x = pack_bf16(acc.x * inv, acc.y * inv);
            packed.y = pack_bf16(acc.z * inv, acc.w * inv);
            *(uint2*)((__nv_bfloat16*)p.out + ((long long)(sp.q_row0 + i) * p.hq + h) * kD + lane * 4) = packed;
            if (p.lse && lane == 0) p.lse[(long long)(sp.q_row0 + i) * p.hq + h] = (m_all + log2f(l_all)) * 0.6931471805599453f;
        }
        cluster_sync();   // no CTA leaves while its rows may still be read
    }
}

// --------------------------------------------------------------------------------------------
// Scalar kernel for fp32 pools (any q; d = 64 or 128) and for bf16 pools with d = 64 (a correctness path: fp32 arithmetic
// on the FMA pipes).  CTA = 4 warps on one (sequence, row, head, split); a warp takes every 4th token, lanes split the head
// dim, dot products reduce by shuffle.
template <bool kBf16>
__device__ __forceinline__ float load_elem(const void* base, long long idx) {
    if (kBf16) return __bfloat162float(((const __nv_bfloat16*)base)[idx]);
    return ((const float*)base)[idx];
}
template <int D, bool kBf16>
__global__ void __launch_bounds__(128)
attn_simt_kernel(const __grid_constant__ AttnParams p) {
    constexpr int kPer = D / 32;
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int si = find_seq(p, blockIdx.x);
    const SeqPlan sp = p.seq[si];
    int local = blockIdx.x - sp.item0;  // ((i * Hq) + h) * nsplit + split
    const int split = local % sp.nsplit;
    local /= sp.nsplit;
    const int h = local % p.hq;
    const int i = local / p.hq;
    const int G = p.hq / p.hkv;
    const int g = h / G;
    const int tok_begin = split * sp.split_tokens;
    const int tok_end = min(sp.prefix_len + i + 1, tok_begin + sp.split_tokens);  // causal limit for row i
    const int* pt_row = p.page_table + (long long)sp.seq_index * p.pt_stride;

    float qv[kPer], acc[kPer];
    const long long q0 = ((long long)(sp.q_row0 + i) * p.hq + h) * D;
#pragma unroll
    for (int c = 0; c < kPer; ++c) { qv[c] = load_elem<kBf16>(p.q, q0 + lane + 32 * c) * p.scale_log2; acc[c] = 0.f; }
    float m = -INFINITY, l = 0.f;
    for (int tok = tok_begin + warp; tok < tok_end; tok += 4) {
        long long page = __ldg(pt_row + (tok >> 4));
        if (page < 0 || page >= p.num_pages) {
            if (lane == 0) atomicOr(p.status, AGX_DEV_BAD_PAGE);
            continue;
        }
        const long long base = ((page * p.hkv + g) * kPage + (tok & 15)) * (long long)D;
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < kPer; ++c) dot += qv[c] * load_elem<kBf16>(p.k_pool, base + lane + 32 * c);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, off);
        const float m_new = fmaxf(m, dot);
        const float corr = exp2f(m - m_new);
        const float w = exp2f(dot - m_new);
        l = l * corr + w;
#pragma unroll
        for (int c = 0; c < kPer; ++c) acc[c] = acc[c] * corr + w * load_elem<kBf16>(p.v_pool, base + lane + 32 * c);
        m = m_new;
    }
    __shared__ float sm_o[4][D];
    __shared__ float2 sm_ml[4];
#pragma unroll
    for (int c = 0; c < kPer; ++c) sm_o[warp][lane + 32 * c] = acc[c];
    if (lane == 0) sm_ml[warp] = make_float2(m, l);
    __syncthreads();
    for (int c = threadIdx.x; c < D; c += 128) {
        float m_all = -INFINITY;
#pragma unroll
        for (int k = 0; k < 4; ++k) m_all = fmaxf(m_all, sm_ml[k].x);
        float l_all = 0.f, a = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float w = (sm_ml[k].x == -INFINITY) ? 0.f : exp2f(sm_ml[k].x - m_all);
            l_all += sm_ml[k].y * w;
            a += sm_o[k][c] * w;
        }
        if (sp.nsplit == 1) {
            const long long o = ((long long)(sp.q_row0 + i) * p.hq + h) * D + c;
            if (kBf16) ((__nv_bfloat16*)p.out)[o] = __float2bfloat16_rn(a / l_all);
            else ((float*)p.out)[o] = a / l_all;
            if (p.lse && c == 0) p.lse[(long long)(sp.q_row0 + i) * p.hq + h] = (m_all + log2f(l_all)) * 0.6931471805599453f;
        } else {
            const long long e = (long long)sp.part_base + ((long long)i * p.hq + h) * sp.nsplit + split;
            p.part_o[e * D + c] = a;
            if (c == 0) p.part_ml[e] = make_float2(m_all, l_all);
        }
    }
}

// --------------------------------------------------------------------------------------------
// Combine: out[row, h] = sum_k O_k 2^(m_k - m) / sum_k l_k 2^(m_k - m), splits in index order.
// One warp per (row, head); lanes own 4 consecutive floats of each 128-wide chunk.
// kMaxNs: no sequence of the launch has more splits than this (4, 16, or any number).  Four O rows per warp instead of 32
// keep the register count low enough for ten CTAs per SM, which is what the partials of a split prefill need.
// kHalfPart: the partial rows are fp16 and already divided by their own sums l_k (the 256-row tensor-core schedule), so
// split k weighs l_k 2^(m_k - m) instead of 2^(m_k - m).
template <bool kHalfPart>
__device__ __forceinline__ float4 load_part4(const AttnParams& p, long long entry, int c4) {
    if (kHalfPart) {
        const uint2 raw = ld_volatile_u2((const unsigned char*)p.part_o + entry * 512 + c4 * 2);   // written by other SMs just before: past the L1
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        return make_float4(a.x, a.y, b.x, b.y);
    }
    return ld_volatile_f4(p.part_o + entry * p.head_dim + c4);
}
template <bool kBf16Out, int kMaxNs, bool kHalfPart>
__global__ void __launch_bounds__(128, kMaxNs <= 4 ? 10 : kMaxNs <= 16 ? 5 : 3)
attn_combine_kernel(const __grid_constant__ AttnParams p, int total_rows) {
    constexpr bool kFew = kMaxNs <= 16;          // no second batch of 16 rows
    constexpr int kInFlight = kMaxNs <= 4 ? 4 : 16;
    pdl_launch_dependents();
    // (everything up to the wait depends on the kernel arguments only and runs while the attention kernel drains)
    const int lane = threadIdx.x & 31;
    const int rh = blockIdx.x * 4 + (threadIdx.x >> 5);  // index over (local row, head) of the launch's sequences
    if (rh >= total_rows * p.hq) return;
    const int lrow = rh / p.hq, h = rh - lrow * p.hq;
    // sequences are laid out back to back in launch-local row order
    int si = 0, acc_rows = 0;
#pragma unroll 1
    for (int s = 0; s < p.num_seqs; ++s) {
        if (lrow >= acc_rows && lrow < acc_rows + p.seq[s].q_len) { si = s; break; }
        acc_rows += p.seq[s].q_len;
    }
    const SeqPlan sp = p.seq[si];
    if (sp.nsplit == 1) return;  // written directly by the attention kernel
    const int i = lrow - acc_rows;
    const long long e0 = (long long)sp.part_base + ((long long)i * p.hq + h) * sp.nsplit;
    const int ns = sp.nsplit;
    const int D = p.head_dim;
    const int c4 = lane * 4;               // each lane owns 4 output columns
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float m_all, l_all;
    pdl_wait();   // the partials are complete
    if (kMaxNs <= 32 || ns <= 32) {
        // One round trip to memory: lane k fetches (m, l) of split k while every lane already fetches its
        // columns of every split's O row; the weights then travel by shuffle, splits in index order.
        // (volatile loads: the compiler leaves them in this order, ahead of the first use of any of them)
        float2 ml = make_float2(-INFINITY, 0.f);
        if (lane < ns) ml = ld_volatile_f2(p.part_ml + e0 + lane);
        float4 v[kInFlight], v2[kFew ? 1 : 16];
#pragma unroll
        for (int j = 0; j < kInFlight; ++j)
            if (j < ns && c4 < D) v[j] = load_part4<kHalfPart>(p, e0 + j, c4);
        if (!kFew && ns > 16) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (16 + j < ns && c4 < D) v2[j] = load_part4<kHalfPart>(p, e0 + 16 + j, c4);
        }
        m_all = ml.x;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xFFFFFFFFu, m_all, off));
        const float e_mine = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - m_all);
        l_all = ml.y * e_mine;
        const float w_mine = kHalfPart ? l_all : e_mine;   // weight of this lane's split's O row
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) l_all += __shfl_xor_sync(0xFFFFFFFFu, l_all, off);
#pragma unroll
        for (int j = 0; j < kInFlight; ++j) {
            const float w = __shfl_sync(0xFFFFFFFFu, w_mine, j);
            if (j < ns && w != 0.f && c4 < D) {   // a split that saw no token for this row publishes only (m, l) = (-inf, 0)
                acc.x += v[j].x * w; acc.y += v[j].y * w; acc.z += v[j].z * w; acc.w += v[j].w * w;
            }
        }
        if (!kFew && ns > 16) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float w = __shfl_sync(0xFFFFFFFFu, w_mine, 16 + j);
                if (16 + j < ns && w != 0.f && c4 < D) {
                    acc.x += v2[j].x * w; acc.y += v2[j].y * w; acc.z += v2[j].z * w; acc.w += v2[j].w * w;
                }
            }
        }
    } else {
        // many splits: lanes take splits side by side for (m, l), then 4 O rows in flight at a time
        m_all = -INFINITY;
        for (int k = lane; k < ns; k += 32) m_all = fmaxf(m_all, p.part_ml[e0 + k].x);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xFFFFFFFFu, m_all, off));
        l_all = 0.f;
        for (int k = lane; k < ns; k += 32) {
            const float2 ml = p.part_ml[e0 + k];
            l_all += (ml.x == -INFINITY) ? 0.f : ml.y * exp2f(ml.x - m_all);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) l_all += __shfl_xor_sync(0xFFFFFFFFu, l_all, off);
        if (c4 < D) {
            int k = 0;
            for (; k + 4 <= ns; k += 4) {
                float w[4];
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 mlk = p.part_ml[e0 + k + j];
                    w[j] = (mlk.x == -INFINITY) ? 0.f : exp2f(mlk.x - m_all) * (kHalfPart ? mlk.y : 1.f);
                    v[j] = load_part4<kHalfPart>(p, e0 + k + j, c4);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (w[j] != 0.f) { acc.x += v[j].x * w[j]; acc.y += v[j].y * w[j]; acc.z += v[j].z * w[j]; acc.w += v[j].w * w[j]; }
                }
            }
            for (; k < ns; ++k) {
                const float2 mlk = p.part_ml[e0 + k];
                const float w = (mlk.x == -INFINITY) ? 0.f : exp2f(mlk.x - m_all) * (kHalfPart ? mlk.y : 1.f);
                const float4 v = load_part4<kHalfPart>(p, e0 + k, c4);
                if (w != 0.f) { acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w; }
            }
        }
    }
    const float inv = 1.f / l_all;
    const long long off = ((long long)(sp.q_row0 + i) * p.hq + h) * D + c4;
    if (c4 < D) {
        if (kBf16Out) {
            uint2 packed;
            packed.x = pack_bf16(acc.x * inv, acc.y * inv);
            packed.y = pack_bf16(acc.z * inv, acc.w * inv);
            *(uint2*)((__nv_bfloat16*)p.out + off) = packed;
        } else {
            *(float4*)((float*)p.out + off) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        }
    }
    if (p.lse && lane == 0) p.lse[(long long)(sp.q_row0 + i) * p.hq + h] = (m_all + log2f(l_all)) * 0.6931471805599453f;
}

// The same merge for the partials of the 256-row tensor-core schedule (fp16 rows divided by their own sums, at most 4
// splits): each warp takes two (row, head) pairs with all their loads in flight at once, so that the merge of a split
// prefill (12288 pairs, 9 MB of partials) is about one wave of CTAs and one memory round trip per warp instead of several
// waves of short-lived CTAs, and a larger merge has half the CTAs with twice the bytes in flight each.  (Measured: one /
// two / three / four pairs per warp give 29.1 / 19.8 / 20.5-21.6 / - us for the 65536 pairs of the long prefill under
// ncu; c3 29.9 / 29.9 / 31.0 us and (1500, 200) 17.8 / 18.3 / 19.3 us per call for two / three / four.)
constexpr int kCombineRows = 2;
__global__ void __launch_bounds__(128, 8)
attn_combine_half4_kernel(const __grid_constant__ AttnParams p, int total_rows) {
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int n_pairs = total_rows * p.hq;
    const int stride = gridDim.x * 4;
    const int rh0 = blockIdx.x * 4 + (threadIdx.x >> 5);
    long long e0[kCombineRows], out_off[kCombineRows];
    int ns[kCombineRows];
#pragma unroll
    for (int j = 0; j < kCombineRows; ++j) {
        const int rh = rh0 + j * stride;
        ns[j] = 0; e0[j] = 0; out_off[j] = 0;
        if (rh < n_pairs) {
            const int lrow = rh / p.hq, h = rh - lrow * p.hq;
            int si = 0, acc_rows = 0;
#pragma unroll 1
            for (int s = 0; s < p.num_seqs; ++s) {
                if (lrow >= acc_rows && lrow < acc_rows + p.seq[s].q_len) { si = s; break; }
                acc_rows += p.seq[s].q_len;
            }
            const SeqPlan& sp = p.seq[si];
            if (sp.nsplit > 1) {   // (a single split was written directly by the attention kernel)
                const int i = lrow - acc_rows;
                ns[j] = sp.nsplit;
                e0[j] = (long long)sp.part_base + ((long long)i * p.hq + h) * sp.nsplit;
                out_off[j] = (long long)(sp.q_row0 + i) * p.hq + h;
            }
        }
    }
    pdl_wait();   // the partials are complete
    float2 ml[kCombineRows];
    uint2 v[kCombineRows][4];
#pragma unroll
    for (int j = 0; j < kCombineRows; ++j) {
        ml[j] = make_float2(-INFINITY, 0.f);
        if (lane < ns[j]) ml[j] = ld_volatile_f2(p.part_ml + e0[j] + lane);
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (k < ns[j]) v[j][k] = ld_volatile_u2((const unsigned char*)p.part_o + (e0[j] + k) * 512 + lane * 8);
    }
#pragma unroll
    for (int j = 0; j < kCombineRows; ++j) {
        if (ns[j] == 0) continue;   // (uniform over the warp)
        float m_all = ml[j].x;
#pragma unroll
        for (int off = 2; off > 0; off >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xFFFFFFFFu, m_all, off));   // splits sit in lanes 0..3
        const float w_mine = (ml[j].x == -INFINITY) ? 0.f : exp2f(ml[j].x - m_all) * ml[j].y;
        float l_all = w_mine;
#pragma unroll
        for (int off = 2; off > 0; off >>= 1) l_all += __shfl_xor_sync(0xFFFFFFFFu, l_all, off);
        m_all = __shfl_sync(0xFFFFFFFFu, m_all, 0);
        l_all = __shfl_sync(0xFFFFFFFFu, l_all, 0);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float w = __shfl_sync(0xFFFFFFFFu, w_mine, k);
            if (k < ns[j] && w != 0.f) {   // a split that saw no token for this row publishes only (m, l) = (-inf, 0)
                const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v[j][k].x));
                const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v[j][k].y));
                acc.x += a.x * w; acc.y += a.y * w; acc.z += b.x * w; acc.w += b.y * w;
            }
        }
        const float inv = 1.f / l_all;
        uint2 packed;
        packed.x = pack_bf16(acc.x * inv, acc.y * inv);
        packed.y = pack_bf16(acc.z * inv, acc.w * inv);
        *(uint2*)((__nv_bfloat16*)p.out + out_off[j] * kD + lane * 4) = packed;
        if (p.lse && lane == 0) p.lse[out_off[j]] = (m_all + log2f(l_all)) * 0.6931471805599453f;
    }
}

// The same merge for the fp16 partials of the small-q kernel (5 to 32 KV splits): one (row, head) pair per warp, lane k
// holding split k's (m, l) and every lane four columns of every split's row, all loads in flight at once.  CTAs of two
// warps with few registers (12 or 8 CTAs per SM), so that the merge of a one-wave launch fits the few SMs the planner
// leaves out of the attention grid for it.
template <int kNsMax>
__global__ void __launch_bounds__(64, kNsMax <= 20 ? 12 : 8)
attn_combine_half32_kernel(const __grid_constant__ AttnParams p, int total_rows) {
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int rh = blockIdx.x * 2 + (threadIdx.x >> 5);
    int ns = 1, si = 0, acc_rows = 0, lrow = 0, h = 0;
    if (rh < total_rows * p.hq) {
        lrow = rh / p.hq; h = rh - lrow * p.hq;
#pragma unroll 1
        for (int s = 0; s < p.num_seqs; ++s) {
            if (lrow >= acc_rows && lrow < acc_rows + p.seq[s].q_len) { si = s; break; }
            acc_rows += p.seq[s].q_len;
        }
        ns = p.seq[si].nsplit;
    }
    if (ns > 1) {   // (a single split was written directly by the attention kernel)
        const SeqPlan& sp = p.seq[si];
        const int i = lrow - acc_rows;
        const long long e0 = (long long)sp.part_base + ((long long)i * p.hq + h) * ns;
        const long long out_off = (long long)(sp.q_row0 + i) * p.hq + h;
        const unsigned char* rows = (const unsigned char*)p.part_o + e0 * 512 + lane * 8;
        pdl_wait();   // the partials are complete
        // Every load is issued before the first use of any of them: volatile loads keep their place in the instruction stream
        // (left to itself the compiler moved the row loads behind the reduction of the maxima, i.e. behind a first trip to
        // memory: 0.6 us on decode verify).  No branch between the loads: slots past the last split repeat its row, and weigh
        // nothing below.
        uint2 v[kNsMax];
#pragma unroll
        for (int k = 0; k < kNsMax; ++k) v[k] = ld_volatile_u2(rows + min(k, ns - 1) * 512);
        float2 ml = make_float2(-INFINITY, 0.f);
        if (lane < ns) ml = ld_volatile_f2(p.part_ml + e0 + lane);
        float m_all = ml.x;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xFFFFFFFFu, m_all, off));
        const float w_mine = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - m_all) * ml.y;   // 0 in lanes past the last split
        float l_all = w_mine;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) l_all += __shfl_xor_sync(0xFFFFFFFFu, l_all, off);   // (a fixed order: reproducible)
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < kNsMax; ++k) {
            const float w = __shfl_sync(0xFFFFFFFFu, w_mine, k);
            // a split that saw no token for this row publishes only (m, l) = (-inf, 0): its row may hold anything, NaN included
            const bool use = w != 0.f;
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v[k].x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v[k].y));
            acc.x += use ? a.x * w : 0.f; acc.y += use ? a.y * w : 0.f; acc.z += use ? b.x * w : 0.f; acc.w += use ? b.y * w : 0.f;
        }
        const float inv = 1.f / l_all;
        uint2 packed;
        packed.x = pack_bf16(acc.x * inv, acc.y * inv);
        packed.y = pack_bf16(acc.z * inv, acc.w * inv);
        *(uint2*)((__nv_bfloat16*)p.out + out_off * kD + lane * 4) = packed;
        if (p.lse && lane == 0) p.lse[out_off] = (m_all + log2f(l_all)) * 0.6931471805599453f;
    }
}

// --------------------------------------------------------------------------------------------
namespace {
template <int MT, int KW, int NS>
constexpr int small_smem_bytes() {
    constexpr int kClusterBytes = MT * 16 * (kD * 4 + 8);
    constexpr int kRing = NS * 2 * KW * kPage * kRowBytes;
    constexpr int kExchange = 2 * MT * 16 * KW * 4 + MT * KW * 32 * 16;
    // [ring | cluster rows][Q tile][2 * NS barriers + abort flag][exchange area] + slack for the 1024-byte alignment
    return (kRing > kClusterBytes ? kRing : kClusterBytes) + MT * 16 * kRowBytes + 2 * NS * 8 + 16 + kExchange + 1024;
}

template <int MT, int KW, int NS, int MW = 1>
cudaError_t launch_small(const AttnParams& p, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
    constexpr int kSmem = small_smem_bytes<MT, KW, NS>();
    // the attribute is per device: remember which devices have it (a process normally drives one GPU)
    static bool configured_on[64] = {false};
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return cudaErrorInvalidDevice;
    bool& configured = configured_on[device];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(attn_small_bf16_kernel<MT, KW, NS, MW>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(attn_small_bf16_kernel<MT, KW, NS, MW>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);   // clusters of up to 16
        if (e != cudaSuccess) return e;
        configured = true;
    }
    if (p.cluster_size > 1)
        return launch_chained_cluster(attn_small_bf16_kernel<MT, KW, NS, MW>, dim3(p.num_items), dim3(32 * (MT / MW) * KW), kSmem,
                                      (unsigned)p.cluster_size, stream, p, map_k, map_v);
    return launch_chained(attn_small_bf16_kernel<MT, KW, NS, MW>, dim3(p.num_items), dim3(32 * (MT / MW) * KW), kSmem, stream, p, map_k, map_v);
}

template <int MT, int KW, int NS, int MW = 1>
int max_clusters(int cluster) {
    static int cached[64][17];   // 0 = not asked yet, else 1 + answer
    int device = 0;
    if (cluster < 2 || cluster > 16 || cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return 0;
    if (cached[device][cluster]) return cached[device][cluster] - 1;
    constexpr int kSmem = small_smem_bytes<MT, KW, NS>();
    int n = 0;
    if (cudaFuncSetAttribute(attn_small_bf16_kernel<MT, KW, NS, MW>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) == cudaSuccess &&
        cudaFuncSetAttribute(attn_small_bf16_kernel<MT, KW, NS, MW>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(cluster * 64); cfg.blockDim = dim3(32 * (MT / MW) * KW); cfg.dynamicSmemBytes = kSmem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n, attn_small_bf16_kernel<MT, KW, NS, MW>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    } else {
        (void)cudaGetLastError();
    }
    cached[device][cluster] = n + 1;
    return n;
}
}  // namespace

// 32-row blocks on 8-page stages: both m-tiles in every warp (8 warps; decode verify 9.84 -> 9.42 us) or, with AGX_SMALL_MW=1,
// one m-tile per warp (16 warps).  On 4-page stages two tiles per warp are slower (4 x 4096 verify 20.1 -> 20.3 us).
static bool two_tiles_per_warp() {
    static const bool on = !(getenv("AGX_SMALL_MW") && atoi(getenv("AGX_SMALL_MW")) == 1);
    return on;
}

int attn_small_max_clusters(int mt, int kw, int cluster) {
    if (mt == 2 && kw == 8 && two_tiles_per_warp()) return max_clusters<2, 8, 3, 2>(cluster);
    switch (mt * 16 + kw) {
        case 1 * 16 + 4: return max_clusters<1, 4, 3>(cluster);
        case 2 * 16 + 4: return max_clusters<2, 4, 3>(cluster);
        case 1 * 16 + 8: return max_clusters<1, 8, 3>(cluster);
        case 2 * 16 + 8: return max_clusters<2, 8, 3>(cluster);
        case 4 * 16 + 4: return max_clusters<4, 4, 5>(cluster);
        default: return 0;
    }
}

cudaError_t launch_attn_small_bf16(const AttnParams& p, int mt, int kw, const CUtensorMap& map_k, const CUtensorMap& map_v,
                                   cudaStream_t stream) {
    if (p.num_items == 0) return cudaSuccess;
    if (mt == 2 && kw == 8 && two_tiles_per_warp()) return launch_small<2, 8, 3, 2>(p, map_k, map_v, stream);
    switch (mt * 16 + kw) {
        case 1 * 16 + 4: return launch_small<1, 4, 3>(p, map_k, map_v, stream);
        case 2 * 16 + 4: return launch_small<2, 4, 3>(p, map_k, map_v, stream);
        case 1 * 16 + 8: return launch_small<1, 8, 3>(p, map_k, map_v, stream);
        case 2 * 16 + 8: return launch_small<2, 8, 3>(p, map_k, map_v, stream);
        case 4 * 16 + 4: return launch_small<4, 4, 5>(p, map_k, map_v, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_attn_simt(const AttnParams& p, int dtype, cudaStream_t stream) {
    if (p.num_items == 0) return cudaSuccess;
    if (dtype == AGX_F32 && p.head_dim == 64) return launch_chained(attn_simt_kernel<64, false>, dim3(p.num_items), dim3(128), 0, stream, p);
    if (dtype == AGX_F32 && p.head_dim == 128) return launch_chained(attn_simt_kernel<128, false>, dim3(p.num_items), dim3(128), 0, stream, p);
    if (dtype == AGX_BF16 && p.head_dim == 64) return launch_chained(attn_simt_kernel<64, true>, dim3(p.num_items), dim3(128), 0, stream, p);
    return cudaErrorInvalidValue;
}

cudaError_t launch_attn_combine(const AttnParams& p, int dtype, int total_rows, cudaStream_t stream) {
    const long long n = (long long)total_rows * p.hq;
    if (n == 0) return cudaSuccess;
    const int blocks = (int)((n + 3) / 4);
    int ns_max = 1;
    for (int i = 0; i < p.num_seqs; ++i) ns_max = p.seq[i].nsplit > ns_max ? p.seq[i].nsplit : ns_max;
    if (dtype == AGX_BF16 && p.part_half) {
        if (ns_max <= 4) {
            // CTAs whose warps take kCombineRows pairs each
            const int want = (int)((n + 4 * kCombineRows - 1) / (4 * kCombineRows));
            return launch_chained(attn_combine_half4_kernel, dim3(want > 0 ? want : 1), dim3(128), 0, stream, p, total_rows);
        }
        if (ns_max <= 32) {
            if (ns_max <= 8) return launch_chained(attn_combine_half32_kernel<8>, dim3((int)((n + 1) / 2)), dim3(64), 0, stream, p, total_rows);
            if (ns_max <= 12) return launch_chained(attn_combine_half32_kernel<12>, dim3((int)((n + 1) / 2)), dim3(64), 0, stream, p, total_rows);
            if (ns_max <= 20) return launch_chained(attn_combine_half32_kernel<20>, dim3((int)((n + 1) / 2)), dim3(64), 0, stream, p, total_rows);
            return launch_chained(attn_combine_half32_kernel<32>, dim3((int)((n + 1) / 2)), dim3(64), 0, stream, p, total_rows);
        }
        return launch_chained(attn_combine_kernel<true, 1 << 30, true>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
    }
    if (dtype == AGX_BF16) {
        if (ns_max <= 4) return launch_chained(attn_combine_kernel<true, 4, false>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
        if (ns_max <= 16) return launch_chained(attn_combine_kernel<true, 16, false>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
        return launch_chained(attn_combine_kernel<true, 1 << 30, false>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
    }
    if (ns_max <= 4) return launch_chained(attn_combine_kernel<false, 4, false>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
    if (ns_max <= 16) return launch_chained(attn_combine_kernel<false, 16, false>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
    return launch_chained(attn_combine_kernel<false, 1 << 30, false>, dim3(blocks), dim3(128), 0, stream, p, total_rows);
}

}  // namespace agx
