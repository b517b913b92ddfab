// Large-q attention over a paged KV cache: the uncached suffix of a prompt attending over its cached
// prefix plus itself (Sec. 2.3, prefix caching; Sec. 4.2 makes the suffix a few hundred tokens over a
// prefix of thousands).  Here Q K^T and P V are dense contractions, so they run on the 5th-generation
// tensor cores: tcgen05.mma issued by one thread, operands staged in shared memory by TMA,
// accumulators in tensor memory (TMEM).
//
// Work item = (sequence, KV head g, chunk of 256 query rows, KV split).  The q * G rows of one KV
// head (row r = i * G + h % G) are cut into two 128-row tiles A and B that share every K/V tile.
// CTA = 12 warps:
//   warp 0      TMA producer: per 128-token tile, 8 pages x 2 boxes of [16 tokens][64 dims] for K and
//               for V (SWIZZLE_128B), page ids read through the page table; 2-stage rings.
//   warp 1      MMA issuer (one lane) and TMEM owner.  Order on the tensor pipe:
//               S_A(0) S_B(0) | O_A+=P_A V(t)  S_A(t+1)  O_B+=P_B V(t)  S_B(t+1) | ...
//               so the softmax of one tile overlaps the MMAs of the other.
//   warps 4-7   softmax of tile A, warps 8-11 softmax of tile B: one thread per query row (TMEM lane).
//               The whole 128-column score row is held in registers (the two softmax warpgroups take
//               registers from warps 0-3 with setmaxnreg), so S is read from TMEM once: row maximum,
//               exponentials with packed f32x2 arithmetic, P written back over S as packed bf16 (the A
//               operand of the P V MMA comes from TMEM), O rescaled in TMEM only when the row maximum
//               grew by more than 2^8.
// The Q tiles arrive by cp.async from warps 2-11 while warp 0 already streams K/V; results leave through
// a per-warp shared-memory staging area so that global stores are whole rows.
// TMEM columns: S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512).
// Every mbarrier wait is bounded: on time-out the CTA records AGX_DEV_WAIT_TIMEOUT and tears down.
#include <cuda.h>
#include <math.h>

#include "agx_internal.cuh"
#include "agx_sm100.cuh"

namespace agx {

namespace {

constexpr int kD = 128;
constexpr int kBN = 128;                    // KV tokens per tile
constexpr int kStagesK = 3;                 // K is wanted right after the previous tile's softmax: one more stage
// Two schedules share the kernel (template parameter kStreams):
//   false  two 128-row Q tiles A and B per CTA (256 rows), both meet every KV tile;
//   true   ONE 128-row Q tile per CTA (verify blocks and short suffixes: q * G <= 128 rows, most of them
//          padding); the two softmax warpgroups take the even and the odd KV tiles of the same rows, each with
//          its own S and O accumulators in TMEM, and are merged inside the CTA at the end.  The step is
//          HBM-bound, so the padded MMA rows cost nothing that matters, while every K/V byte is read once
//          and the softmax of one tile hides behind the MMAs and copies of the next.
template <bool kStreams> struct Sched {
    static constexpr int kRows = kStreams ? 128 : 256;     // query rows per CTA
    static constexpr int kStagesV = kStreams ? 3 : 2;      // the second Q tile's shared memory becomes a V stage
};
constexpr int kThreads = 384;
constexpr uint32_t kTileBytes = 128 * 256;  // one operand tile: [2 halves of 64 dims][128 rows][128 B]
constexpr uint32_t kHalfBytes = 128 * 128;
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = 2 * kTileBytes;
constexpr uint32_t kOffV = kOffK + kStagesK * kTileBytes;
constexpr uint32_t kOffBar = kOffV + 2 * kTileBytes;
// V stage s: the first two behind the K ring, the third (kStreams only) in the unused second Q tile
__host__ __device__ constexpr uint32_t v_stage_off(int s) { return s < 2 ? kOffV + s * kTileBytes : kOffQ + kTileBytes; }
constexpr uint32_t kOffPark = kOffK + 2 * kTileBytes;   // kStreams epilogue: stream 1's O rows (64 KB), then its (m, l)
constexpr uint32_t kOffCtx = kOffBar + 256;            // what the epilogue needs to know, parked at kernel start
constexpr uint32_t kSmemBytes = kOffBar + 512 + 1024;  // + barriers + epilogue context + alignment slack
constexpr float kRescaleThreshold = 8.0f;              // log2 units
// Of every 8 column pairs, this many take the polynomial 2^x instead of the special-function unit.
// Measured on B200 (P = 30720, q = 2048): 0 -> 950 us, 1 -> 957, 2 -> 964, 4 -> 982: the extra FMA-pipe
// instructions cost more issue slots (shared with the MMA-issuing warp) than the special-function unit
// gives back, so the default is 0 and the option only remains for experiments.
#ifndef AGX_POLY_PAIRS
#define AGX_POLY_PAIRS 0
#endif
constexpr int kPolyPairsOf8 = AGX_POLY_PAIRS;

// barrier slots (8 bytes each)
enum { BAR_K_FULL = 0, BAR_K_EMPTY = 3, BAR_V_FULL = 6, BAR_V_EMPTY = 9, BAR_S_FULL = 12, BAR_P_READY = 14,
       BAR_O_FULL = 16, BAR_Q_FULL = 17, BAR_P_TAIL = 18, BAR_CTX = 20, BAR_COUNT = 21 };
// P is handed to the MMA warp in two parts: the first kPvHeadSteps k-steps (16 tokens each) as soon as they are
// stored, so that their PV MMAs run while the softmax warpgroup still works on the last columns
constexpr int kPvHeadSteps = 6;
constexpr int kQLoadThreads = kThreads - 64;  // warps 2..11 bring the Q tiles in
constexpr int kRegsLow = 96, kRegsHigh = 200; // 128 * 96 + 256 * 200 <= 384 * 168

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256;  // + 128 * tile

// tcgen05 instruction descriptor, kind::f16: D = f32, A = B = bf16, M = 128, N = 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;              // A, B both K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16); // B (= V) is MN-major

// shared-memory matrix descriptor, SWIZZLE_128B, descriptor version 1
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_st_x16(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n"
                 :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]));
}
__device__ __forceinline__ void tmem_st_x32(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
                 :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]));
}


// Packed pairs of floats in one 64-bit register, for the f32x2 arithmetic instructions.
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;\n" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2p(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2p(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^x for a packed pair on the FMA pipes instead of the special-function unit: n = round(x) by the
// 1.5 * 2^23 trick, f = x - n in [-0.5, 0.5], 2^f by a cubic fitted to minimise the maximum relative
// error on that interval (7.5e-5, far below the 2^-9 rounding of P to bfloat16), then n is added
// into the exponent field.  x is clamped at -126 so the exponent cannot wrap.
__device__ __forceinline__ void ex2_poly2(uint64_t x, float& p0, float& p1) {
    float x0, x1;
    upk2(x, x0, x1);
    x = pk2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
    const uint64_t magic = pk2(12582912.f, 12582912.f), neg_magic = pk2(-12582912.f, -12582912.f);
    const uint64_t t = add2p(x, magic);
    const uint64_t n = add2p(t, neg_magic);
    const uint64_t f = fma2p(n, pk2(-1.f, -1.f), x);
    uint64_t q = fma2p(f, pk2(0.0551716648042202f, 0.0551716648042202f), pk2(0.2426111251115799f, 0.2426111251115799f));
    q = fma2p(q, f, pk2(0.6932609677314758f, 0.6932609677314758f));
    q = fma2p(q, f, pk2(0.9999280571937561f, 0.9999280571937561f));
    float q0, q1, t0, t1;
    upk2(q, q0, q1);
    upk2(t, t0, t1);
    p0 = __int_as_float(__float_as_int(t0) * 8388608 + __float_as_int(q0));
    p1 = __int_as_float(__float_as_int(t1) * 8388608 + __float_as_int(q1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {
    upk2(add2p(pk2(d0, d1), pk2(a0, a1)), d0, d1);
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

__device__ __forceinline__ int find_seq(const AttnParams& p, int item) {
    int s = 0;
#pragma unroll 1
    for (int i = 1; i < p.num_seqs; ++i)
        if (p.seq[i].item0 <= item) s = i;
    return s;
}

// What one CTA works on, derived from its block index alone.
struct TileItem {
    int g, G, P, q, rows, row0, split, nsplit, n_tiles, kv_begin, kv_end, vis_end, q_row0, seq_index;
};
// Everything the epilogue needs, kept in shared memory: kernel parameters reached through a pointer are
// slow to read, and registers are too precious across the main loop.
struct EpiCtx {
    TileItem it;
    int part_base, hq;
    int part_half;   // split partials leave as fp16 rows divided by their own sums (always so on the 256-row schedule)
    void* out;
    float* part_o;
    float2* part_ml;
    float* lse;
    unsigned long long magic;   // (row * magic) >> 32 == row / G exactly for rows < 2^22
};
template <bool kStreams>
__device__ __forceinline__ TileItem locate_item(const AttnParams& p, int block) {
    constexpr int kRowsPerCta = Sched<kStreams>::kRows;
    const int si = find_seq(p, block);
    const SeqPlan& sp = p.seq[si];
    TileItem it;
    int local = block - sp.item0;  // ((g * row_chunks) + rc) * nsplit + split
    it.nsplit = sp.nsplit;
    it.split = local % sp.nsplit;
    local /= sp.nsplit;
    const int rc = local % sp.row_chunks;
    it.g = local / sp.row_chunks;
    it.G = p.hq / p.hkv;
    it.P = sp.prefix_len; it.q = sp.q_len;
    it.rows = it.q * it.G;
    it.row0 = rc * kRowsPerCta;
    it.vis_end = it.P + min(it.q - 1, (it.row0 + kRowsPerCta - 1) / it.G) + 1;  // tokens the chunk's last row sees
    it.kv_begin = it.split * sp.split_tokens;
    it.kv_end = min(it.vis_end, it.kv_begin + sp.split_tokens);
    it.n_tiles = max(0, (it.kv_end - it.kv_begin + kBN - 1) / kBN);
    it.q_row0 = sp.q_row0; it.seq_index = sp.seq_index;
    return it;
}

// Epilogue of a softmax thread: the un-normalised fp32 O row leaves TMEM through this warp's 16 KB of
// the (now idle) K/V rings, so that global stores are whole rows written by whole warps.  With a single
// KV split the rows are normalised and written as bf16; otherwise fp32 partials and (m, l) go to the
// workspace for the combine kernel.  Kept out of line, and re-deriving its indices from the block index,
// so that nothing but its few arguments has to stay alive across the register-hungry main loop.
template <bool kStreams>
__device__ __noinline__ void tile_epilogue(unsigned char* smem, uint32_t tO, float m_ref, float l_run, bool ok) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    {   // the context is written by another warp at kernel start: wait for its arrival (long complete, normally)
        const uint32_t ctx_bar = smem_u32(smem) + kOffBar + 8u * BAR_CTX;
        volatile int* abort_flag = (volatile int*)(smem + kOffBar + BAR_COUNT * 8);
        if (!mbar_wait(ctx_bar, 0, abort_flag, nullptr, *(const long long*)(smem + kOffBar + BAR_COUNT * 8 + 16))) ok = false;
    }
    const EpiCtx cx = *(const EpiCtx*)(smem + kOffCtx);
    const TileItem& it = cx.it;
    const bool warp_has_rows = it.row0 + ((warp & 3) << 5) + (kStreams ? 0 : ((warp - 4) >> 2) * 128) < it.rows;
    float w_own = 1.f, w_other = 0.f;   // kStreams: weights of the two streams' accumulators
    if (kStreams) {
        // Stream 1 (warps 8-11) parks its rows in shared memory; stream 0 (warps 4-7) adds them to its own.
        const int rt = ((warp & 3) << 5) + lane;
        unsigned char* park = smem + kOffPark + rt * 512;
        float2* park_ml = (float2*)(smem + kOffPark + 128 * 512);
        if (warp >= 8 && ok && warp_has_rows) {
            tc_fence_after();
            uint32_t oreg[32];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                tmem_ld_x32(tO + c4 * 32, oreg);
                tmem_wait_ld();
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *(uint4*)(park + (((c4 * 8 + v) ^ lane) << 4)) = make_uint4(oreg[4 * v], oreg[4 * v + 1], oreg[4 * v + 2], oreg[4 * v + 3]);
            }
            park_ml[rt] = make_float2(m_ref, l_run);
        }
        // every softmax thread reaches this barrier, also after a bounded wait gave up somewhere in the CTA
        asm volatile("bar.sync 1, 256;\n" ::: "memory");
        if (warp >= 8 || !ok || !warp_has_rows || *(volatile int*)(smem + kOffBar + BAR_COUNT * 8)) return;
        const float2 other = park_ml[rt];
        const float m_new = fmaxf(m_ref, other.x);
        w_own = (m_ref == -INFINITY) ? 0.f : ex2(m_ref - m_new);
        w_other = (other.x == -INFINITY) ? 0.f : ex2(other.x - m_new);
        l_run = l_run * w_own + other.y * w_other;
        m_ref = m_new;
    }
    if (!warp_has_rows) return;
    unsigned char* stage = smem + kOffK + (warp - 4) * 16384;    // [32 rows][512 B], 16-byte units XOR-swizzled by row
    const int r_warp0 = it.row0 + (warp - 4) * 32;               // first row of this warp
    const uint64_t magic = cx.magic;                             // (row * magic) >> 32 == row / G exactly for rows < 2^22
    const bool single = it.nsplit == 1;
    const float inv = (l_run > 0.f) ? 1.f / l_run : 0.f;
    // per-row scalars, and the row's destination: lane j works them out for row j once, the copy loop below fetches
    // them by shuffle (a single warp doing the index arithmetic row by row took longer than the copies themselves)
    unsigned long long row_dst = 0;
    {
        const int r = r_warp0 + lane;
        if (r < it.rows) {
            const int i = (int)(((uint64_t)(uint32_t)r * magic) >> 32), h = it.g * it.G + (r - i * it.G);
            if (single) {
                if (cx.lse) cx.lse[(long long)(it.q_row0 + i) * cx.hq + h] = (m_ref + log2f(l_run)) * 0.6931471805599453f;
                row_dst = (unsigned long long)((unsigned char*)cx.out + ((long long)(it.q_row0 + i) * cx.hq + h) * 256);
            } else {
                const long long e = (long long)cx.part_base + ((long long)i * cx.hq + h) * it.nsplit + it.split;
                cx.part_ml[e] = make_float2(m_ref, l_run);
                row_dst = (unsigned long long)(cx.part_o + e * kD);
            }
        }
    }
    tc_fence_after();
    {
        uint32_t oreg[64];   // two 32-column chunks per TMEM round trip
#pragma unroll
        for (int c8 = 0; c8 < 4; c8 += 2) {
            tmem_ld_x32(tO + c8 * 32, oreg);
            tmem_ld_x32(tO + c8 * 32 + 32, oreg + 32);
            tmem_wait_ld();
            if (kStreams) {
                const unsigned char* park = smem + kOffPark + ((((warp & 3) << 5) + lane) * 512);
#pragma unroll
                for (int v = 0; v < 16; ++v) {
                    const float4 o1 = *(const float4*)(park + (((c8 * 8 + v) ^ lane) << 4));
                    oreg[4 * v + 0] = __float_as_uint(__uint_as_float(oreg[4 * v + 0]) * w_own + (w_other != 0.f ? o1.x * w_other : 0.f));
                    oreg[4 * v + 1] = __float_as_uint(__uint_as_float(oreg[4 * v + 1]) * w_own + (w_other != 0.f ? o1.y * w_other : 0.f));
                    oreg[4 * v + 2] = __float_as_uint(__uint_as_float(oreg[4 * v + 2]) * w_own + (w_other != 0.f ? o1.z * w_other : 0.f));
                    oreg[4 * v + 3] = __float_as_uint(__uint_as_float(oreg[4 * v + 3]) * w_own + (w_other != 0.f ? o1.w * w_other : 0.f));
                }
            }
            const bool half_part = kStreams && !single && cx.part_half;
            if (single || !kStreams || half_part) {   // (the 256-row schedule normalises its split partials too: they leave as fp16)
#pragma unroll
                for (int c = 0; c < 64; ++c) oreg[c] = __float_as_uint(__uint_as_float(oreg[c]) * inv);
            }
            if (kStreams) {
                // one warp with at most 32 rows: each lane stores its own row straight from registers (16 KB in all;
                // staging it through shared memory for whole-row stores took a single warp longer than these do)
                if (row_dst) {
#pragma unroll
                    for (int v = 0; v < 16; ++v) {
                        if (single) {
                            uint2 pk;
                            pk.x = pack_bf16(__uint_as_float(oreg[4 * v]), __uint_as_float(oreg[4 * v + 1]));
                            pk.y = pack_bf16(__uint_as_float(oreg[4 * v + 2]), __uint_as_float(oreg[4 * v + 3]));
                            *(uint2*)((unsigned char*)row_dst + (c8 * 8 + v) * 8) = pk;
                        } else if (half_part) {
                            uint2 pk;
                            pk.x = pack_f16(__uint_as_float(oreg[4 * v]), __uint_as_float(oreg[4 * v + 1]));
                            pk.y = pack_f16(__uint_as_float(oreg[4 * v + 2]), __uint_as_float(oreg[4 * v + 3]));
                            __stcg((uint2*)((unsigned char*)row_dst + (c8 * 8 + v) * 8), pk);
                        } else {
                            __stcg((uint4*)((unsigned char*)row_dst + (c8 * 8 + v) * 16),
                                   make_uint4(oreg[4 * v], oreg[4 * v + 1], oreg[4 * v + 2], oreg[4 * v + 3]));
                        }
                    }
                }
            } else {
                // pack to the 16-bit output format first (bf16 results, fp16 split partials): 256 bytes per row go through
                // the staging area, 16-byte units XOR-swizzled by row
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    uint4 pk;
                    if (single) {
                        pk.x = pack_bf16(__uint_as_float(oreg[8 * v + 0]), __uint_as_float(oreg[8 * v + 1]));
                        pk.y = pack_bf16(__uint_as_float(oreg[8 * v + 2]), __uint_as_float(oreg[8 * v + 3]));
                        pk.z = pack_bf16(__uint_as_float(oreg[8 * v + 4]), __uint_as_float(oreg[8 * v + 5]));
                        pk.w = pack_bf16(__uint_as_float(oreg[8 * v + 6]), __uint_as_float(oreg[8 * v + 7]));
                    } else {
                        pk.x = pack_f16(__uint_as_float(oreg[8 * v + 0]), __uint_as_float(oreg[8 * v + 1]));
                        pk.y = pack_f16(__uint_as_float(oreg[8 * v + 2]), __uint_as_float(oreg[8 * v + 3]));
                        pk.z = pack_f16(__uint_as_float(oreg[8 * v + 4]), __uint_as_float(oreg[8 * v + 5]));
                        pk.w = pack_f16(__uint_as_float(oreg[8 * v + 6]), __uint_as_float(oreg[8 * v + 7]));
                    }
                    *(uint4*)(stage + lane * 256 + ((((c8 >> 1) * 8 + v) ^ (lane & 15)) << 4)) = pk;
                }
            }
        }
    }
    if (kStreams) return;
    __syncwarp();
    // a half-warp writes one 256-byte row per instruction (lane j moves 16-byte unit j % 16 of row 2 u + j / 16); eight
    // row pairs' loads are in flight before the first store
    const int n_valid = min(32, it.rows - r_warp0);
    for (int rl0 = 0; rl0 < n_valid; rl0 += 16) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int rl = rl0 + 2 * u + (lane >> 4);
            v[u] = *(const uint4*)(stage + rl * 256 + (((lane & 15) ^ (rl & 15)) << 4));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int rl = rl0 + 2 * u + (lane >> 4);
            const unsigned long long dst = __shfl_sync(0xFFFFFFFFu, row_dst, rl & 31);
            if (rl < n_valid) {
                if (single) *(uint4*)((unsigned char*)dst + (lane & 15) * 16) = v[u];
                else __stcg((uint4*)((unsigned char*)dst + (lane & 15) * 16), v[u]);   // split partial: read next by other SMs
            }
        }
    }
}

}  // namespace

template <bool kStreams>
__global__ void __launch_bounds__(kThreads, 1)
attn_tile_bf16_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile int* abort_flag = (volatile int*)(smem + kOffBar + BAR_COUNT * 8);
    uint32_t* tmem_slot = (uint32_t*)(smem + kOffBar + BAR_COUNT * 8 + 8);
    auto bar = [&](int i) { return smem_base + kOffBar + 8u * i; };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    constexpr int kRowsPerCta = Sched<kStreams>::kRows;
    constexpr int kStagesV = Sched<kStreams>::kStagesV;
    // ---- work item
    const TileItem it = locate_item<kStreams>(p, blockIdx.x);
    const SeqPlan& sp = p.seq[find_seq(p, blockIdx.x)];
    const int split = it.split, g = it.g, G = it.G, P = it.P, q = it.q, L = P + q, rows = it.rows, row0 = it.row0;
    const int kv_begin = it.kv_begin, kv_end = it.kv_end, n_tiles = it.n_tiles;

    pdl_launch_dependents();
    if (n_tiles == 0) {  // nothing visible in this split (nsplit > 1 by construction): publish (m, l) = (-inf, 0);
                         // the combine kernel does not read the O rows of such entries
        pdl_wait();
        for (int rl = tid; rl < kRowsPerCta; rl += kThreads) {
            const int r = row0 + rl;
            if (r >= rows) break;
            const int i = r / G, h = g * G + (r - i * G);
            p.part_ml[(long long)sp.part_base + ((long long)i * p.hq + h) * sp.nsplit + split] = make_float2(-INFINITY, 0.f);
        }
        return;
    }

    // ---- setup: barriers, TMEM, Q tiles
    if (tid == 0) {
        for (int i = 0; i < BAR_COUNT; ++i)
            mbar_init(bar(i), (i == BAR_P_READY || i == BAR_P_READY + 1 || i == BAR_P_TAIL || i == BAR_P_TAIL + 1) ? 128u : (i == BAR_Q_FULL) ? (uint32_t)kQLoadThreads : 1u);
        *abort_flag = 0;
        *(long long*)(smem + kOffBar + BAR_COUNT * 8 + 16) = p.wait_limit_cycles;   // for the out-of-line epilogue
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&map_v) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    // Early loads: with p.early_prefix the caller vouches that the page table and the K/V pages below the cached-prefix
    // length are not written by any launch still in flight, so the producer warp may fetch them while the launch in
    // front of this one drains.  A CTA that first stores block rows of its own (fused append) keeps to the usual order.
    const bool own_rows = p.k_new && kv_begin < L && kv_begin + sp.split_tokens > P;
    const bool early_cta = p.early_prefix && !own_rows;
    if (!(warp == 0 && early_cta)) pdl_wait();   // from here on global memory written by the launch before this one is read (Q, page table, K/V)
    // fused append (one row chunk per sequence): the block's own K/V rows of this split go into the pages first
    if (own_rows && warp >= 2) append_rows_bf16(p, sp, g, kv_begin, kv_begin + sp.split_tokens, tid - 64, kQLoadThreads);
    // Q: 256 rows x 256 B by 16-byte cp.async (all of a thread's copies in flight at once), written in
    // the 128-byte-swizzled K-major operand layout; rows past q * G are zero-filled.
    if (warp >= 2) {
        for (int c = tid - 64; c < kRowsPerCta * 16; c += kQLoadThreads) {   // kStreams: one tile
            const int rl = c >> 4, ch = c & 15;     // row in chunk, 16-byte chunk of the 256-byte row
            const int r = row0 + rl;
            const bool valid = r < rows;
            const int rr = valid ? r : 0;
            const int i = (int)(((uint64_t)(uint32_t)rr * p.row_div_magic) >> 32), hg = rr - i * G;   // rr / G without the division
            const unsigned char* src = (const unsigned char*)p.q + (((long long)(sp.q_row0 + i) * p.hq + g * G + hg) * 256 + ch * 16);
            const int tile = rl >> 7, rt = rl & 127, half = ch >> 3, u = ch & 7;
            cp_async_16(smem_base + kOffQ + tile * kTileBytes + half * kHalfBytes + rt * 128 + ((u ^ (rt & 7)) << 4), src, valid ? 16u : 0u);
        }
    }
    // Barriers initialised, TMEM address published.  Warp 0 (which set the barriers up and needs nothing
    // from the others) only signals and goes straight to the page table and its first K/V copies.
    tc_fence_before();
    if (warp == 0 && !own_rows) { __syncwarp(); asm volatile("bar.arrive 2, %0;\n" ::"n"(kThreads) : "memory"); }   // (a fused append must land first)
    else asm volatile("bar.sync 2, %0;\n" ::"n"(kThreads) : "memory");
    tc_fence_after();
    const uint32_t tmem_base = (warp == 0) ? 0u : *tmem_slot;
    if (warp >= 2) {
        asm volatile("cp.async.wait_all;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        mbar_arrive(bar(BAR_Q_FULL));
    }
    auto pages_in_tile = [&](int t) { return min(8, (kv_end - (kv_begin + t * kBN) + kPage - 1) / kPage); };

    // the softmax warpgroups keep a whole score row in registers: warps 0-3 hand registers over to them
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsLow));
    if (warp == 0) {
        // ================= TMA producer: lane l of the warp copies page l of the tile =================
        const int* pt_row = p.page_table + (long long)sp.seq_index * p.pt_stride;
        const int page0 = kv_begin / kPage;
        const int n_pages_total = (kv_end - kv_begin + kPage - 1) / kPage;
        int ids = 0;  // page ids of the current group of 4 tiles: lane l holds page (group * 32 + l)
        bool ok = true;
        bool waited = !early_cta;       // has this warp passed the dependency wait?
        const int stable_end = P & ~(kPage - 1);   // tokens below this sit in pages no append of this block touches
        int last_k = -1, last_v = -1;   // last tiles whose copies were armed (for the drain below)
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int tok0 = kv_begin + t * kBN;
            const bool stable = tok0 + kBN <= stable_end;
            // K/V tiles wholly inside the cached prefix, as far as free stages go, may be requested before the wait
            if (!waited && !(stable && t < kStagesK)) { pdl_wait(); waited = true; }
            if ((t & 3) == 0) {
                const int pi = t * 8 + lane;
                long long id = 0;
                if (pi < n_pages_total) {
                    id = __ldg(pt_row + page0 + pi);
                    if (id < 0 || id >= p.num_pages) { id = 0; atomicOr(p.status, AGX_DEV_BAD_PAGE); }
                }
                ids = (int)id;
            }
            if (t == p.drop_stage) continue;   // test hook: this tile never arrives, its consumers' waits run out
            const int ks = t % kStagesK, kph = (t / kStagesK) & 1;
            const int vs = t % kStagesV, vph = (t / kStagesV) & 1;
            const int npg = pages_in_tile(t);
            const int pg = lane - (t & 3) * 8;              // this lane's page of the tile
            const bool mine = pg >= 0 && pg < npg;
            const int y = (ids * p.hkv + g) * kPage;
            // ---- K
            ok = mbar_wait(bar(BAR_K_EMPTY + ks), kph ^ 1, abort_flag, p.status, p.wait_limit_cycles);
            if (!ok) break;
            if (lane == 0) mbar_arrive_expect_tx(bar(BAR_K_FULL + ks), npg * 4096u);
            __syncwarp();
            last_k = t;
            if (mine) {
                const uint32_t dst = smem_base + kOffK + ks * kTileBytes + pg * 2048;
                tma_load_2d(dst, &map_k, 0, y, bar(BAR_K_FULL + ks));
                tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar(BAR_K_FULL + ks));
            }
            // ---- V (the page that holds token L, if L is not page-aligned, is copied by hand so that
            //      slots past the end of the sequence are zeros whatever the pool holds there)
            if (!waited && !(stable && t < kStagesV)) { pdl_wait(); waited = true; }
            ok = mbar_wait(bar(BAR_V_EMPTY + vs), vph ^ 1, abort_flag, p.status, p.wait_limit_cycles);
            if (!ok) break;
            const int ragged_pg = ((L & 15) != 0 && (L >> 4) >= (tok0 >> 4) && (L >> 4) < (tok0 >> 4) + npg) ? (L >> 4) - (tok0 >> 4) : -1;
            if (ragged_pg >= 0) {
                const int id = __shfl_sync(0xFFFFFFFFu, ids, (t & 3) * 8 + ragged_pg);
                const unsigned char* src = (const unsigned char*)p.v_pool + ((long long)id * p.hkv + g) * (kPage * 256);
                const int valid_rows = L & 15;
                for (int idx = lane; idx < 256; idx += 32) {
                    const int r = idx >> 4, ch = idx & 15, half = ch >> 3, u = ch & 7;
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (r < valid_rows) v = __ldcg((const uint4*)(src + r * 256 + ch * 16));   // (rows a fused append may just have written)
                    *(uint4*)(smem + v_stage_off(vs) + half * kHalfBytes + ragged_pg * 2048 + r * 128 + ((u ^ (r & 7)) << 4)) = v;
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                __syncwarp();
            }
            if (lane == 0) mbar_arrive_expect_tx(bar(BAR_V_FULL + vs), (npg - (ragged_pg >= 0 ? 1 : 0)) * 4096u);
            __syncwarp();
            last_v = t;
            if (mine && pg != ragged_pg) {
                const uint32_t dst = smem_base + v_stage_off(vs) + pg * 2048;
                tma_load_2d(dst, &map_v, 0, y, bar(BAR_V_FULL + vs));
                tma_load_2d(dst + kHalfBytes, &map_v, 64, y, bar(BAR_V_FULL + vs));
            }
        }
        // drain: the copies this warp started must land before the CTA's shared memory goes away.  Bounded by the
        // clock alone: after a time-out elsewhere in the CTA the abort flag is up, and the copies still have to land.
        if (lane == 0) {
            for (int t = max(0, last_k - kStagesK + 1); t <= last_k; ++t)
                if (t != p.drop_stage) mbar_drain(bar(BAR_K_FULL + t % kStagesK), (t / kStagesK) & 1, p.wait_limit_cycles);
            for (int t = max(0, last_v - kStagesV + 1); t <= last_v; ++t)
                if (t != p.drop_stage) mbar_drain(bar(BAR_V_FULL + t % kStagesV), (t / kStagesV) & 1, p.wait_limit_cycles);
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            const uint32_t tS[2] = {tmem_base + kColS, tmem_base + kColS + 128};
            const uint32_t tO[2] = {tmem_base + kColO, tmem_base + kColO + 128};
            // descriptors differ only in the start address: add (byte offset >> 4) to a base descriptor
            const uint64_t q_desc[2] = {make_desc(smem_base + kOffQ, 16, 1024), make_desc(smem_base + kOffQ + kTileBytes, 16, 1024)};
            const uint64_t k_desc0 = make_desc(smem_base + kOffK, 16, 1024);
            auto issue_qk = [&](int qt, int stage, int x) {   // S_x = Q_qt K^T : 8 k-steps of 16 dims
                const uint64_t kd = k_desc0 + (uint64_t)((stage * kTileBytes) >> 4);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t off = (uint64_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
                    umma_ss(tS[x], q_desc[qt] + off, kd + off, kIdescQK, ks > 0);
                }
            };
            // O_x += P_x V, one k-step per page: the head part (pages 0 .. kPvHeadSteps-1) once P_READY says those columns
            // of P are stored, the tail part after P_TAIL
            auto issue_pv = [&](int x, int stage, int npg, bool first, bool tail) {
                const uint64_t vd = make_desc(smem_base + v_stage_off(stage), kHalfBytes, 1024);
                if (npg == 8) {
                    if (!tail) {
#pragma unroll
                        for (int ks = 0; ks < kPvHeadSteps; ++ks)
                            umma_ts(tO[x], tS[x] + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), kIdescPV, !(first && ks == 0));
                    } else {
#pragma unroll
                        for (int ks = kPvHeadSteps; ks < 8; ++ks)
                            umma_ts(tO[x], tS[x] + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), kIdescPV, true);
                    }
                } else {
                    for (int ks = tail ? kPvHeadSteps : 0; ks < (tail ? npg : min(npg, kPvHeadSteps)); ++ks)
                        umma_ts(tO[x], tS[x] + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), kIdescPV, !(first && ks == 0));
                }
            };
            bool ok = mbar_wait(bar(BAR_Q_FULL), 0, abort_flag, p.status, p.wait_limit_cycles);
            if (kStreams) {
                // stream x = t & 1 owns KV tile t:  S_0(0) S_1(1) | O_x += P_x V(t), S_x(t + 2) | ...
                for (int t = 0; t < 2 && t < n_tiles && ok; ++t) {
                    ok = mbar_wait(bar(BAR_K_FULL + t), 0, abort_flag, p.status, p.wait_limit_cycles);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(0, t, t); umma_commit(bar(BAR_S_FULL + t));
                    umma_commit(bar(BAR_K_EMPTY + t));
                }
                for (int t = 0; t < n_tiles && ok; ++t) {
                    const int x = t & 1, vs = t % kStagesV, vph = (t / kStagesV) & 1, npg = pages_in_tile(t);
                    ok = mbar_wait(bar(BAR_V_FULL + vs), vph, abort_flag, p.status, p.wait_limit_cycles);
                    if (!ok) break;
                    ok = mbar_wait(bar(BAR_P_READY + x), (t >> 1) & 1, abort_flag, p.status, p.wait_limit_cycles);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(x, vs, npg, t < 2, false);
                    ok = mbar_wait(bar(BAR_P_TAIL + x), (t >> 1) & 1, abort_flag, p.status, p.wait_limit_cycles);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(x, vs, npg, t < 2, true);
                    umma_commit(bar(BAR_V_EMPTY + vs));
                    if (t + 2 < n_tiles) {
                        const int nks = (t + 2) % kStagesK, nkph = ((t + 2) / kStagesK) & 1;
                        ok = mbar_wait(bar(BAR_K_FULL + nks), nkph, abort_flag, p.status, p.wait_limit_cycles);
                        if (!ok) break;
                        tc_fence_after();
                        issue_qk(0, nks, x); umma_commit(bar(BAR_S_FULL + x));
                        umma_commit(bar(BAR_K_EMPTY + nks));
                    }
                }
            } else {
            if (ok) ok = mbar_wait(bar(BAR_K_FULL + 0), 0, abort_flag, p.status, p.wait_limit_cycles);
            if (ok) {
                tc_fence_after();
                issue_qk(0, 0, 0); umma_commit(bar(BAR_S_FULL + 0));
                issue_qk(1, 0, 1); umma_commit(bar(BAR_S_FULL + 1));
                umma_commit(bar(BAR_K_EMPTY + 0));
            }
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int vs = t % kStagesV, vph = (t / kStagesV) & 1, npg = pages_in_tile(t);
                const bool more = t + 1 < n_tiles;
                const int nks = (t + 1) % kStagesK, nkph = ((t + 1) / kStagesK) & 1;
                ok = mbar_wait(bar(BAR_V_FULL + vs), vph, abort_flag, p.status, p.wait_limit_cycles);
                if (!ok) break;
                ok = mbar_wait(bar(BAR_P_READY + 0), t & 1, abort_flag, p.status, p.wait_limit_cycles);
                if (!ok) break;
                tc_fence_after();
                issue_pv(0, vs, npg, t == 0, false);
                ok = mbar_wait(bar(BAR_P_TAIL + 0), t & 1, abort_flag, p.status, p.wait_limit_cycles);
                if (!ok) break;
                tc_fence_after();
                issue_pv(0, vs, npg, t == 0, true);
                if (more) {
                    ok = mbar_wait(bar(BAR_K_FULL + nks), nkph, abort_flag, p.status, p.wait_limit_cycles);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(0, nks, 0); umma_commit(bar(BAR_S_FULL + 0));
                }
                ok = mbar_wait(bar(BAR_P_READY + 1), t & 1, abort_flag, p.status, p.wait_limit_cycles);
                if (!ok) break;
                tc_fence_after();
                issue_pv(1, vs, npg, t == 0, false);
                ok = mbar_wait(bar(BAR_P_TAIL + 1), t & 1, abort_flag, p.status, p.wait_limit_cycles);
                if (!ok) break;
                tc_fence_after();
                issue_pv(1, vs, npg, t == 0, true);
                umma_commit(bar(BAR_V_EMPTY + vs));
                if (more) {
                    issue_qk(1, nks, 1); umma_commit(bar(BAR_S_FULL + 1));
                    umma_commit(bar(BAR_K_EMPTY + nks));
                }
            }
            }
            umma_commit(bar(BAR_O_FULL));  // arrives when every MMA issued above has completed
            mbar_wait(bar(BAR_O_FULL), 0, abort_flag, p.status, p.wait_limit_cycles);
        }
        __syncwarp();
    } else if (tid == 32 * 3) {   // an otherwise idle warp parks the epilogue's context
        EpiCtx* cx = (EpiCtx*)(smem + kOffCtx);
        cx->it = locate_item<kStreams>(p, blockIdx.x);
        cx->part_base = sp.part_base; cx->hq = p.hq;
        cx->out = p.out; cx->part_o = p.part_o; cx->part_ml = p.part_ml; cx->lse = p.lse;
        cx->magic = p.row_div_magic;
        cx->part_half = p.part_half;
        mbar_arrive(bar(BAR_CTX));   // (release) the epilogue waits on this before it reads the context
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsHigh));
        // ================= softmax + epilogue: one thread per query row =================
        const int x = (warp - 4) >> 2;                       // tile A / B
        const int rt = ((warp & 3) << 5) + lane;             // row in tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t tS = tmem_base + lane_addr + kColS + x * 128;
        const uint32_t tO = tmem_base + lane_addr + kColO + x * 128;
        const int q_tile_row0 = row0 + (kStreams ? 0 : x * 128);   // kStreams: both warpgroups hold the same rows
        const int r = q_tile_row0 + rt;
        const int limit = P + min(r / G, q - 1);             // last token this row sees
        const int tile_i_min = min(q_tile_row0 / G, q - 1);
        // a warp whose 32 rows are all padding only keeps the barriers in step
        const bool warp_has_rows = q_tile_row0 + ((warp & 3) << 5) < rows;
        const float sc = p.scale_log2;
        float m_ref = -INFINITY;
        float l_run = 0.f;                                   // running row sum, relative to m_ref
        bool ok = true;
        constexpr int kStep = kStreams ? 2 : 1;
        const int t_first = kStreams ? x : 0;
        if (!warp_has_rows) {   // keep S_FULL / P_READY in step, nothing else
            for (int t = t_first; t < n_tiles && ok; t += kStep) {
                ok = mbar_wait(bar(BAR_S_FULL + x), ((t - t_first) / kStep) & 1, abort_flag, p.status, p.wait_limit_cycles);
                if (ok) { mbar_arrive(bar(BAR_P_READY + x)); mbar_arrive(bar(BAR_P_TAIL + x)); }
            }
        } else
        for (int t = t_first; t < n_tiles; t += kStep) {
            const int j = (t - t_first) / kStep;             // this warpgroup's j-th tile
            ok = mbar_wait(bar(BAR_S_FULL + x), j & 1, abort_flag, p.status, p.wait_limit_cycles);
            if (!ok) break;
            tc_fence_after();
            uint32_t sreg[128];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) tmem_ld_x32(tS + c4 * 32, sreg + c4 * 32);
            tmem_wait_ld();
            const int tok0 = kv_begin + t * kBN;
            const bool masked = (tok0 + kBN - 1 > P + tile_i_min) || (tok0 + kBN > kv_end);  // uniform per tile
            float lt0 = 0.f, lt1 = 0.f, lt2 = 0.f, lt3 = 0.f;   // this tile's row sum, four partial sums
            if (masked) {
                const int nvis = max(0, min(min(limit + 1, kv_end) - tok0, kBN));        // visible columns: [0, nvis)
#pragma unroll
                for (int c = 0; c < 128; ++c)
                    if (c >= nvis) sreg[c] = 0xFF800000u;  // -inf: its exponential is exactly 0
            }
            // ---- row maximum (four independent chains of 3-input max).  The exponentials below are taken against the
            //      running reference m_ref (the maximum of earlier tiles, so P may exceed 1); only if this tile's
            //      maximum tops it by more than 2^8 is the reference moved and O rescaled.
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 128; c += 8) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    mx[k] = max3(mx[k], __uint_as_float(sreg[c + 2 * k]), __uint_as_float(sreg[c + 2 * k + 1]));
            }
            const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * sc;
            const bool need = m_tile > m_ref + kRescaleThreshold;
            if (__any_sync(0xFFFFFFFFu, need)) {
                const float m_new = need ? m_tile : m_ref;
                const float factor = need ? ex2(m_ref - m_new) : 1.f;   // m_ref = -inf gives 0
                if (j > 0) {
                    uint32_t oreg[32];
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4) {
                        tmem_ld_x32(tO + c4 * 32, oreg);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) oreg[c] = __float_as_uint(__uint_as_float(oreg[c]) * factor);
                        tmem_st_x32(tO + c4 * 32, oreg);
                    }
                    tmem_wait_st();
                }
                l_run *= factor;
                m_ref = m_new;
            }
            // ---- P = 2^(S * scale - m_ref) as packed bf16 pairs, in place: sreg[c / 2] <- (p[c], p[c + 1]); the
            //      first kPvHeadSteps * 16 columns are stored and handed over before the rest is computed
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            const uint64_t sc2 = pk2(sc, sc), nm2 = pk2(neg_m, neg_m);
            auto sweep = [&](const int c_lo, const int c_hi) {
#pragma unroll
                for (int c = c_lo; c < c_hi; c += 4) {
                    const uint64_t xa = fma2p(pk2(__uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1])), sc2, nm2);
                    const uint64_t xb = fma2p(pk2(__uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3])), sc2, nm2);
                    float a0, a1, b0, b1;
                    if (((c >> 1) & 7) < kPolyPairsOf8) ex2_poly2(xa, a0, a1);
                    else { upk2(xa, a0, a1); a0 = ex2(a0); a1 = ex2(a1); }
                    if ((((c >> 1) + 1) & 7) < kPolyPairsOf8) ex2_poly2(xb, b0, b1);
                    else { upk2(xb, b0, b1); b0 = ex2(b0); b1 = ex2(b1); }
                    add2(lt0, lt1, a0, a1);
                    add2(lt2, lt3, b0, b1);
                    sreg[c >> 1] = pack_bf16(a0, a1);
                    sreg[(c >> 1) + 1] = pack_bf16(b0, b1);
                }
            };
            constexpr int kHeadCols = kPvHeadSteps * 16;   // 96 score columns = 48 packed registers
            sweep(0, kHeadCols);
            tmem_st_x32(tS, sreg);
            tmem_st_x16(tS + 32, sreg + 32);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(BAR_P_READY + x));
            sweep(kHeadCols, 128);
            l_run += (lt0 + lt1) + (lt2 + lt3);
            tmem_st_x16(tS + 48, sreg + 48);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(BAR_P_TAIL + x));
        }
        if (ok) ok = mbar_wait(bar(BAR_O_FULL), 0, abort_flag, p.status, p.wait_limit_cycles);
        if (ok || kStreams) tile_epilogue<kStreams>(smem, tO, m_ref, l_run, ok);
    }
    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// --------------------------------------------------------------------------------------------
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}
// 2-D view of a pool: [num_pages * Hkv * 16 rows][128 dims] bf16; box = 16 rows x 64 dims, 128-byte swizzle
bool make_pool_map_impl(CUtensorMap* map, const void* pool, long long num_pages, int hkv) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)num_pages * hkv * kPage};
    const cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kPage};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(pool), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace

bool make_pool_map(CUtensorMap* map, const void* pool, long long num_pages, int hkv) {
    return make_pool_map_impl(map, pool, num_pages, hkv);
}

namespace {
template <bool kStreams>
cudaError_t launch_tile(const AttnParams& p, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
    // the attribute is per device: remember which devices have it (a process normally drives one GPU)
    static bool configured_on[64] = {false};
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return cudaErrorInvalidDevice;
    bool& configured = configured_on[device];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(attn_tile_bf16_kernel<kStreams>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_chained(attn_tile_bf16_kernel<kStreams>, dim3(p.num_items), dim3(kThreads), kSmemBytes, stream, p, map_k, map_v);
}
}  // namespace

cudaError_t launch_attn_tile_bf16(const AttnParams& p, bool streams, const CUtensorMap& map_k, const CUtensorMap& map_v,
                                  cudaStream_t stream) {
    if (p.num_items == 0) return cudaSuccess;
    return streams ? launch_tile<true>(p, map_k, map_v, stream) : launch_tile<false>(p, map_k, map_v, stream);
}

}  // namespace agx

