// PTX wrappers shared by the sm_100a kernels: mbarrier (with bounded waits), TMA tile loads, fast exp2.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "agx.h"
#include "agx_internal.cuh"

namespace agx {

namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) when the limit is hit or another
// role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long limit_cycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                *abort_flag = 1;
                if (status) atomicOr(status, AGX_DEV_WAIT_TIMEOUT);
                return false;
            }
        }
    }
}

// Wait of the copy-issuing lane for copies it has armed itself, when the CTA winds down: bounded by the clock only.
// The abort flag is ignored on purpose, since the shared memory the copies land in must stay allocated until they have.
__device__ __forceinline__ bool mbar_drain(uint32_t bar, uint32_t parity, long long limit_cycles) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit_cycles) return false;
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Programmatic dependent launch: a kernel lets the next launch in the stream start early (its CTAs then run
// their set-up and block in pdl_wait), and itself waits, before it touches global memory, until the launch
// before it has completed and its writes are visible.  Both are no-ops for launches without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

// Fused KV append (bf16, d = 128): the CTA that will read tokens [t_lo, t_hi) of KV head g writes the block's own
// rows in that range into the sequence's pages first (Sec. 2.3: the block's KV joins the cache before it is attended
// to), then makes them visible to the TMA copies that follow: a generic-proxy fence here, a CTA barrier at the caller.
__device__ __forceinline__ void append_rows_bf16(const AttnParams& p, const SeqPlan& sp, int g, int t_lo, int t_hi, int tid,
                                                 int nthreads) {
    const int lo = max(t_lo, sp.prefix_len), hi = min(t_hi, sp.prefix_len + sp.q_len);
    if (hi > lo) {
        const int* pt_row = p.page_table + (long long)sp.seq_index * p.pt_stride;
        for (int idx = tid; idx < (hi - lo) * 32; idx += nthreads) {
            const int tok = lo + (idx >> 5), is_v = (idx >> 4) & 1, c = idx & 15;
            const long long page = (tok >> 4) < p.pt_stride ? __ldg(pt_row + (tok >> 4)) : -1;
            if (page < 0 || page >= p.num_pages) { if (c == 0) atomicOr(p.status, AGX_DEV_BAD_PAGE); continue; }
            const unsigned char* src = (const unsigned char*)(is_v ? p.v_new : p.k_new) +
                                       (((long long)(sp.q_row0 + tok - sp.prefix_len) * p.hkv + g) * 256 + c * 16);
            unsigned char* dst = (unsigned char*)(is_v ? p.v_pool : p.k_pool) + (((page * p.hkv + g) * kPage + (tok & 15)) * 256 + c * 16);
            *(uint4*)dst = __ldg((const uint4*)src);
        }
        __threadfence();
        asm volatile("fence.proxy.async;\n" ::: "memory");
    }
}

// ---- thread-block clusters: barrier over all threads of all CTAs, and loads from a peer CTA's shared memory
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_map(uint32_t smem_addr, uint32_t cta_rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];\n" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace
}  // namespace agx
