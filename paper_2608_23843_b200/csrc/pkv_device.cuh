// Device-side helpers shared by the decode kernels (the pipeline kernel and the row-block kernels): unit
// numbering of a (sequence, KV head) run, mbarrier and bulk-copy wrappers, bf16 packing.  Everything here has
// internal linkage: each translation unit that includes the file gets its own copy.
#pragma once

#include <cuda_bf16.h>

#include "pkv_internal.h"

namespace pkv {

namespace {

constexpr float kNegInf = -1e30f;      // finite stand-in for -inf: exp2(kNegInf - x) == 0, no NaN from inf - inf
constexpr float kMasked = -2e30f;      // score of a token a query must not see: exp2(kMasked - m) == 0 even while m == kNegInf
constexpr int kKindDense = 0, kKindFactor = 1, kKindEnd = 2;
// Global SVD form: a region's shared basis travels through the ring like a page, once per consumer warp
constexpr int kKindBasisK = 3, kKindBasisV = 4;

struct HeadUnits { int d0, nf, units, fb, fe; };

__device__ __forceinline__ HeadUnits head_units(const Geometry &g, const PlanEntry &e) {
    HeadUnits h;
    h.fb = min(e.f_begin, e.n_pages);
    h.fe = min(max(e.f_end, h.fb), e.n_pages);
    h.d0 = h.fb * g.blocks_per_page;
    h.nf = h.fe - h.fb;
    h.units = h.d0 + h.nf + (e.n_pages - h.fe) * g.blocks_per_page;
    return h;
}

// unit index within an (entry, head) run -> logical page, block inside the page, kind
// (bpp: blocks a dense page is cut into)
__device__ __forceinline__ void unit_to_page(int bpp, const HeadUnits &h, int u, int &page, int &blk, int &kind) {
    if (u < h.d0) { page = u / bpp; blk = u % bpp; kind = kKindDense; }
    else if (u < h.d0 + h.nf) { page = h.fb + (u - h.d0); blk = 0; kind = kKindFactor; }
    else { int v = u - h.d0 - h.nf; page = h.fe + v / bpp; blk = v % bpp; kind = kKindDense; }
}
__device__ __forceinline__ void unit_to_page(const Geometry &g, const HeadUnits &h, int u, int &page, int &blk,
                                             int &kind) {
    unit_to_page(g.blocks_per_page, h, u, page, blk, kind);
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` clocks (kWaitClocks, about a second, unless a test shortened it) and reports
// failure.
constexpr long long kWaitClocks = 2000000000LL;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit = kWaitClocks) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}
// Pages are read once per launch: ask L2 to drop them first, so that the plan, the queries and the split-K partial
// states stay resident.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    unsigned long long policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
// The row-block kernel reads a sequence's pages once per block of 64 query rows: there the copies leave the
// lines in L2 for the other blocks.
__device__ __forceinline__ void bulk_g2s_keep(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// two floats -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16lo_f(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16hi_f(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

struct StageDesc { int kind, rows, seg, after; };

// Shapes fixed at compile time: P tokens per page, NT = ceil(rank / 8) rank tiles (K and V alike), I4 = factors
// stored as INT4 codes.
// rows per dense block: 32 where a stage has to be that large for a bf16 factor page anyway
// F = storage form of the factors: 0 = bf16 page-wise (Eq. 2), 1 = INT4 page-wise (Section 4.3), 2 = Global SVD form
// (Section 4.2: pages hold A rows only, the basis is shared by the region)
template <int P, int NT, int F>
constexpr int kDenseBlock = (F != 1 && P >= 32 && NT >= 3) ? 32 : 16;

}  // namespace

}  // namespace pkv
