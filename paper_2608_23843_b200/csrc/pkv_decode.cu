// Decode attention over mixed dense / factor pages (paper: Eq. 4, Eq. 5).
//
// One launch covers one layer.  The (sequence, KV head, page) list is cut by the
// host into byte-balanced contiguous ranges, one per persistent CTA.  Inside a
// CTA a producer warp walks the page table and streams whole factor blobs / dense
// row blocks into a shared-memory ring with bulk async copies (TMA, mbarrier
// completion); five consumer warps each take one unit at a time and evaluate
//     q~ = B_k q          (tensor cores, bf16 x bf16 -> fp32)
//     s  = A_k q~ * scale (q~ split into two bf16 terms so the exponent sees ~fp32)
//     online softmax      (fp32, exp2 with the scale folded in)
//     w  = A_v^T p,  o += B_v^T w
// for all query heads that share the KV head, keeping (m, l, o) in registers.
// K^ and V^ are never formed.  At the end of each (sequence, KV head) segment the
// warps combine their states; a segment split over several CTAs leaves one
// partial state per CTA and the CTA that finishes last applies Eq. 5 across them
// (ticket counter, no waiting).  A scalar fp32 kernel with the same plan and
// partial format, followed by a separate merge kernel, exists as a debugging
// reference (decode_variant = 1).
#include <cuda_bf16.h>

#include "pkv_device.cuh"
#include "pkv_internal.h"

// Scratch of pkv_decode_attention_static_scratch(): split-K partial states followed by the merge
// tickets.  It lives in the library image, so every GPU that loads the library holds these bytes
// (about 4.1 MiB) until the process exits, and every call on a device shares them.
static constexpr int kStaticPartialStates = 1024;
static constexpr int kStaticTickets = 1024;
static constexpr size_t kStaticTicketOffset = (size_t)kStaticPartialStates * pkv::kPartialFloats * sizeof(float);
static constexpr size_t kStaticScratchBytes = kStaticTicketOffset + kStaticTickets * sizeof(int);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace pkv {

namespace {

struct Range {
    PlanCta start, end;
    PlanEntry first_entry;             // the entry `start` lies in
    int n_used, seg_first, n_local_segs;
};

__device__ __forceinline__ bool load_range(const DecodeArgs &a, Range &r) {
    // All four loads are issued together (the arrays have an element for every CTA of the grid, used or not), so
    // that the header's latency is not paid a second time before the CTA knows its range.
    // With several query blocks per sequence the CTAs come in groups of q_group that share a range: CTA b walks
    // range b / q_group for the (b % q_group)-th query block of the range's plan entry.  The siblings start
    // together and read the same pages in the same order, so all but the first find them in L2.
    const int range = blockIdx.x / a.q_group;
    const PlanCta *ctas = reinterpret_cast<const PlanCta *>(a.plan + a.plan_cta);
    const PlanHeader hdr = *reinterpret_cast<const PlanHeader *>(a.plan);
    r.start = ctas[range];
    r.end = ctas[range + 1];
    r.first_entry = reinterpret_cast<const PlanEntry *>(a.plan + a.plan_cta_entry)[range];
    r.n_used = hdr.n_used_ctas;
    if (range >= hdr.n_used_ctas) return false;
    const int H = a.geo.n_kv_heads;
    r.seg_first = r.start.entry * H + r.start.head;
    int seg_last = r.end.entry * H + r.end.head;
    if (r.end.unit == 0) seg_last -= 1;
    r.n_local_segs = seg_last - r.seg_first + 1;
    return true;
}

// =============================================================================
// Scalar reference kernel (debugging aid): same plan, same partial format.
// =============================================================================
__device__ __forceinline__ float bf16_at(const unsigned char *base, int byte_off) {
    return __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(base + byte_off));
}
__device__ __forceinline__ int swz_off(int row, int col) {     // byte offset of element (row, col) of a 256-byte-row matrix
    return row * kRowBytes + swz_chunk(row, col >> 3) * 16 + (col & 7) * 2;
}

__global__ void __launch_bounds__(128) decode_scalar_kernel(const __grid_constant__ DecodeArgs a) {
    Range rg;
    if (!load_range(a, rg)) return;
    const Geometry &g = a.geo;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = g.group, H = g.n_kv_heads, r_k = g.rank_k, r_v = g.rank_v, P = g.page;
    __shared__ float qs[kMaxGroup][kHeadDim];
    __shared__ float qt[kMaxGroup][32];
    __shared__ float sc[kMaxGroup][kMaxPage];
    __shared__ float wv[kMaxGroup][32];
    __shared__ float m_s[kMaxGroup], l_s[kMaxGroup], alpha_s[kMaxGroup];
    float o[kMaxGroup];
    const PlanEntry *entries = reinterpret_cast<const PlanEntry *>(a.plan + a.plan_entry);

    PlanCta cur = rg.start;
    while (!(cur.entry == rg.end.entry && cur.head == rg.end.head && cur.unit == rg.end.unit)) {
        const PlanEntry e = entries[cur.entry];
        const HeadUnits hu = head_units(g, e);
        const bool last_run = cur.entry == rg.end.entry && cur.head == rg.end.head;
        const int u_end = last_run ? rg.end.unit : hu.units;
        const int T = a.n_tokens[(long long)e.seq * g.n_layers + a.layer];
        // new segment: load q, reset state
        __syncthreads();
        for (int i = tid; i < G * kHeadDim; i += 128)
            qs[i / kHeadDim][i % kHeadDim] = __bfloat162float(
                reinterpret_cast<const __nv_bfloat16 *>(a.q)[((long long)cur.entry * g.n_q_heads + cur.head * G) * kHeadDim + i]);
        if (tid < kMaxGroup) { m_s[tid] = kNegInf; l_s[tid] = 0.f; }
        for (int gq = 0; gq < kMaxGroup; ++gq) o[gq] = 0.f;
        __syncthreads();
        for (int u = cur.unit; u < u_end; ++u) {
            int page, blk, kind;
            unit_to_page(g, hu, u, page, blk, kind);
            const int slot = a.page_table[((long long)e.seq * g.n_layers + a.layer) * g.max_pages + page];
            int rows;
            const unsigned char *base;
            if (kind == kKindFactor) {
                rows = P;
                base = a.factor_pool + (long long)slot * g.factor_slot_bytes + (long long)cur.head * g.blob_bytes;
                for (int i = tid; i < G * r_k; i += 128) {           // q~ = B_k q
                    const int gq = i / r_k, j = i % r_k;
                    float acc = 0.f;
                    for (int c = 0; c < kHeadDim; ++c) acc += blob_value(g, base, 1, j, c) * qs[gq][c];
                    qt[gq][j] = acc;
                }
                __syncthreads();
                for (int i = tid; i < G * P; i += 128) {             // s = A_k q~ * scale
                    const int gq = i / P, p = i % P;
                    float acc = 0.f;
                    for (int j = 0; j < r_k; ++j) acc += blob_value(g, base, 0, j, p) * qt[gq][j];
                    sc[gq][p] = acc * g.scale_log2e;
                }
            } else {
                const int row0 = blk * g.block_tokens;
                rows = min(g.block_tokens, T - page * P - row0);
                if (rows <= 0) continue;
                base = a.dense_pool + (long long)slot * g.dense_slot_bytes + (long long)cur.head * g.dense_head_bytes;
                for (int i = tid; i < G * rows; i += 128) {
                    const int gq = i / rows, p = i % rows;
                    float acc = 0.f;
                    for (int c = 0; c < kHeadDim; ++c) acc += bf16_at(base, swz_off(row0 + p, c)) * qs[gq][c];
                    sc[gq][p] = acc * g.scale_log2e;
                }
            }
            __syncthreads();
            for (int gq = warp; gq < G; gq += 4) {                   // online softmax, one warp per head
                float mx = kNegInf;
                for (int p = lane; p < rows; p += 32) mx = fmaxf(mx, sc[gq][p]);
                for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
                const float m_new = fmaxf(m_s[gq], mx);
                float sum = 0.f;
                for (int p = lane; p < rows; p += 32) { float e2 = exp2f(sc[gq][p] - m_new); sc[gq][p] = e2; sum += e2; }
                for (int off = 16; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                if (lane == 0) {
                    const float al = exp2f(m_s[gq] - m_new);
                    alpha_s[gq] = al;
                    l_s[gq] = l_s[gq] * al + sum;
                    m_s[gq] = m_new;
                }
            }
            __syncthreads();
            if (kind == kKindFactor) {
                for (int i = tid; i < G * r_v; i += 128) {           // w = A_v^T p
                    const int gq = i / r_v, j = i % r_v;
                    float acc = 0.f;
                    for (int p = 0; p < P; ++p) acc += sc[gq][p] * blob_value(g, base, 2, j, p);
                    wv[gq][j] = acc;
                }
                __syncthreads();
                for (int gq = 0; gq < G; ++gq) {                     // o = o*alpha + B_v^T w
                    float acc = 0.f;
                    for (int j = 0; j < r_v; ++j) acc += wv[gq][j] * blob_value(g, base, 3, j, tid);
                    o[gq] = o[gq] * alpha_s[gq] + acc;
                }
            } else {
                const int row0 = blk * g.block_tokens;
                for (int gq = 0; gq < G; ++gq) {
                    float acc = 0.f;
                    for (int p = 0; p < rows; ++p)
                        acc += sc[gq][p] * bf16_at(base + P * kRowBytes, swz_off(row0 + p, tid));
                    o[gq] = o[gq] * alpha_s[gq] + acc;
                }
            }
            __syncthreads();
        }
        // segment (or range) done: write the partial state
        const int seg = cur.entry * H + cur.head;
        float *part = a.partials + ((long long)blockIdx.x + seg) * kPartialFloats;
        for (int gq = 0; gq < kMaxGroup; ++gq) part[gq * kHeadDim + tid] = gq < G ? o[gq] : 0.f;
        if (tid < kMaxGroup) {
            part[kMaxGroup * kHeadDim + tid] = tid < G ? m_s[tid] : kNegInf;
            part[kMaxGroup * kHeadDim + kMaxGroup + tid] = tid < G ? l_s[tid] : 0.f;
        }
        if (last_run) break;
        cur.unit = 0;
        if (++cur.head == H) { cur.head = 0; ++cur.entry; }
    }
}

// =============================================================================
// Eq. 5 across CTAs: one block per (entry, KV head) segment.
// =============================================================================
__global__ void __launch_bounds__(256) merge_kernel(const __grid_constant__ DecodeArgs a) {
    const Geometry &g = a.geo;
    const int seg = blockIdx.x;
    const PlanSeg ps = reinterpret_cast<const PlanSeg *>(a.plan + a.plan_seg)[seg];
    const int entry = seg / g.n_kv_heads, head = seg % g.n_kv_heads;
    const int hq = threadIdx.x >> 5, d4 = (threadIdx.x & 31) * 4;
    if (hq >= g.group) return;
    const float *part = a.partials + ((long long)ps.cta_first + seg) * kPartialFloats;
    float M = kNegInf;
    for (int k = 0; k < ps.n_parts; ++k) M = fmaxf(M, part[(long long)k * kPartialFloats + kMaxGroup * kHeadDim + hq]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    for (int k = 0; k < ps.n_parts; ++k) {
        const float *pk = part + (long long)k * kPartialFloats;
        const float w = exp2f(pk[kMaxGroup * kHeadDim + hq] - M);
        const float4 o = *reinterpret_cast<const float4 *>(pk + hq * kHeadDim + d4);
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        L += w * pk[kMaxGroup * kHeadDim + kMaxGroup + hq];
    }
    const float inv = 1.f / L;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    const long long off = ((long long)entry * g.n_q_heads + head * g.group + hq) * kHeadDim + d4;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 packed;
    packed.x = *reinterpret_cast<unsigned *>(&lo);
    packed.y = *reinterpret_cast<unsigned *>(&hi);
    *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + off) = packed;
    if (a.out_f32) *reinterpret_cast<float4 *>(a.out_f32 + off) = acc;
}

// =============================================================================
// Tensor-core pipeline kernel.
// =============================================================================
__device__ __forceinline__ int ld_acquire_smem(const volatile int *p) {
    int v;
    asm volatile("ld.acquire.cta.shared.b32 %0, [%1];" : "=r"(v) : "r"(smem_u32(const_cast<const int *>(p))) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_smem(volatile int *p, int v) {
    asm volatile("st.release.cta.shared.b32 [%0], %1;" ::"r"(smem_u32(const_cast<int *>(p))), "r"(v) : "memory");
}
// Bounded spin until the producer has armed unit k in its stage (the stage's tag then reads k + 1).
__device__ __forceinline__ bool wait_armed(volatile int *tag, int k, long long limit) {
    if (ld_acquire_smem(tag) == k + 1) return true;
    const long long t0 = clock64();
    while (ld_acquire_smem(tag) != k + 1) {
        if (clock64() - t0 > limit) return false;
        __nanosleep(20);
    }
    return true;
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t (&r)[2], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t (&r)[2], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma1688(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ uint32_t movm_t(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
// Per-warp running state for the query heads 2t, 2t+1 (t = lane & 3) of one KV head.
struct WarpState {
    float o[8][4];        // o[i]: (d = 16i+g, heads 2t,2t+1), (d = 16i+8+g, heads 2t,2t+1);  g = lane >> 2
    float m[2], l[2];     // l is this lane's share; summed over g at flush time
};

template <int P, int NT>
struct Tc {
    static constexpr int kMT = P / 16;                                  // 16-token tiles per page
    static constexpr int kPitchA = 2 * P;                               // bytes per A^T row
};

// chunk swizzle of an A^T row as a function of the row's low bits (see swz_a_chunk)
template <int P>
__device__ __forceinline__ int a_swz(int l7) { return P == 64 ? l7 : (P == 32 ? (l7 >> 1) : (l7 >> 2)); }

template <int NI>         // softmax over NI score tiles of 16 tokens; leaves p in place and its bf16, transposed copies
__device__ __forceinline__ void online_softmax(float (&s)[4][4], WarpState &st, uint32_t (&T0)[4], uint32_t (&T1)[4],
                                               float &al0_out, float &al1_out) {
    float mx0 = kNegInf, mx1 = kNegInf;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        mx0 = fmaxf(mx0, fmaxf(s[i][0], s[i][2]));
        mx1 = fmaxf(mx1, fmaxf(s[i][1], s[i][3]));
    }
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
    }
    const float mn0 = fmaxf(st.m[0], mx0), mn1 = fmaxf(st.m[1], mx1);
    const float al0 = exp2f(st.m[0] - mn0), al1 = exp2f(st.m[1] - mn1);
    al0_out = al0; al1_out = al1;                       // (for accumulators the caller keeps besides st.o)
    st.m[0] = mn0; st.m[1] = mn1;
    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        s[i][0] = exp2f(s[i][0] - mn0); s[i][2] = exp2f(s[i][2] - mn0);
        s[i][1] = exp2f(s[i][1] - mn1); s[i][3] = exp2f(s[i][3] - mn1);
        sum0 += s[i][0] + s[i][2];
        sum1 += s[i][1] + s[i][3];
    }
    st.l[0] = st.l[0] * al0 + sum0;
    st.l[1] = st.l[1] * al1 + sum1;
    if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { st.o[i][0] *= al0; st.o[i][1] *= al1; st.o[i][2] *= al0; st.o[i][3] *= al1; }
    }
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        T0[i] = movm_t(pack_bf16(s[i][0], s[i][1]));   // (head g; tokens 16i+2t, +1)
        T1[i] = movm_t(pack_bf16(s[i][2], s[i][3]));   // (head g; tokens 16i+8+2t, +1)
    }
}

template <int NI>
__device__ __forceinline__ void online_softmax(float (&s)[4][4], WarpState &st, uint32_t (&T0)[4], uint32_t (&T1)[4]) {
    float a0, a1;
    online_softmax<NI>(s, st, T0, T1, a0, a1);
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
// one bf16 from shared memory, copied into both halves of a register
__device__ __forceinline__ uint32_t lds16x2(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v * 0x10001u;
}

// One factor page.  sb = shared address of the blob; ak/bk/av/bv = byte offsets of its four matrices;
// rk, rv = true ranks (tile rows past them hold other finite data and are multiplied by exact zeros).
template <int P, int NT>
__device__ __forceinline__ void factor_unit(uint32_t sb, int ak, int bk, int av, int bv, int rk, int rv,
                                            const uint32_t (&qf)[8][2], float scale, WarpState &st, int lane) {
    using C = Tc<P, NT>;
    const int l7 = lane & 7, mi = lane >> 3, t2 = (lane & 3) * 2;
    const int asw = a_swz<P>(l7);
    // ---- q~^T [G][r] = q [G][d] . B_k^T ----
    // (the loops run over the independent accumulators innermost, so that consecutive mma do not wait for
    // one another)
    uint32_t qhi[NT], qlo[NT];
    {
        float qt[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) qt[j][0] = qt[j][1] = qt[j][2] = qt[j][3] = 0.f;
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
            uint32_t b[NT][4];
#pragma unroll
            for (int j = 0; j < NT; ++j) ldsm_x4(b[j], sb + bk + (8 * j + l7) * kRowBytes + (((4 * qd + mi) ^ l7) << 4));
#pragma unroll
            for (int j = 0; j < NT; ++j) mma16816(qt[j], qf[2 * qd][0], 0u, qf[2 * qd][1], 0u, b[j][0], b[j][1]);
#pragma unroll
            for (int j = 0; j < NT; ++j) mma16816(qt[j], qf[2 * qd + 1][0], 0u, qf[2 * qd + 1][1], 0u, b[j][2], b[j][3]);
        }
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const float x0 = (8 * j + t2 < rk) ? qt[j][0] * scale : 0.f;
            const float x1 = (8 * j + t2 + 1 < rk) ? qt[j][1] * scale : 0.f;
            qhi[j] = pack_bf16(x0, x1);
            qlo[j] = pack_bf16(x0 - bf16lo_f(qhi[j]), x1 - bf16hi_f(qhi[j]));
        }
    }
    // ---- s [P][G] = A_k [P][r] . q~   (A_k^T in shared memory: transposed tile loads) ----
    float s[4][4];
#pragma unroll
    for (int i = 0; i < C::kMT; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < NT / 2; ++kk) {
        uint32_t a4[C::kMT][4];
#pragma unroll
        for (int i = 0; i < C::kMT; ++i)
            ldsm_x4_t(a4[i], sb + ak + (16 * kk + (mi >> 1) * 8 + l7) * C::kPitchA + (((2 * i + (mi & 1)) ^ asw) << 4));
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) mma16816(s[i], a4[i][0], a4[i][1], a4[i][2], a4[i][3], qhi[2 * kk], qhi[2 * kk + 1]);
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) mma16816(s[i], a4[i][0], a4[i][1], a4[i][2], a4[i][3], qlo[2 * kk], qlo[2 * kk + 1]);
    }
    if (NT % 2) {
        uint32_t a2[C::kMT][2];
#pragma unroll
        for (int i = 0; i < C::kMT; ++i)
            ldsm_x2_t(a2[i], sb + ak + (8 * (NT - 1) + l7) * C::kPitchA + (((2 * i + (mi & 1)) ^ asw) << 4));
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) mma1688(s[i], a2[i][0], a2[i][1], qhi[NT - 1]);
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) mma1688(s[i], a2[i][0], a2[i][1], qlo[NT - 1]);
    }
    uint32_t T0[4], T1[4];
    online_softmax<C::kMT>(s, st, T0, T1);
    // ---- w^T [G][r] = p^T [G][P] . A_v [P][r] ----
    uint32_t wh[NT];
    {
        float wt[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) wt[j][0] = wt[j][1] = wt[j][2] = wt[j][3] = 0.f;
#pragma unroll
        for (int qd = 0; qd < C::kMT / 2; ++qd) {
            uint32_t b[NT][4];
#pragma unroll
            for (int j = 0; j < NT; ++j) ldsm_x4(b[j], sb + av + (8 * j + l7) * C::kPitchA + (((4 * qd + mi) ^ asw) << 4));
#pragma unroll
            for (int j = 0; j < NT; ++j) mma16816(wt[j], T0[2 * qd], 0u, T1[2 * qd], 0u, b[j][0], b[j][1]);
#pragma unroll
            for (int j = 0; j < NT; ++j) mma16816(wt[j], T0[2 * qd + 1], 0u, T1[2 * qd + 1], 0u, b[j][2], b[j][3]);
        }
        if (C::kMT % 2) {
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                uint32_t b[2];
                ldsm_x2(b, sb + av + (8 * j + l7) * C::kPitchA + (((2 * (C::kMT - 1) + (mi & 1)) ^ asw) << 4));
                mma16816(wt[j], T0[C::kMT - 1], 0u, T1[C::kMT - 1], 0u, b[0], b[1]);
            }
        }
#pragma unroll
        for (int j = 0; j < NT; ++j)
            wh[j] = pack_bf16((8 * j + t2 < rv) ? wt[j][0] : 0.f, (8 * j + t2 + 1 < rv) ? wt[j][1] : 0.f);
    }
    // ---- o [d][G] += B_v^T [d][r] . w ----
#pragma unroll
    for (int kk = 0; kk < NT / 2; ++kk) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t a4[4];
            ldsm_x4_t(a4, sb + bv + (16 * kk + (mi >> 1) * 8 + l7) * kRowBytes + (((2 * i + (mi & 1)) ^ l7) << 4));
            mma16816(st.o[i], a4[0], a4[1], a4[2], a4[3], wh[2 * kk], wh[2 * kk + 1]);
        }
    }
    if (NT % 2) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t a2[2];
            ldsm_x2_t(a2, sb + bv + (8 * (NT - 1) + l7) * kRowBytes + (((2 * i + (mi & 1)) ^ l7) << 4));
            mma1688(st.o[i], a2[0], a2[1], wh[NT - 1]);
        }
    }
}

// Register n (a compile-time constant after unrolling) of this lane out of its code words: the two codes as
// bf16(code * scale).  (word >> 4t) & 0x000F000F | 0x43004300 is the bf16 pair (128 + u_lo, 128 + u_hi) with
// u = code + 8; subtracting 136 is exact and the product with the scale pair rounds once.
__device__ __forceinline__ uint32_t int4_pair(uint32_t word, int t, uint32_t scale2) {
    const uint32_t x = ((word >> (4 * t)) & 0x000F000Fu) | 0x43004300u;
    uint32_t c, v;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(c) : "r"(x), "r"(0x43084308u));
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(v) : "r"(c), "r"(scale2));
    return v;
}
#define PKV_I4(words, n, scale2) int4_pair((words)[(n) >> 2], (n) & 3, (scale2))

// One factor page stored as INT4 codes in operand-register order (see int4_a_pos / int4_b_pos): the same four
// products as factor_unit, with every operand register made from its codes and scales in registers.  Ranks
// past the true ones are stored as zero codes, so nothing needs masking.
template <int P, int NT>
__device__ __forceinline__ void factor_unit_int4(uint32_t sb, const Geometry &g, const uint32_t (&qf)[8][2],
                                                 WarpState &st, int lane) {
    using C = Tc<P, NT>;
    constexpr int kMT = C::kMT;
    constexpr int kWA = (kMT * 2 * NT + 3) / 4;        // words per lane: A~_K
    constexpr int kWV = (NT * (P / 8) + 3) / 4;        //                 A~_V
    constexpr int kWR = (8 * 2 * NT + 3) / 4;          //                 B~_V
    const int gq = lane >> 2, c2 = (lane & 3) * 2;
    const uint32_t sc = sb + g.codes_bytes, lane4 = lane * 4;
    // ---- q~^T [G][r] = q [G][d] . B~_K^T   (scales per channel: pairs d = 16 kk + 8 b + 2c, +1) ----
    uint32_t qhi[NT], qlo[NT];
    {
        uint32_t sk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) sk[i] = lds32(sc + g.sbk_off + 2 * (8 * i + c2));
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            float qt[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int wq = 0; wq < 4; ++wq) {
                const uint32_t w = lds32(sb + g.cbk_off + (j * 4 + wq) * 128 + lane4);
                mma16816(qt, qf[2 * wq][0], 0u, qf[2 * wq][1], 0u, int4_pair(w, 0, sk[4 * wq]), int4_pair(w, 1, sk[4 * wq + 1]));
                mma16816(qt, qf[2 * wq + 1][0], 0u, qf[2 * wq + 1][1], 0u, int4_pair(w, 2, sk[4 * wq + 2]),
                         int4_pair(w, 3, sk[4 * wq + 3]));
            }
            const float x0 = qt[0] * g.scale_log2e, x1 = qt[1] * g.scale_log2e;
            qhi[j] = pack_bf16(x0, x1);
            qlo[j] = pack_bf16(x0 - bf16lo_f(qhi[j]), x1 - bf16hi_f(qhi[j]));
        }
    }
    // ---- s [P][G] = A~_K [P][r] . q~   (scales per rank: pairs 8 jt + 2c, +1) ----
    float s[4][4];
    {
        uint32_t sa[NT], wa[kWA];
#pragma unroll
        for (int jt = 0; jt < NT; ++jt) sa[jt] = lds32(sc + g.sak_off + 2 * (8 * jt + c2));
#pragma unroll
        for (int w = 0; w < kWA; ++w) wa[w] = lds32(sb + g.cak_off + w * 128 + lane4);
#pragma unroll
        for (int i = 0; i < kMT; ++i) {
            s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < NT / 2; ++kk) {
                const int n0 = i * 2 * NT + 4 * kk;
                const uint32_t a0 = PKV_I4(wa, n0, sa[2 * kk]), a1 = PKV_I4(wa, n0 + 1, sa[2 * kk]);
                const uint32_t a2 = PKV_I4(wa, n0 + 2, sa[2 * kk + 1]), a3 = PKV_I4(wa, n0 + 3, sa[2 * kk + 1]);
                mma16816(s[i], a0, a1, a2, a3, qhi[2 * kk], qhi[2 * kk + 1]);
                mma16816(s[i], a0, a1, a2, a3, qlo[2 * kk], qlo[2 * kk + 1]);
            }
            if (NT % 2) {
                const int n0 = i * 2 * NT + 4 * (NT / 2);
                const uint32_t a0 = PKV_I4(wa, n0, sa[NT - 1]), a1 = PKV_I4(wa, n0 + 1, sa[NT - 1]);
                mma1688(s[i], a0, a1, qhi[NT - 1]);
                mma1688(s[i], a0, a1, qlo[NT - 1]);
            }
        }
    }
    uint32_t T0[4], T1[4];
    online_softmax<kMT>(s, st, T0, T1);
    // ---- w^T [G][r] = p^T [G][P] . A~_V [P][r]   (scales per token: pairs 16 kk + 8 b + 2c, +1) ----
    uint32_t wh[NT];
    {
        uint32_t sv[2 * kMT], wv[kWV];
#pragma unroll
        for (int i = 0; i < 2 * kMT; ++i) sv[i] = lds32(sc + g.sav_off + 2 * (8 * i + c2));
#pragma unroll
        for (int w = 0; w < kWV; ++w) wv[w] = lds32(sb + g.cav_off + w * 128 + lane4);
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            float wt[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kk = 0; kk < kMT; ++kk) {
                const int n0 = j * (P / 8) + 2 * kk;
                mma16816(wt, T0[kk], 0u, T1[kk], 0u, PKV_I4(wv, n0, sv[2 * kk]), PKV_I4(wv, n0 + 1, sv[2 * kk + 1]));
            }
            wh[j] = pack_bf16(wt[0], wt[1]);
        }
    }
    // ---- o [d][G] += B~_V^T [d][r] . w   (scales per channel = per row of the operand) ----
    {
        uint32_t wr[kWR];
#pragma unroll
        for (int w = 0; w < kWR; ++w) wr[w] = lds32(sb + g.cbv_off + w * 128 + lane4);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t s0 = lds16x2(sc + g.sbv_off + 2 * (16 * i + gq)), s1 = lds16x2(sc + g.sbv_off + 2 * (16 * i + 8 + gq));
#pragma unroll
            for (int kk = 0; kk < NT / 2; ++kk) {
                const int n0 = i * 2 * NT + 4 * kk;
                mma16816(st.o[i], PKV_I4(wr, n0, s0), PKV_I4(wr, n0 + 1, s1), PKV_I4(wr, n0 + 2, s0), PKV_I4(wr, n0 + 3, s1),
                         wh[2 * kk], wh[2 * kk + 1]);
            }
            if (NT % 2) {
                const int n0 = i * 2 * NT + 4 * (NT / 2);
                mma1688(st.o[i], PKV_I4(wr, n0, s0), PKV_I4(wr, n0 + 1, s1), wh[NT - 1]);
            }
        }
    }
}
#undef PKV_I4


// One block of DB rows of a dense page: K rows at sb, V rows at sb + DB*256; `rows` of them are valid.  Query
// columns 2t and 2t+1 of this lane see the first lim0 and lim1 of them (all `rows` unless the call carries several
// query tokens per sequence and the block holds positions after the column's own).
template <int DB>
__device__ __forceinline__ void dense_unit(uint32_t sb, unsigned char *sp, int rows, int lim0, int lim1,
                                           const uint32_t (&qf)[8][2], float scale, WarpState &st, int lane,
                                           float *alphas = nullptr) {
    constexpr int NI = DB / 16;
    const int l7 = lane & 7, mi = lane >> 3, g = lane >> 2;
    if (rows < DB) {
        // unfilled V rows hold stale bytes: zero them so that 0 * garbage cannot make a NaN
        uint4 *v = reinterpret_cast<uint4 *>(sp + DB * kRowBytes + rows * kRowBytes);
        for (int i = lane; i < (DB - rows) * 16; i += 32) v[i] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
    }
    float s[4][4];
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            uint32_t a4[4];
            ldsm_x4(a4, sb + (16 * i + (mi & 1) * 8 + l7) * kRowBytes + (((2 * kk + (mi >> 1)) ^ l7) << 4));
            mma16816(s[i], a4[0], a4[1], a4[2], a4[3], qf[kk][0], qf[kk][1]);
        }
        s[i][0] = 16 * i + g < lim0 ? s[i][0] * scale : kMasked;     s[i][1] = 16 * i + g < lim1 ? s[i][1] * scale : kMasked;
        s[i][2] = 16 * i + 8 + g < lim0 ? s[i][2] * scale : kMasked; s[i][3] = 16 * i + 8 + g < lim1 ? s[i][3] * scale : kMasked;
    }
    uint32_t T0[4], T1[4];
    float al0, al1;
    online_softmax<NI>(s, st, T0, T1, al0, al1);
    if (alphas) { alphas[0] = al0; alphas[1] = al1; }
#pragma unroll
    for (int ii = 0; ii < 8; ++ii) {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            uint32_t a4[4];
            ldsm_x4_t(a4, sb + DB * kRowBytes + (16 * i + (mi >> 1) * 8 + l7) * kRowBytes +
                              (((2 * ii + (mi & 1)) ^ l7) << 4));
            mma16816(st.o[ii], a4[0], a4[1], a4[2], a4[3], T0[i], T1[i]);
        }
    }
}

// ---- Global SVD form (Section 4.2) ------------------------------------------------------------------------
// A region shares its bases; a page holds A_k^T and A_v^T (r x P each).  Per CTA and segment every consumer warp
// gets one copy of B_k before the pages (it computes q~ = B_k q once and keeps it, as two bf16 terms, in its own part
// of the combine area) and one copy of B_v after them (it turns its rank-space sum w = sum_pages A_v^T p into
// o += B_v^T w).  Between the two a page costs s = A_k q~, the softmax, and w += A_v^T p.
// w lives in registers as the mma accumulator of w^T [heads][ranks]: wacc[j] = (head lane >> 2; ranks 8j + 2t, +1).

// The factor that a rescaling of query head lane >> 2 applies to this lane's wacc (the softmax keeps its factors by
// column pair: head 2t in al0, head 2t + 1 in al1, t = lane & 3).
__device__ __forceinline__ float alpha_of_row_head(float al0, float al1, int lane) {
    const int g = lane >> 2;
    const float a0 = __shfl_sync(0xffffffffu, al0, g >> 1), a1 = __shfl_sync(0xffffffffu, al1, g >> 1);
    return (g & 1) ? a1 : a0;
}

template <int NT>
__device__ __forceinline__ void scale_wacc(float (&wacc)[NT][2], float al0, float al1, int lane) {
    if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
        const float aw = alpha_of_row_head(al0, al1, lane);
#pragma unroll
        for (int j = 0; j < NT; ++j) { wacc[j][0] *= aw; wacc[j][1] *= aw; }
    }
}

// B_k (r x d, at sb): q~^T [G][r] = q . B_k^T, scaled, split into two bf16 terms, stored for this lane at
// qts + (2j, 2j + 1) * 128 bytes + lane * 4.  (Rank tiles are taken two at a time: NT is even in this form.)
template <int NT>
__device__ __forceinline__ void global_basis_k(uint32_t sb, const uint32_t (&qf)[8][2], float scale, uint32_t qts, int lane) {
    static_assert(NT % 2 == 0, "the Global SVD form uses ranks that are multiples of 16");
    const int l7 = lane & 7, mi = lane >> 3;
#pragma unroll
    for (int jc = 0; jc < NT; jc += 2) {
        float qt[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j) qt[j][0] = qt[j][1] = qt[j][2] = qt[j][3] = 0.f;
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
            uint32_t b[2][4];
#pragma unroll
            for (int j = 0; j < 2; ++j) ldsm_x4(b[j], sb + (8 * (jc + j) + l7) * kRowBytes + (((4 * qd + mi) ^ l7) << 4));
#pragma unroll
            for (int j = 0; j < 2; ++j) mma16816(qt[j], qf[2 * qd][0], 0u, qf[2 * qd][1], 0u, b[j][0], b[j][1]);
#pragma unroll
            for (int j = 0; j < 2; ++j) mma16816(qt[j], qf[2 * qd + 1][0], 0u, qf[2 * qd + 1][1], 0u, b[j][2], b[j][3]);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float x0 = qt[j][0] * scale, x1 = qt[j][1] * scale;
            const uint32_t hi = pack_bf16(x0, x1);
            const uint32_t lo = pack_bf16(x0 - bf16lo_f(hi), x1 - bf16hi_f(hi));
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(qts + (2 * (jc + j)) * 128 + lane * 4), "r"(hi) : "memory");
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(qts + (2 * (jc + j) + 1) * 128 + lane * 4), "r"(lo) : "memory");
        }
    }
    __syncwarp();
}

// One page: A_k^T at sb, A_v^T at sb + av.
template <int P, int NT>
__device__ __forceinline__ void global_page_unit(uint32_t sb, int av, uint32_t qts, WarpState &st, float (&wacc)[NT][2],
                                                 int lane) {
    using C = Tc<P, NT>;
    static_assert(NT % 2 == 0, "the Global SVD form uses ranks that are multiples of 16");
    const int l7 = lane & 7, mi = lane >> 3;
    const int asw = a_swz<P>(l7);
    float s[4][4];
#pragma unroll
    for (int i = 0; i < C::kMT; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < NT / 2; ++kk) {
        uint32_t a4[C::kMT][4];
#pragma unroll
        for (int i = 0; i < C::kMT; ++i)
            ldsm_x4_t(a4[i], sb + (16 * kk + (mi >> 1) * 8 + l7) * C::kPitchA + (((2 * i + (mi & 1)) ^ asw) << 4));
        const uint32_t h0 = lds32(qts + (4 * kk) * 128 + lane * 4), l0 = lds32(qts + (4 * kk + 1) * 128 + lane * 4);
        const uint32_t h1 = lds32(qts + (4 * kk + 2) * 128 + lane * 4), l1 = lds32(qts + (4 * kk + 3) * 128 + lane * 4);
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) mma16816(s[i], a4[i][0], a4[i][1], a4[i][2], a4[i][3], h0, h1);
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) mma16816(s[i], a4[i][0], a4[i][1], a4[i][2], a4[i][3], l0, l1);
    }
    uint32_t T0[4], T1[4];
    float al0, al1;
    online_softmax<C::kMT>(s, st, T0, T1, al0, al1);
    scale_wacc<NT>(wacc, al0, al1, lane);
    // ---- w^T [G][r] += p^T [G][P] . A_v [P][r] ----
#pragma unroll
    for (int jc = 0; jc < NT; jc += 2) {
        float wt[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j) { wt[j][0] = wacc[jc + j][0]; wt[j][1] = wacc[jc + j][1]; wt[j][2] = wt[j][3] = 0.f; }
#pragma unroll
        for (int qd = 0; qd < C::kMT / 2; ++qd) {
            uint32_t b[2][4];
#pragma unroll
            for (int j = 0; j < 2; ++j) ldsm_x4(b[j], sb + av + (8 * (jc + j) + l7) * C::kPitchA + (((4 * qd + mi) ^ asw) << 4));
#pragma unroll
            for (int j = 0; j < 2; ++j) mma16816(wt[j], T0[2 * qd], 0u, T1[2 * qd], 0u, b[j][0], b[j][1]);
#pragma unroll
            for (int j = 0; j < 2; ++j) mma16816(wt[j], T0[2 * qd + 1], 0u, T1[2 * qd + 1], 0u, b[j][2], b[j][3]);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) { wacc[jc + j][0] = wt[j][0]; wacc[jc + j][1] = wt[j][1]; }
    }
}

// B_v (r x d, at sb): o [d][G] += B_v^T . w, then w = 0.
template <int NT>
__device__ __forceinline__ void global_basis_v(uint32_t sb, float (&wacc)[NT][2], WarpState &st, int lane) {
    const int l7 = lane & 7, mi = lane >> 3;
    uint32_t wh[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) { wh[j] = pack_bf16(wacc[j][0], wacc[j][1]); wacc[j][0] = wacc[j][1] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < NT / 2; ++kk) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t a4[4];
            ldsm_x4_t(a4, sb + (16 * kk + (mi >> 1) * 8 + l7) * kRowBytes + (((2 * i + (mi & 1)) ^ l7) << 4));
            mma16816(st.o[i], a4[0], a4[1], a4[2], a4[3], wh[2 * kk], wh[2 * kk + 1]);
        }
    }
}

__device__ __forceinline__ void reset_state(WarpState &st) {
#pragma unroll
    for (int i = 0; i < 8; ++i) st.o[i][0] = st.o[i][1] = st.o[i][2] = st.o[i][3] = 0.f;
    st.m[0] = st.m[1] = kNegInf;
    st.l[0] = st.l[1] = 0.f;
}

// Index of (sequence, query block, KV head) - what q, out and the tickets are indexed by - for segment `seg` of the
// plan, which is (sequence, KV head); the query block is this CTA's.
__device__ __forceinline__ int query_seg(const DecodeArgs &a, int seg) {
    if (a.q_group == 1) return seg;
    const int H = a.geo.n_kv_heads;
    return ((seg / H) * a.q_group + (int)(blockIdx.x % a.q_group)) * H + seg % H;
}
// This CTA's partial state of segment `seg`, or with `cta` = the segment's first range, the first of its partial
// states; consecutive ranges' states of one query block are q_group slots apart.
__device__ __forceinline__ float *partial_slot(const DecodeArgs &a, int cta_range, int seg) {
    return a.partials + (((long long)cta_range + seg) * a.q_group + blockIdx.x % a.q_group) * kPartialFloats;
}

// Query column n of a segment's score tile = query head n % G of the (n / G)-th query token of the plan entry's
// block; with one query per sequence (q_len = 1) that is query head n.  Row of q / out it maps to, or -1.
// (`seg` here is a query_seg() index.)
template <bool kFast = true>
__device__ __forceinline__ long long q_row(const DecodeArgs &a, int seg, int n) {
    // one query per sequence: seg = entry * H + head and H_q = H * G, so the row is seg * G + n - no division (this
    // sits between a stand-alone launch's release and its first load, and on the merging CTA's way out).  kFast = false
    // leaves the shortcut out: the Global SVD form of the decode kernel has no register to spare for a second copy of
    // the code behind it (its inner loop spills more with it).
    if (kFast && a.q_len == 1) return n < a.geo.group ? (long long)seg * a.geo.group + n : -1;
    const int H = a.geo.n_kv_heads, G = a.geo.group;
    const int entry = seg / H, head = seg % H, jl = n / G, j = (entry % a.q_nblk) * a.q_tpt + jl;
    if (jl >= a.q_tpt || j >= a.q_len) return -1;
    return ((long long)(entry / a.q_nblk) * a.q_len + j) * a.geo.n_q_heads + head * G + n % G;
}

// Loads the lane's share of the segment's queries.  Returns, packed in 16-bit halves, how many of the sequence's
// newest positions the lane's columns 2t and 2t+1 must not see (q_len - 1 - the column's query token).
__device__ __forceinline__ int load_q(const DecodeArgs &a, int seg, uint32_t (&qf)[8][2], int lane, long long row) {
    const int t = lane & 3;
    if (row >= 0) {
        const uint32_t *q = reinterpret_cast<const uint32_t *>(reinterpret_cast<const __nv_bfloat16 *>(a.q) + row * kHeadDim);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) { qf[kk][0] = __ldg(q + 8 * kk + t); qf[kk][1] = __ldg(q + 8 * kk + 4 + t); }
    } else {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) qf[kk][0] = qf[kk][1] = 0u;
    }
    if (a.q_len == 1) return 0;
    const int G = a.geo.group, j0 = ((seg / a.geo.n_kv_heads) % a.q_nblk) * a.q_tpt;
    const int b0 = max(0, a.q_len - 1 - j0 - (2 * t) / G), b1 = max(0, a.q_len - 1 - j0 - (2 * t + 1) / G);
    return b0 | (b1 << 16);
}
template <bool kFast = true>
__device__ __forceinline__ int load_q(const DecodeArgs &a, int seg, uint32_t (&qf)[8][2], int lane) {
    return load_q(a, seg, qf, lane, q_row<kFast>(a, seg, lane >> 2));
}

// Writes the final result of one (entry, KV head) for query column hq, dims d4..d4+3.
// With a.state set the call returns the softmax state instead (Eq. 5's inputs, for a merge across caches that
// hold different token ranges of the sequence): row = o[0..d) unnormalised, then m (the running maximum of the
// scaled scores in base-2 units, i.e. of s * softmax_scale * log2 e), then l.
template <bool kFast = true>
__device__ __forceinline__ void store_out(const DecodeArgs &a, int seg, int hq, int d4, float4 acc, float M, float L) {
    const long long row = q_row<kFast>(a, seg, hq);
    if (row < 0) return;
    if (a.state) {
        float *st = a.state + row * (kHeadDim + 2);
        *reinterpret_cast<float2 *>(st + d4) = make_float2(acc.x, acc.y);     // rows are 8-byte aligned only
        *reinterpret_cast<float2 *>(st + d4 + 2) = make_float2(acc.z, acc.w);
        if (d4 == 0) { st[kHeadDim] = M; st[kHeadDim + 1] = L; }
        return;
    }
    const float inv = 1.f / L;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    const long long off = row * kHeadDim + d4;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 packed;
    packed.x = *reinterpret_cast<unsigned *>(&lo);
    packed.y = *reinterpret_cast<unsigned *>(&hi);
    *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + off) = packed;
    if (a.out_f32) *reinterpret_cast<float4 *>(a.out_f32 + off) = acc;
}

// One step of Eq. 5: folds the state (o, m, l) into the running (tot, Mr, Lr).  Spelled with explicit roundings so
// that every caller (the merge inside the decode kernel, the separate merge kernel) produces the same bits.
__device__ __forceinline__ void fold_state(float4 &tot, float &Mr, float &Lr, const float4 o, float m, float l) {
    const float Mn = fmaxf(Mr, m);
    const float fa = exp2f(Mr - Mn), fb = exp2f(m - Mn);
    tot.x = __fmaf_rn(fb, o.x, __fmul_rn(tot.x, fa)); tot.y = __fmaf_rn(fb, o.y, __fmul_rn(tot.y, fa));
    tot.z = __fmaf_rn(fb, o.z, __fmul_rn(tot.z, fa)); tot.w = __fmaf_rn(fb, o.w, __fmul_rn(tot.w, fa));
    Lr = __fmaf_rn(fb, l, __fmul_rn(Lr, fa));
    Mr = Mn;
}

// Eq. 5 across CTAs: partial states summed in CTA order with a running maximum (one pass).
// A thread owns E items (query head, four dims): ctid, ctid + kThreads, ...; kBatch parts' loads are in flight at a
// time, because with dozens of parts it is the latency of these loads that the rest of the GPU waits for.
template <int E, int kBatch, bool kFast = true>
__device__ __forceinline__ void merge_parts(const DecodeArgs &a, const float *first, int np, int seg, int ctid,
                                            float *dst) {
    const long long stride = (long long)a.q_group * kPartialFloats;     // between the states of consecutive ranges
    constexpr int kThreads = kConsumerWarps * 32;
    const int n_items = a.q_cols * 32;
    const int d4 = (ctid & 31) * 4;                               // kThreads is a multiple of 32
    bool has[E];
    int hq[E];
    float4 tot[E];
    float Mr[E], Lr[E];
#pragma unroll
    for (int e = 0; e < E; ++e) {
        has[e] = ctid + e * kThreads < n_items;
        hq[e] = has[e] ? (ctid + e * kThreads) >> 5 : 0;
        tot[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        Mr[e] = kNegInf;
        Lr[e] = 0.f;
    }
    for (int k0 = 0; k0 < np; k0 += kBatch) {
        float4 o[E][kBatch];
        float m[E][kBatch], l[E][kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const float *pk = first + (long long)min(k0 + j, np - 1) * stride;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                o[e][j] = __ldcg(reinterpret_cast<const float4 *>(pk + hq[e] * kHeadDim + d4));
                m[e][j] = __ldcg(pk + kMaxGroup * kHeadDim + hq[e]);
                l[e][j] = __ldcg(pk + kMaxGroup * kHeadDim + kMaxGroup + hq[e]);
            }
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            if (k0 + j < np) {
#pragma unroll
                for (int e = 0; e < E; ++e) fold_state(tot[e], Mr[e], Lr[e], o[e][j], m[e][j], l[e][j]);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (!has[e]) continue;
        if (dst) {                                                    // the sum is itself a partial state (of a group)
            *reinterpret_cast<float4 *>(dst + hq[e] * kHeadDim + d4) = tot[e];
            if (d4 == 0) { dst[kMaxGroup * kHeadDim + hq[e]] = Mr[e]; dst[kMaxGroup * kHeadDim + kMaxGroup + hq[e]] = Lr[e]; }
        } else {
            store_out<kFast>(a, seg, hq[e], d4, tot[e], Mr[e], Lr[e]);
        }
    }
}

// One ticket of a counter in global memory, with release and acquire semantics at device scope.
__device__ __forceinline__ int draw_ticket(int *counter) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
    return old;
}

#define PKV_CONSUMER_BARRIER() asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory")

// All consumer warps combine their states of one segment (Eq. 5 inside the CTA).  If the segment
// lies wholly in this CTA the result is final; otherwise the CTA writes one partial state, takes a
// ticket, and the CTA that draws the last ticket of the segment applies Eq. 5 across CTAs.  Partials
// are always summed in CTA order, so the result does not depend on which CTA arrives last.
template <bool kFast = true>
__device__ __forceinline__ void flush_segment(const DecodeArgs &a, float *comb, volatile int *last_flag, WarpState &st,
                                              int seg, const PlanSeg ps, int warp, int lane, int ctid, int n_active,
                                              long long *trace) {
    constexpr int kThreads = kConsumerWarps * 32, kItems = kMaxGroup * 32;   // item = (query head, 4 dims)
    const int g = lane >> 2, t = lane & 3;
    if (trace && ctid == 0) trace[9] = clock64();
    if (warp < n_active) {
        float l0 = st.l[0], l1 = st.l[1];
#pragma unroll
        for (int off = 4; off <= 16; off <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, off);
            l1 += __shfl_xor_sync(0xffffffffu, l1, off);
        }
        float *mine = comb + warp * kPartialFloats;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            mine[(2 * t) * kHeadDim + 16 * i + g] = st.o[i][0];
            mine[(2 * t + 1) * kHeadDim + 16 * i + g] = st.o[i][1];
            mine[(2 * t) * kHeadDim + 16 * i + 8 + g] = st.o[i][2];
            mine[(2 * t + 1) * kHeadDim + 16 * i + 8 + g] = st.o[i][3];
        }
        if (g == 0) {
            mine[kMaxGroup * kHeadDim + 2 * t] = st.m[0];
            mine[kMaxGroup * kHeadDim + 2 * t + 1] = st.m[1];
            mine[kMaxGroup * kHeadDim + kMaxGroup + 2 * t] = l0;
            mine[kMaxGroup * kHeadDim + kMaxGroup + 2 * t + 1] = l1;
        }
    }
    // (where the state goes is worked out while the other warps arrive: divisions by run-time values)
    const int qseg = query_seg(a, seg);
    float *part = partial_slot(a, blockIdx.x / a.q_group, seg);
    PKV_CONSUMER_BARRIER();
    // overlap mode 1: partial states, tickets and `out` may still be in use by the preceding launch
    if (a.overlap == 1) asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int item = ctid; item < kItems; item += kThreads) {
        const int hq = item >> 5, d4 = (item & 31) * 4;
        float M = kNegInf;
        for (int w = 0; w < n_active; ++w) M = fmaxf(M, comb[w * kPartialFloats + kMaxGroup * kHeadDim + hq]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float L = 0.f;
        for (int w = 0; w < n_active; ++w) {
            const float *cw = comb + w * kPartialFloats;
            const float f = exp2f(cw[kMaxGroup * kHeadDim + hq] - M);
            const float4 o = *reinterpret_cast<const float4 *>(cw + hq * kHeadDim + d4);
            acc.x += f * o.x; acc.y += f * o.y; acc.z += f * o.z; acc.w += f * o.w;
            L += f * cw[kMaxGroup * kHeadDim + kMaxGroup + hq];
        }
        if (ps.n_parts <= 1) {
            if (hq < a.q_cols) store_out<kFast>(a, qseg, hq, d4, acc, M, L);
        } else {
            *reinterpret_cast<float4 *>(part + hq * kHeadDim + d4) = acc;
            if ((item & 31) == 0) {
                part[kMaxGroup * kHeadDim + hq] = M;
                part[kMaxGroup * kHeadDim + kMaxGroup + hq] = L;
            }
        }
    }
    if (ps.n_parts > 1) {
        // Drawing a ticket: the barrier orders every thread's stores of the state before thread 0's atomic, whose
        // release half makes them visible device-wide before the ticket is drawn; on the way back its acquire half
        // and the barrier order the other CTAs' states (whose tickets this one has seen) before every thread's reads
        // of them (the pattern of a cooperative grid sync, with the two fences folded into the atomic).
        // A segment held by more than kMergeFan CTAs is summed in two levels: the CTAs form groups of kMergeFan
        // consecutive ranges; the last of a group to arrive sums the group's states into a group state, and the last
        // group to arrive sums the group states.  The slowest CTA of the launch then has one short sum of its
        // group and one of the groups ahead of it instead of one long sum of everything, and the other groups'
        // sums are over before it arrives.  The grouping is fixed, so the bits do not depend on who arrives when.
        const float *first = partial_slot(a, ps.cta_first, seg);
        int np = ps.n_parts;
        bool mine = true;                                  // this CTA still carries the sum upwards
        if (a.q_group == 1 && ps.n_parts > kMergeFan) {
            const int k = blockIdx.x - ps.cta_first, g = k / kMergeFan;
            const int gsize = min(kMergeFan, ps.n_parts - g * kMergeFan);
            const int gslot0 = (ps.cta_first + seg) / kMergeFan + seg;     // group slots of consecutive groups and segments never collide
            PKV_CONSUMER_BARRIER();
            if (ctid == 0) *last_flag = (draw_ticket(a.gtickets + gslot0 + g) == gsize - 1);
            PKV_CONSUMER_BARRIER();
            mine = *last_flag != 0;
            if (mine) {
                float *dst = a.gpartials + (long long)(gslot0 + g) * kPartialFloats;
                const float *gfirst = first + (long long)g * kMergeFan * kPartialFloats;
                if (a.q_cols * 32 <= kThreads) merge_parts<1, 16, kFast>(a, gfirst, gsize, qseg, ctid, dst);
                else merge_parts<2, 8, kFast>(a, gfirst, gsize, qseg, ctid, dst);
                if (ctid == 0) a.gtickets[gslot0 + g] = 0;     // ready for the next launch
                first = a.gpartials + (long long)gslot0 * kPartialFloats;
                np = (ps.n_parts + kMergeFan - 1) / kMergeFan;
            }
        }
        if (mine) {
            PKV_CONSUMER_BARRIER();
            if (ctid == 0) *last_flag = (draw_ticket(a.tickets + qseg) == np - 1);
            PKV_CONSUMER_BARRIER();
            if (trace && ctid == 0) trace[10] = clock64();
            if (*last_flag) {
                if (a.q_cols * 32 <= kThreads) merge_parts<1, 16, kFast>(a, first, np, qseg, ctid, nullptr);
                else merge_parts<2, 8, kFast>(a, first, np, qseg, ctid, nullptr);
                if (ctid == 0) a.tickets[qseg] = 0;         // ready for the next launch
                if (trace && ctid == 0) trace[13] = clock64();
            }
        }
    }
    PKV_CONSUMER_BARRIER();
}

template <int P, int NT, int F>
__global__ void __launch_bounds__(kDecodeThreads, 2) decode_tc_kernel(const __grid_constant__ DecodeArgs a) {
    constexpr int kDB = kDenseBlock<P, NT, F>;
    constexpr bool I4 = F == 1, kGlobal = F == 2;
    Range rg;
    if (!load_range(a, rg)) return;
    const Geometry &geo = a.geo;
    const int S = geo.n_stages;
    // A warp that has reached the next segment keeps its stage until every warp has; so no more warps may
    // take units than there are stages.  The others only take part in the flush barriers.
    const int W = min(kConsumerWarps, S);
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *stages = smem;
    const int stage_bytes = geo.stage_bytes, blob_bytes = geo.blob_bytes;
    float *comb = reinterpret_cast<float *>(smem + (size_t)S * stage_bytes);
    unsigned long long *full_bar = reinterpret_cast<unsigned long long *>(comb + kConsumerWarps * kPartialFloats);
    unsigned long long *empty_bar = full_bar + S;
    StageDesc *descs = reinterpret_cast<StageDesc *>(empty_bar + S);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(descs + S);
    volatile int *last_flag = abort_flag + 1;
    // armed[s] = 1 + the unit last armed in stage s.  A parity wait cannot tell phase n from phase n-2, and bulk
    // copies may land out of order, so a consumer first makes sure that its own unit has been armed (which the
    // producer does only after the stage's previous occupant was consumed) and only then waits on the barrier.
    volatile int *armed = abort_flag + 2;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    long long *trace = a.trace ? a.trace + (long long)kTraceSlots * blockIdx.x : nullptr;
    if (trace && tid == 0) {
        unsigned long long gt;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(gt));
        trace[0] = (long long)gt;
        trace[2] = clock64();
        for (int i = 8; i < kTraceSlots; ++i) trace[i] = 0;
    }
    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(full_bar + s), 1); mbar_init(smem_u32(empty_bar + s), 1); }
        *abort_flag = 0;
        for (int s = 0; s < S; ++s) armed[s] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (F == 0 && stage_bytes > blob_bytes) {
        // Tile loads of 8 rows read past a rank that is not a multiple of 8; past the last matrix that is the
        // tail of the stage, which no copy of a factor page ever writes.  Those values are multiplied by exact
        // zeros, so they only have to be finite: clear the tails once.
        const int tail16 = (stage_bytes - blob_bytes) >> 4;
        for (int i = tid; i < S * tail16; i += kDecodeThreads)
            reinterpret_cast<uint4 *>(stages + (size_t)(i / tail16) * stage_bytes + blob_bytes)[i % tail16] =
                make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch: let the next kernel on the stream begin as SMs free up.  What the producer
    // reads - plan, page table, token counts, pages - is written only by this library's own uploads and kernels
    // (append, compression, pkv_write_factors), and the host makes the first decode launch after any of those an
    // ordinary one, which starts when they are done; so the producer never has to wait for the kernel before this
    // one and fills the ring while that kernel is still finishing.  The queries may come from that kernel:
    // mode 0 (no promise from the caller) makes every consumer warp wait for it before it reads q.  Mode 1 waits
    // later, before the shared split-K scratch is touched (flush_segment); mode 2 never waits: the host rotates
    // the scratch and drains the stream in time.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kConsumerWarps) {
        // ------------------------------ producer ------------------------------
        const PlanEntry *entries = reinterpret_cast<const PlanEntry *>(a.plan + a.plan_entry);
        int k = 0, seg_local = 0;
        bool ok = true;
        const bool keep = a.q_group > 1;     // sibling CTAs read the same pages: leave them in L2 for one another
        // Lanes 0 .. n_here-1 arm their own units (kind, rows, after, src are per lane), S at a time (one stage
        // each).  No lane blocks the others: all lanes poll together, and a unit is armed and tagged the moment its
        // stage is free.  (Waiting for a whole group before telling the consumers can deadlock: a consumer may have
        // to see unit k, of a later segment, to join the flush barrier that another warp must pass before it
        // releases the stage that unit k + 1 is waiting for.)
        auto arm = [&](int n_here, int kind, int rows, int after, const unsigned char *src) {
            for (int j0 = 0; j0 < n_here && ok; j0 += S) {
                const int kj = k + lane, s = kj % S;
                bool pending = lane >= j0 && lane < min(j0 + S, n_here);
                const long long t0 = clock64();
                while (__any_sync(0xffffffffu, pending)) {
                    if (pending && a.drop_unit == kj && blockIdx.x == 0) {
                        pending = false;             // test hook: this unit is never armed, so its consumer's wait runs out
                    } else if (pending && (kj < S || mbar_try_wait(smem_u32(empty_bar + s), ((kj / S) - 1) & 1))) {
                        descs[s] = StageDesc{kind, rows, seg_local, after};
                        const uint32_t bar = smem_u32(full_bar + s);
                        const uint32_t dst = smem_u32(stages + (size_t)s * stage_bytes);
                        if (kind == kKindFactor) {
                            mbar_arrive_expect_tx(bar, blob_bytes);
                            if (keep) bulk_g2s_keep(dst, src, blob_bytes, bar);
                            else bulk_g2s(dst, src, blob_bytes, bar);
                        } else if (kind == kKindBasisK || kind == kKindBasisV) {
                            // (every CTA of the segment reads the same basis: leave it in L2)
                            mbar_arrive_expect_tx(bar, geo.global_rank * kRowBytes);
                            bulk_g2s_keep(dst, src, geo.global_rank * kRowBytes, bar);
                        } else if (rows > 0) {
                            mbar_arrive_expect_tx(bar, 2 * rows * kRowBytes);
                            if (keep) {
                                bulk_g2s_keep(dst, src, rows * kRowBytes, bar);
                                bulk_g2s_keep(dst + kDB * kRowBytes, src + P * kRowBytes, rows * kRowBytes, bar);
                            } else {
                                bulk_g2s(dst, src, rows * kRowBytes, bar);
                                bulk_g2s(dst + kDB * kRowBytes, src + P * kRowBytes, rows * kRowBytes, bar);
                            }
                        } else {
                            mbar_arrive(bar);
                        }
                        st_release_smem(armed + s, kj + 1);
                        if (trace && kj == 0) trace[3] = clock64();
                        pending = false;
                    }
                    if (clock64() - t0 > a.wait_clocks) break;         // about a second: give up
                }
                ok = !__any_sync(0xffffffffu, pending);
            }
            k += n_here;
        };
        PlanCta cur = rg.start;
        while (ok && !(cur.entry == rg.end.entry && cur.head == rg.end.head && cur.unit == rg.end.unit)) {
            const PlanEntry e = cur.entry == rg.start.entry ? rg.first_entry : entries[cur.entry];
            const HeadUnits hu = head_units(geo, e);
            const bool last_run = cur.entry == rg.end.entry && cur.head == rg.end.head;
            const int u_end = last_run ? rg.end.unit : hu.units;
            const int T = a.n_tokens[(long long)e.seq * geo.n_layers + a.layer];
            const int *pt = a.page_table + ((long long)e.seq * geo.n_layers + a.layer) * geo.max_pages;
            // Global SVD form: if this run holds factor pages, every consumer warp gets the region's B_k ahead of
            // them and its B_v behind them (W consecutive units go to W different warps)
            const bool run_global = kGlobal && max(cur.unit, hu.d0) < min(u_end, hu.d0 + hu.nf);
            const unsigned char *bsrc = kGlobal ? a.basis + (((long long)e.seq * geo.n_layers + a.layer) * geo.n_kv_heads + cur.head) *
                                                                geo.basis_head_bytes : nullptr;
            if (run_global) arm(W, kKindBasisK, 1, 0, bsrc);
            for (int u0 = cur.unit; u0 < u_end && ok; u0 += 32) {
                const int u = u0 + lane;
                int kind = kKindDense, rows = 0, after = 0;
                const unsigned char *src = nullptr;
                if (u < u_end) {
                    int page, blk;
                    unit_to_page(geo, hu, u, page, blk, kind);
                    const int slot = pt[page];
                    if (slot < 0 || slot >= (kind == kKindFactor ? geo.n_factor_slots : geo.n_dense_slots)) {
                        atomicAdd(a.status + 2, 1);          // corrupt page table: skip the unit, leave a mark
                        kind = kKindDense;
                        rows = 0;
                    } else if (kind == kKindFactor) {
                        rows = P;
                        src = a.factor_pool + (long long)slot * geo.factor_slot_bytes + (long long)cur.head * geo.blob_bytes;
                    } else {
                        rows = max(0, min(kDB, T - page * P - blk * kDB));
                        after = max(0, T - page * P - blk * kDB - rows);
                        src = a.dense_pool + (long long)slot * geo.dense_slot_bytes +
                              (long long)cur.head * geo.dense_head_bytes + blk * kDB * kRowBytes;
                    }
                }
                arm(min(32, u_end - u0), kind, rows, after, src);
            }
            if (run_global && ok) arm(W, kKindBasisV, 1, 0, bsrc + geo.global_rank * kRowBytes);
            if (last_run) break;
            cur.unit = 0;
            if (++cur.head == geo.n_kv_heads) { cur.head = 0; ++cur.entry; }
            ++seg_local;
        }
        // one end marker per consumer warp
        for (int w = 0; w < W && ok; ++w, ++k) {
            if (lane == 0) {
                const int s = k % S;
                if (k >= S && !mbar_wait(smem_u32(empty_bar + s), ((k / S) - 1) & 1, a.wait_clocks)) ok = false;
                if (ok) {
                    descs[s] = StageDesc{kKindEnd, 0, rg.n_local_segs, 0};
                    mbar_arrive(smem_u32(full_bar + s));
                    st_release_smem(armed + s, k + 1);
                }
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicAdd(a.status, 1);
            // let copies already in flight land before the CTA retires
            for (int back = 1; back <= min(k, S); ++back) {
                const int kk = k - back;
                (void)mbar_wait(smem_u32(full_bar + kk % S), (kk / S) & 1, a.wait_clocks);
            }
        }
    } else {
        // ------------------------------ consumers ------------------------------
        WarpState st;
        reset_state(st);
        // Only the first and the last segment of a range can be shared with other CTAs.  What their flushes need
        // from global memory - the segment's place in the plan, its ticket - is fetched now, while the warp would
        // otherwise just wait for the kernel before this one (the plan is host-written, the tickets are zero
        // between launches).
        const PlanSeg *plan_segs = reinterpret_cast<const PlanSeg *>(a.plan + a.plan_seg);
        const PlanSeg ps_first = plan_segs[rg.seg_first], ps_last = plan_segs[rg.seg_first + rg.n_local_segs - 1];
        if (lane == 0 && a.q_group == 1) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(a.tickets + rg.seg_first));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(a.tickets + rg.seg_first + rg.n_local_segs - 1));
        }
        auto seg_info = [&](int sg) { return sg == 0 ? ps_first : (sg == rg.n_local_segs - 1 ? ps_last : PlanSeg{(int)(blockIdx.x / a.q_group), 1}); };
        // (where this lane's queries of the first segment lie is worked out before the wait: several divisions by
        // run-time values, which a stand-alone launch would otherwise pay between its release and its first load)
        const long long first_q_row = warp < W ? q_row<!kGlobal>(a, query_seg(a, rg.seg_first), lane >> 2) : -1;
        if (!a.overlap) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (trace && tid == 0) trace[8] = clock64();
        if (warp >= W) {
            for (int sg = 0; sg < rg.n_local_segs; ++sg)
                flush_segment<!kGlobal>(a, comb, last_flag, st, rg.seg_first + sg, seg_info(sg), warp, lane, tid, W, nullptr);
            return;
        }
        uint32_t qf[8][2];
        int cur_seg = 0;
        int hidden = load_q(a, query_seg(a, rg.seg_first), qf, lane, first_q_row);
        // Global SVD form: this warp's rank-space sum, and where it keeps q~ (its own part of the combine area, which it
        // overwrites with its state only at a flush, when q~ of that segment is no longer needed)
        float wacc[kGlobal ? NT : 1][2];
#pragma unroll
        for (int j = 0; j < (kGlobal ? NT : 1); ++j) wacc[j][0] = wacc[j][1] = 0.f;
        const uint32_t qts = smem_u32(comb + warp * kPartialFloats);
        bool ok = true;
        for (int k = warp;; k += W) {
            const int s = k % S;
            if (ok && (*abort_flag || !wait_armed(armed + s, k, a.wait_clocks) ||
                       !mbar_wait(smem_u32(full_bar + s), (k / S) & 1, a.wait_clocks))) {
                ok = false;
                if (lane == 0) { *abort_flag = 1; atomicAdd(a.status, 1); }
            }
            StageDesc dsc = ok ? descs[s] : StageDesc{kKindEnd, 0, rg.n_local_segs, 0};
            if (trace && k == 0 && lane == 0) trace[4] = clock64();
            if (trace && dsc.kind == kKindEnd && warp == 0 && lane == 0) { trace[5] = clock64(); trace[7] = k; }
            if (cur_seg < dsc.seg) {
                // the old segment's queries are no longer needed: fetch the new ones now, so that their latency
                // hides behind the flush
                if (dsc.seg < rg.n_local_segs) hidden = load_q<!kGlobal>(a, query_seg(a, rg.seg_first + dsc.seg), qf, lane);
                while (cur_seg < dsc.seg) {
                    flush_segment<!kGlobal>(a, comb, last_flag, st, rg.seg_first + cur_seg, seg_info(cur_seg), warp, lane, tid, W, trace);
                    ++cur_seg;
                    reset_state(st);
                }
            }
            if (dsc.kind == kKindEnd) break;
            dsc.rows = min(dsc.rows, dsc.kind == kKindFactor ? P : kDB);
            if (dsc.rows > 0) {
                const uint32_t sb = smem_u32(stages + (size_t)s * stage_bytes);
                if constexpr (kGlobal) {
                    if (dsc.kind == kKindBasisK) global_basis_k<NT>(sb, qf, geo.scale_log2e, qts, lane);
                    else if (dsc.kind == kKindBasisV) global_basis_v<NT>(sb, wacc, st, lane);
                    else if (dsc.kind == kKindFactor) global_page_unit<P, NT>(sb, geo.av_off, qts, st, wacc, lane);
                    else {
                        float al[2];
                        dense_unit<kDB>(sb, stages + (size_t)s * stage_bytes, dsc.rows, dsc.rows, dsc.rows, qf, geo.scale_log2e, st,
                                        lane, al);
                        scale_wacc<NT>(wacc, al[0], al[1], lane);
                        if (dsc.rows < kDB) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    }
                } else if (dsc.kind == kKindFactor) {
                    if (I4) factor_unit_int4<P, NT>(sb, geo, qf, st, lane);
                    else factor_unit<P, NT>(sb, geo.ak_off, geo.bk_off, geo.av_off, geo.bv_off, geo.rank_k, geo.rank_v, qf,
                                            geo.scale_log2e, st, lane);
                } else {
                    // a column does not see the sequence's last `hidden` positions; `after` of those lie beyond
                    // this unit's rows
                    const int lim0 = dsc.rows - max(0, (hidden & 0xffff) - dsc.after);
                    const int lim1 = dsc.rows - max(0, (hidden >> 16) - dsc.after);
                    dense_unit<kDB>(sb, stages + (size_t)s * stage_bytes, dsc.rows, lim0, lim1, qf, geo.scale_log2e, st, lane);
                    if (dsc.rows < kDB) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(empty_bar + s));
        }
        if (trace && warp == 0 && lane == 0) {
            unsigned long long gt;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(gt));
            trace[1] = (long long)gt;
            trace[6] = clock64();
        }
    }
}

// =============================================================================
// Row-block kernel: many queries per sequence (a chunk of a prefill).
//
// The pipeline kernel above keeps queries in the 8-wide column operand, which suits G <= 8 query heads of one
// token.  With q_len * G >= 64 query rows per (sequence, KV head) the roles are swapped: 16 (query token, query
// head) rows are the row operand of every product, a warp owns 16 rows, a CTA 64, and all four warps read each
// unit from the same shared-memory stage, so the sequence's pages are fetched once per 64 rows instead of once
// per 8 columns.  The tile loads are the very ones of factor_unit / dense_unit (the storage swizzles serve both
// roles); only which operand they feed changes.  One CTA handles one (sequence, KV head, block of 64 rows)
// from the first unit to the last, so there is no split-K state to merge.
// =============================================================================
constexpr int kBlockWarps = 4;
constexpr int kBlockRows = 16 * kBlockWarps;
constexpr int kBlockThreads = (kBlockWarps + 1) * 32;

// Running state of rows g and g + 8 (g = lane >> 2) of a warp's 16 rows.
struct RowState {
    float o[16][4];       // o[c]: (row g, channels 8c+2t, +1), (row g+8, same channels);  t = lane & 3
    float m[2], l[2];     // l is this lane's share of the row sum; summed over t at the end
};

// Softmax over NS score tiles of 8 tokens for rows g, g+8; returns p as the row operand of the next product:
// pa[i] = k-step over tokens 16i .. 16i+15.
template <int NS>
__device__ __forceinline__ void row_softmax(float (&s)[NS][4], RowState &st, uint32_t (&pa)[NS / 2][4]) {
    float mx0 = kNegInf, mx1 = kNegInf;
#pragma unroll
    for (int b = 0; b < NS; ++b) {
        mx0 = fmaxf(mx0, fmaxf(s[b][0], s[b][1]));
        mx1 = fmaxf(mx1, fmaxf(s[b][2], s[b][3]));
    }
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
    }
    const float mn0 = fmaxf(st.m[0], mx0), mn1 = fmaxf(st.m[1], mx1);
    const float al0 = exp2f(st.m[0] - mn0), al1 = exp2f(st.m[1] - mn1);
    st.m[0] = mn0; st.m[1] = mn1;
    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
    for (int b = 0; b < NS; ++b) {
        s[b][0] = exp2f(s[b][0] - mn0); s[b][1] = exp2f(s[b][1] - mn0);
        s[b][2] = exp2f(s[b][2] - mn1); s[b][3] = exp2f(s[b][3] - mn1);
        sum0 += s[b][0] + s[b][1];
        sum1 += s[b][2] + s[b][3];
    }
    st.l[0] = st.l[0] * al0 + sum0;
    st.l[1] = st.l[1] * al1 + sum1;
    if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
        for (int c = 0; c < 16; ++c) { st.o[c][0] *= al0; st.o[c][1] *= al0; st.o[c][2] *= al1; st.o[c][3] *= al1; }
    }
#pragma unroll
    for (int i = 0; i < NS / 2; ++i) {
        pa[i][0] = pack_bf16(s[2 * i][0], s[2 * i][1]);
        pa[i][1] = pack_bf16(s[2 * i][2], s[2 * i][3]);
        pa[i][2] = pack_bf16(s[2 * i + 1][0], s[2 * i + 1][1]);
        pa[i][3] = pack_bf16(s[2 * i + 1][2], s[2 * i + 1][3]);
    }
}

// One factor page for 16 query rows (Eq. 4 with the queries as rows): q~ = q B_k^T, s = q~ A_k^T, p = softmax
// numerators, w = p A_v, o += w B_v.  qf[kk] = the row operand of q for channels 16kk .. 16kk+15.
template <int P, int NT>
__device__ __forceinline__ void block_factor_unit(uint32_t sb, int ak, int bk, int av, int bv, int rk, int rv,
                                                  const uint32_t (&qf)[8][4], float scale, RowState &st, int lane) {
    using C = Tc<P, NT>;
    constexpr int NS = P / 8;
    const int l7 = lane & 7, mi = lane >> 3, t2 = (lane & 3) * 2;
    const int asw = a_swz<P>(l7);
    // ---- q~ [16][r] = q [16][d] . B_k^T, scaled, split into two bf16 terms ----
    uint32_t qh[NT][2], ql[NT][2];                  // per rank tile: rows g, g+8
    {
        float qt[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) qt[j][0] = qt[j][1] = qt[j][2] = qt[j][3] = 0.f;
        // The asm statements keep their order, so loads are issued by hand ahead of the products that use them:
        // here one group of NT tiles ahead.
        uint32_t b[2][NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) ldsm_x4(b[0][j], sb + bk + (8 * j + l7) * kRowBytes + ((mi ^ l7) << 4));
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
            if (qd + 1 < 4) {
#pragma unroll
                for (int j = 0; j < NT; ++j)
                    ldsm_x4(b[(qd + 1) & 1][j], sb + bk + (8 * j + l7) * kRowBytes + (((4 * (qd + 1) + mi) ^ l7) << 4));
            }
#pragma unroll
            for (int j = 0; j < NT; ++j)
                mma16816(qt[j], qf[2 * qd][0], qf[2 * qd][1], qf[2 * qd][2], qf[2 * qd][3], b[qd & 1][j][0], b[qd & 1][j][1]);
#pragma unroll
            for (int j = 0; j < NT; ++j)
                mma16816(qt[j], qf[2 * qd + 1][0], qf[2 * qd + 1][1], qf[2 * qd + 1][2], qf[2 * qd + 1][3], b[qd & 1][j][2], b[qd & 1][j][3]);
        }
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const bool v0 = 8 * j + t2 < rk, v1 = 8 * j + t2 + 1 < rk;
            const float x0 = v0 ? qt[j][0] * scale : 0.f, x1 = v1 ? qt[j][1] * scale : 0.f;
            const float y0 = v0 ? qt[j][2] * scale : 0.f, y1 = v1 ? qt[j][3] * scale : 0.f;
            qh[j][0] = pack_bf16(x0, x1);
            qh[j][1] = pack_bf16(y0, y1);
            ql[j][0] = pack_bf16(x0 - bf16lo_f(qh[j][0]), x1 - bf16hi_f(qh[j][0]));
            ql[j][1] = pack_bf16(y0 - bf16lo_f(qh[j][1]), y1 - bf16hi_f(qh[j][1]));
        }
    }
    // ---- s [16][P] = q~ . A_k^T   (A_k^T rows = ranks: transposed tile loads give the column operand) ----
    float s[NS][4];
#pragma unroll
    for (int b = 0; b < NS; ++b) s[b][0] = s[b][1] = s[b][2] = s[b][3] = 0.f;
    if (NT >= 2) {
        // a4 = (ranks lo, tokens 16i..), (ranks lo, tokens 16i+8..), (ranks hi, 16i..), (ranks hi, 16i+8..); one item ahead
        constexpr int kItems = (NT / 2) * C::kMT;
        uint32_t a4[2][4];
        ldsm_x4_t(a4[0], sb + ak + ((mi >> 1) * 8 + l7) * C::kPitchA + (((mi & 1) ^ asw) << 4));
#pragma unroll
        for (int it = 0; it < kItems; ++it) {
            const int kk = it / C::kMT, i = it % C::kMT;
            if (it + 1 < kItems) {
                const int kn = (it + 1) / C::kMT, in = (it + 1) % C::kMT;
                ldsm_x4_t(a4[(it + 1) & 1], sb + ak + (16 * kn + (mi >> 1) * 8 + l7) * C::kPitchA + (((2 * in + (mi & 1)) ^ asw) << 4));
            }
            const uint32_t *x = a4[it & 1];
            mma16816(s[2 * i], qh[2 * kk][0], qh[2 * kk][1], qh[2 * kk + 1][0], qh[2 * kk + 1][1], x[0], x[2]);
            mma16816(s[2 * i + 1], qh[2 * kk][0], qh[2 * kk][1], qh[2 * kk + 1][0], qh[2 * kk + 1][1], x[1], x[3]);
            mma16816(s[2 * i], ql[2 * kk][0], ql[2 * kk][1], ql[2 * kk + 1][0], ql[2 * kk + 1][1], x[0], x[2]);
            mma16816(s[2 * i + 1], ql[2 * kk][0], ql[2 * kk][1], ql[2 * kk + 1][0], ql[2 * kk + 1][1], x[1], x[3]);
        }
    }
    if (NT % 2) {
        uint32_t a2[2][2];
        ldsm_x2_t(a2[0], sb + ak + (8 * (NT - 1) + l7) * C::kPitchA + (((mi & 1) ^ asw) << 4));
#pragma unroll
        for (int i = 0; i < C::kMT; ++i) {
            if (i + 1 < C::kMT)
                ldsm_x2_t(a2[(i + 1) & 1], sb + ak + (8 * (NT - 1) + l7) * C::kPitchA + (((2 * (i + 1) + (mi & 1)) ^ asw) << 4));
            const uint32_t *x = a2[i & 1];
            mma1688(s[2 * i], qh[NT - 1][0], qh[NT - 1][1], x[0]);
            mma1688(s[2 * i + 1], qh[NT - 1][0], qh[NT - 1][1], x[1]);
            mma1688(s[2 * i], ql[NT - 1][0], ql[NT - 1][1], x[0]);
            mma1688(s[2 * i + 1], ql[NT - 1][0], ql[NT - 1][1], x[1]);
        }
    }
    uint32_t pa[NS / 2][4];
    row_softmax<NS>(s, st, pa);
    // ---- w [16][r] = p [16][P] . A_v ----
    uint32_t wa[NT][2];
    {
        float wt[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) wt[j][0] = wt[j][1] = wt[j][2] = wt[j][3] = 0.f;
        if (C::kMT >= 2) {
            // the score registers are free by now: all tiles of A_v are fetched before the first product
            uint32_t b[C::kMT / 2 > 0 ? C::kMT / 2 : 1][NT][4];
#pragma unroll
            for (int qd = 0; qd < C::kMT / 2; ++qd)
#pragma unroll
                for (int j = 0; j < NT; ++j) ldsm_x4(b[qd][j], sb + av + (8 * j + l7) * C::kPitchA + (((4 * qd + mi) ^ asw) << 4));
#pragma unroll
            for (int qd = 0; qd < C::kMT / 2; ++qd) {
#pragma unroll
                for (int j = 0; j < NT; ++j)
                    mma16816(wt[j], pa[2 * qd][0], pa[2 * qd][1], pa[2 * qd][2], pa[2 * qd][3], b[qd][j][0], b[qd][j][1]);
#pragma unroll
                for (int j = 0; j < NT; ++j)
                    mma16816(wt[j], pa[2 * qd + 1][0], pa[2 * qd + 1][1], pa[2 * qd + 1][2], pa[2 * qd + 1][3], b[qd][j][2], b[qd][j][3]);
            }
        }
        if (C::kMT % 2) {
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                uint32_t b[2];
                ldsm_x2(b, sb + av + (8 * j + l7) * C::kPitchA + (((2 * (C::kMT - 1) + (mi & 1)) ^ asw) << 4));
                mma16816(wt[j], pa[C::kMT - 1][0], pa[C::kMT - 1][1], pa[C::kMT - 1][2], pa[C::kMT - 1][3], b[0], b[1]);
            }
        }
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const bool v0 = 8 * j + t2 < rv, v1 = 8 * j + t2 + 1 < rv;
            wa[j][0] = pack_bf16(v0 ? wt[j][0] : 0.f, v1 ? wt[j][1] : 0.f);
            wa[j][1] = pack_bf16(v0 ? wt[j][2] : 0.f, v1 ? wt[j][3] : 0.f);
        }
    }
    // ---- o [16][d] += w . B_v ----
    if (NT >= 2) {
        // a4 = (ranks lo, channels 16i..), (ranks lo, 16i+8..), (ranks hi, 16i..), (ranks hi, 16i+8..); two items ahead
        constexpr int kItems = (NT / 2) * 8;
        uint32_t a4[3][4];
        ldsm_x4_t(a4[0], sb + bv + ((mi >> 1) * 8 + l7) * kRowBytes + (((mi & 1) ^ l7) << 4));
        ldsm_x4_t(a4[1], sb + bv + ((mi >> 1) * 8 + l7) * kRowBytes + (((2 + (mi & 1)) ^ l7) << 4));
#pragma unroll
        for (int it = 0; it < kItems; ++it) {
            const int kk = it / 8, i = it % 8;
            if (it + 2 < kItems) {
                const int kn = (it + 2) / 8, in = (it + 2) % 8;
                ldsm_x4_t(a4[(it + 2) % 3], sb + bv + (16 * kn + (mi >> 1) * 8 + l7) * kRowBytes + (((2 * in + (mi & 1)) ^ l7) << 4));
            }
            const uint32_t *x = a4[it % 3];
            mma16816(st.o[2 * i], wa[2 * kk][0], wa[2 * kk][1], wa[2 * kk + 1][0], wa[2 * kk + 1][1], x[0], x[2]);
            mma16816(st.o[2 * i + 1], wa[2 * kk][0], wa[2 * kk][1], wa[2 * kk + 1][0], wa[2 * kk + 1][1], x[1], x[3]);
        }
    }
    if (NT % 2) {
        uint32_t a2[3][2];
        ldsm_x2_t(a2[0], sb + bv + (8 * (NT - 1) + l7) * kRowBytes + (((mi & 1) ^ l7) << 4));
        ldsm_x2_t(a2[1], sb + bv + (8 * (NT - 1) + l7) * kRowBytes + (((2 + (mi & 1)) ^ l7) << 4));
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (i + 2 < 8)
                ldsm_x2_t(a2[(i + 2) % 3], sb + bv + (8 * (NT - 1) + l7) * kRowBytes + (((2 * (i + 2) + (mi & 1)) ^ l7) << 4));
            const uint32_t *x = a2[i % 3];
            mma1688(st.o[2 * i], wa[NT - 1][0], wa[NT - 1][1], x[0]);
            mma1688(st.o[2 * i + 1], wa[NT - 1][0], wa[NT - 1][1], x[1]);
        }
    }
}

// One block of DB rows of a dense page for 16 query rows; rows g / g+8 of the lane see the first lim0 / lim1 of
// the block's `rows` valid tokens.  Stale V rows past `rows` have been zeroed by the caller.
template <int DB>
__device__ __forceinline__ void block_dense_unit(uint32_t sb, int lim0, int lim1, const uint32_t (&qf)[8][4],
                                                 float scale, RowState &st, int lane) {
    constexpr int NI = DB / 16, NS = DB / 8;
    const int l7 = lane & 7, mi = lane >> 3, t2 = (lane & 3) * 2;
    float s[NS][4];
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        s[2 * i][0] = s[2 * i][1] = s[2 * i][2] = s[2 * i][3] = 0.f;
        s[2 * i + 1][0] = s[2 * i + 1][1] = s[2 * i + 1][2] = s[2 * i + 1][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            uint32_t a4[4];       // (tokens 16i.., channels lo), (tokens 16i+8.., lo), (16i.., hi), (16i+8.., hi)
            ldsm_x4(a4, sb + (16 * i + (mi & 1) * 8 + l7) * kRowBytes + (((2 * kk + (mi >> 1)) ^ l7) << 4));
            mma16816(s[2 * i], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], a4[0], a4[2]);
            mma16816(s[2 * i + 1], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], a4[1], a4[3]);
        }
    }
#pragma unroll
    for (int b = 0; b < NS; ++b) {
        const int tok = 8 * b + t2;
        s[b][0] = tok < lim0 ? s[b][0] * scale : kMasked;     s[b][1] = tok + 1 < lim0 ? s[b][1] * scale : kMasked;
        s[b][2] = tok < lim1 ? s[b][2] * scale : kMasked;     s[b][3] = tok + 1 < lim1 ? s[b][3] * scale : kMasked;
    }
    uint32_t pa[NI][4];
    row_softmax<NS>(s, st, pa);
#pragma unroll
    for (int i = 0; i < NI; ++i) {
#pragma unroll
        for (int ii = 0; ii < 8; ++ii) {
            uint32_t a4[4];       // (tokens lo, channels 16ii..), (tokens lo, 16ii+8..), (tokens hi, 16ii..), (tokens hi, 16ii+8..)
            ldsm_x4_t(a4, sb + DB * kRowBytes + (16 * i + (mi >> 1) * 8 + l7) * kRowBytes + (((2 * ii + (mi & 1)) ^ l7) << 4));
            mma16816(st.o[2 * ii], pa[i][0], pa[i][1], pa[i][2], pa[i][3], a4[0], a4[2]);
            mma16816(st.o[2 * ii + 1], pa[i][0], pa[i][1], pa[i][2], pa[i][3], a4[1], a4[3]);
        }
    }
}

#define PKV_BLOCK_BARRIER() asm volatile("bar.sync 2, %0;" ::"n"(kBlockWarps * 32) : "memory")

// Stages of the row-block kernel: as many as fit 100 KiB (two CTAs per SM), at least two, at most eight.
__host__ __device__ inline int block_stages(const Geometry &g) { return max(2, min(8, (100 * 1024) / g.stage_bytes)); }

template <int P, int NT>
__global__ void __launch_bounds__(kBlockThreads, 2) block_tc_kernel(const __grid_constant__ DecodeArgs a) {
    constexpr int kDB = kDenseBlock<P, NT, false>;
    const Geometry &geo = a.geo;
    const int S = block_stages(geo), H = geo.n_kv_heads, G = geo.group;
    const int n_rows = a.q_len * G, n_blk = (n_rows + kBlockRows - 1) / kBlockRows;
    // (the later a block's rows, the more of the sequence they see: the longest blocks of every head are started first,
    // so that what is left for the last wave of CTAs is the short ones)
    const int n_he = (int)gridDim.x / n_blk;              // (entry, head) pairs
    const int rb = n_blk - 1 - (int)blockIdx.x / n_he, head = ((int)blockIdx.x % n_he) % H, entry = ((int)blockIdx.x % n_he) / H;
    const PlanHeader hdr = *reinterpret_cast<const PlanHeader *>(a.plan);
    if (entry >= hdr.n_seqs) return;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *stages = smem;
    const int stage_bytes = geo.stage_bytes, blob_bytes = geo.blob_bytes;
    unsigned long long *full_bar = reinterpret_cast<unsigned long long *>(smem + (size_t)S * stage_bytes);
    unsigned long long *empty_bar = full_bar + S;
    StageDesc *descs = reinterpret_cast<StageDesc *>(empty_bar + S);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(descs + S);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(full_bar + s), 1); mbar_init(smem_u32(empty_bar + s), kBlockWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (stage_bytes > blob_bytes) {          // tails that 8-row tile loads read past a rank that is not a multiple of 8
        const int tail16 = (stage_bytes - blob_bytes) >> 4;
        for (int i = tid; i < S * tail16; i += kBlockThreads)
            reinterpret_cast<uint4 *>(stages + (size_t)(i / tail16) * stage_bytes + blob_bytes)[i % tail16] =
                make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const PlanEntry e = reinterpret_cast<const PlanEntry *>(a.plan + a.plan_entry)[entry];
    const HeadUnits hu = head_units(geo, e);
    const int T = a.n_tokens[(long long)e.seq * geo.n_layers + a.layer];
    // Units are in token order and the block's last row sees the most: units that start after what it sees are
    // hidden from every row of the block and are left out (producer and consumers agree on the count).
    int n_units = hu.units;
    {
        const int last_row = min(n_rows, (rb + 1) * kBlockRows) - 1;
        const int vis = T - (a.q_len - 1 - last_row / G);                 // tokens the last row sees (>= 1)
        const int page = (vis - 1) / P, blk = ((vis - 1) % P) / kDB;
        int need;
        if (page < hu.fb) need = page * geo.blocks_per_page + blk + 1;
        else if (page < hu.fe) need = hu.d0 + hu.nf;
        else need = hu.d0 + hu.nf + (page - hu.fe) * geo.blocks_per_page + blk + 1;
        n_units = max(1, min(need, hu.units));
    }

    if (warp == kBlockWarps) {
        // ------------------------------ producer (one lane) ------------------------------
        if (lane != 0) return;
        const int *pt = a.page_table + ((long long)e.seq * geo.n_layers + a.layer) * geo.max_pages;
        bool ok = true;
        int u = 0;
        // (stage and use count of a unit are counted along: the number of stages is not known at compile time)
        for (int s = 0, round = 0; u < n_units && ok; ++u, s = s + 1 == S ? 0 : s + 1, round += s == 0) {
            if (u >= S && !mbar_wait(smem_u32(empty_bar + s), (round - 1) & 1)) { ok = false; break; }
            int page, blk, kind;
            unit_to_page(geo, hu, u, page, blk, kind);
            const int slot = pt[page];
            int rows = 0, after = 0;
            const unsigned char *src = nullptr;
            if (slot < 0 || slot >= (kind == kKindFactor ? geo.n_factor_slots : geo.n_dense_slots)) {
                atomicAdd(a.status + 2, 1);                  // corrupt page table: skip the unit, leave a mark
                kind = kKindDense;
            } else if (kind == kKindFactor) {
                rows = P;
                src = a.factor_pool + (long long)slot * geo.factor_slot_bytes + (long long)head * geo.blob_bytes;
            } else {
                rows = max(0, min(kDB, T - page * P - blk * kDB));
                after = max(0, T - page * P - blk * kDB - rows);
                src = a.dense_pool + (long long)slot * geo.dense_slot_bytes + (long long)head * geo.dense_head_bytes +
                      blk * kDB * kRowBytes;
            }
            descs[s] = StageDesc{kind, rows, 0, after};
            const uint32_t bar = smem_u32(full_bar + s);
            const uint32_t dst = smem_u32(stages + (size_t)s * stage_bytes);
            if (kind == kKindFactor) {
                mbar_arrive_expect_tx(bar, blob_bytes);
                bulk_g2s_keep(dst, src, blob_bytes, bar);
            } else if (rows > 0) {
                mbar_arrive_expect_tx(bar, 2 * rows * kRowBytes);
                bulk_g2s_keep(dst, src, rows * kRowBytes, bar);
                bulk_g2s_keep(dst + kDB * kRowBytes, src + P * kRowBytes, rows * kRowBytes, bar);
            } else {
                mbar_arrive(bar);
            }
        }
        if (!ok) {
            *abort_flag = 1;
            atomicAdd(a.status, 1);
        }
        // copies already in flight must land before the CTA retires: wait (bounded) for the stages armed last
        for (int back = 1; back <= min(u, S); ++back) {
            const int k = u - back;
            (void)mbar_wait(smem_u32(full_bar + k % S), (k / S) & 1);
        }
        return;
    }
    // ------------------------------ consumers: 16 query rows per warp ------------------------------
    const int g8 = lane >> 2, t = lane & 3;
    const int row0 = rb * kBlockRows + warp * 16 + g8, row1 = row0 + 8;       // row = query token * G + query head
    const int j0 = row0 / G, j1 = row1 / G;
    const bool ok0 = row0 < n_rows, ok1 = row1 < n_rows;
    const long long qrow0 = ((long long)entry * a.q_len + j0) * geo.n_q_heads + head * G + row0 % G;
    const long long qrow1 = ((long long)entry * a.q_len + j1) * geo.n_q_heads + head * G + row1 % G;
    uint32_t qf[8][4];
    {
        const uint32_t *q0 = reinterpret_cast<const uint32_t *>(reinterpret_cast<const __nv_bfloat16 *>(a.q) + qrow0 * kHeadDim);
        const uint32_t *q1 = reinterpret_cast<const uint32_t *>(reinterpret_cast<const __nv_bfloat16 *>(a.q) + qrow1 * kHeadDim);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            qf[kk][0] = ok0 ? __ldg(q0 + 8 * kk + t) : 0u;
            qf[kk][1] = ok1 ? __ldg(q1 + 8 * kk + t) : 0u;
            qf[kk][2] = ok0 ? __ldg(q0 + 8 * kk + 4 + t) : 0u;
            qf[kk][3] = ok1 ? __ldg(q1 + 8 * kk + 4 + t) : 0u;
        }
    }
    // positions of the sequence's newest that rows g / g+8 must not see (rows past the end: none, result unused)
    const int hid0 = ok0 ? a.q_len - 1 - j0 : 0, hid1 = ok1 ? a.q_len - 1 - j1 : 0;
    RowState st;
#pragma unroll
    for (int c = 0; c < 16; ++c) st.o[c][0] = st.o[c][1] = st.o[c][2] = st.o[c][3] = 0.f;
    st.m[0] = st.m[1] = kNegInf;
    st.l[0] = st.l[1] = 0.f;
    bool ok = true;
    for (int u = 0, s = 0, round = 0; u < n_units; ++u, s = s + 1 == S ? 0 : s + 1, round += s == 0) {
        // The only way out is this warp's own wait running out: if the producer gave up, every warp ends up at the
        // same unarmed unit, so no warp is left alone at the block barrier below.
        if (!mbar_wait(smem_u32(full_bar + s), round & 1)) {
            ok = false;
            if (lane == 0) { *abort_flag = 1; atomicAdd(a.status, 1); }
            break;
        }
        const StageDesc dsc = descs[s];
        const int rows = min(dsc.rows, dsc.kind == kKindFactor ? P : kDB);
        if (rows > 0) {
            const uint32_t sb = smem_u32(stages + (size_t)s * stage_bytes);
            if (dsc.kind == kKindFactor) {
                block_factor_unit<P, NT>(sb, geo.ak_off, geo.bk_off, geo.av_off, geo.bv_off, geo.rank_k, geo.rank_v, qf,
                                         geo.scale_log2e, st, lane);
            } else {
                if (rows < kDB) {
                    // unfilled V rows hold stale bytes: zero them (each warp a share) before any warp reads V
                    uint4 *v = reinterpret_cast<uint4 *>(stages + (size_t)s * stage_bytes + kDB * kRowBytes + rows * kRowBytes);
                    for (int i = warp * 32 + lane; i < (kDB - rows) * 16; i += kBlockWarps * 32) v[i] = make_uint4(0u, 0u, 0u, 0u);
                    PKV_BLOCK_BARRIER();
                }
                const int lim0 = rows - max(0, hid0 - dsc.after), lim1 = rows - max(0, hid1 - dsc.after);
                block_dense_unit<kDB>(sb, lim0, lim1, qf, geo.scale_log2e, st, lane);
                if (rows < kDB) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(empty_bar + s));
    }
    if (!ok) return;
    float l0 = st.l[0], l1 = st.l[1];
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
    const float inv0 = 1.f / l0, inv1 = 1.f / l1;
    __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.out);
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        const int ch = 8 * c + 2 * t;
        if (ok0) {
            const float x = st.o[c][0] * inv0, y = st.o[c][1] * inv0;
            if (out) *reinterpret_cast<uint32_t *>(out + qrow0 * kHeadDim + ch) = pack_bf16(x, y);
            if (a.out_f32) *reinterpret_cast<float2 *>(a.out_f32 + qrow0 * kHeadDim + ch) = make_float2(x, y);
        }
        if (ok1) {
            const float x = st.o[c][2] * inv1, y = st.o[c][3] * inv1;
            if (out) *reinterpret_cast<uint32_t *>(out + qrow1 * kHeadDim + ch) = pack_bf16(x, y);
            if (a.out_f32) *reinterpret_cast<float2 *>(a.out_f32 + qrow1 * kHeadDim + ch) = make_float2(x, y);
        }
    }
}

size_t block_smem_bytes(const Geometry &g) {
    const int S = block_stages(g);
    return (size_t)S * g.stage_bytes + S * (8 + 8 + sizeof(StageDesc)) + 64;
}

template <int P, int NT>
cudaError_t launch_block(const DecodeArgs &a, int n_ctas, cudaStream_t st) {
    block_tc_kernel<P, NT><<<n_ctas, kBlockThreads, block_smem_bytes(a.geo), st>>>(a);
    return cudaGetLastError();
}

size_t decode_smem_bytes(const Geometry &g) {
    return (size_t)g.n_stages * g.stage_bytes + kConsumerWarps * kPartialFloats * 4 +
           g.n_stages * (8 + 8 + sizeof(StageDesc) + 4) + 64;
}

template <int P, int NT, int F>
cudaError_t launch_tc(const DecodeArgs &a, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.geo.n_ctas);
    cfg.blockDim = dim3(kDecodeThreads);
    cfg.dynamicSmemBytes = decode_smem_bytes(a.geo);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.plain_launch ? 0 : 1;
    return cudaLaunchKernelEx(&cfg, decode_tc_kernel<P, NT, F>, a);
}

template <int P, int NT>
cudaError_t setup_tc() {
    cudaError_t e = cudaFuncSetAttribute(decode_tc_kernel<P, NT, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget / 2);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(block_tc_kernel<P, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget / 2);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_tc_kernel<P, NT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget / 2);
}

// the Global SVD form: P in {32, 64}, ranks 64, 80, 96
#define PKV_FOR_EACH_GLOBAL_SHAPE(X) X(32, 8) X(32, 10) X(32, 12) X(64, 8) X(64, 10) X(64, 12)

// the instantiated shapes: P in {16, 32, 64}, rank tiles 1..4 (1..2 for P = 16)
#define PKV_FOR_EACH_SHAPE(X) \
    X(16, 1) X(16, 2) X(32, 1) X(32, 2) X(32, 3) X(32, 4) X(64, 1) X(64, 2) X(64, 3) X(64, 4)

}  // namespace

cudaError_t decode_kernel_setup() {
    cudaError_t e;
#define PKV_SETUP(P, NT) if ((e = setup_tc<P, NT>()) != cudaSuccess) return e;
    PKV_FOR_EACH_SHAPE(PKV_SETUP)
#undef PKV_SETUP
#define PKV_SETUP_G(P, NT) \
    if ((e = cudaFuncSetAttribute(decode_tc_kernel<P, NT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget / 2)) != cudaSuccess) return e;
    PKV_FOR_EACH_GLOBAL_SHAPE(PKV_SETUP_G)
#undef PKV_SETUP_G
    return row_block_umma_setup();
}

cudaError_t launch_decode(const DecodeArgs &a, int n_segs, cudaStream_t st) {
    cudaError_t e = cudaErrorInvalidValue;
    if (a.variant == 1) {
        decode_scalar_kernel<<<a.geo.n_ctas, 128, 0, st>>>(a);
        e = cudaGetLastError();
    } else {
        if (a.geo.global_rank > 0) {
#define PKV_LAUNCH_G(P, NT) if (a.geo.page == P && a.geo.rank_tiles == NT) e = launch_tc<P, NT, 2>(a, st);
            PKV_FOR_EACH_GLOBAL_SHAPE(PKV_LAUNCH_G)
#undef PKV_LAUNCH_G
        } else {
#define PKV_LAUNCH(P, NT) if (a.geo.page == P && a.geo.rank_tiles == NT) \
            e = a.geo.factor_bits == 4 ? launch_tc<P, NT, 1>(a, st) : launch_tc<P, NT, 0>(a, st);
            PKV_FOR_EACH_SHAPE(PKV_LAUNCH)
#undef PKV_LAUNCH
        }
    }
    if (e != cudaSuccess || a.variant != 1) return e;
    merge_kernel<<<n_segs, 256, 0, st>>>(a);
    return cudaGetLastError();
}

// Row-block kernels; bf16 factors only.  Shapes the tcgen05 kernel covers go to it (one CTA per 128 query rows of a
// (sequence, KV head)) unless the caller pinned the mma.sync kernel (decode_variant 3); the rest to the latter (one
// CTA per 64 rows).
cudaError_t launch_decode_blocks(const DecodeArgs &a, int n_seqs, const RowBlockMaps &maps, cudaStream_t st) {
    if (a.variant != 3 && maps.valid) return launch_decode_blocks_umma(a, n_seqs, maps, st);
    const int n_blk = (a.q_len * a.geo.group + kBlockRows - 1) / kBlockRows;
    const long long n_ctas = (long long)n_seqs * a.geo.n_kv_heads * n_blk;
    if (a.geo.factor_bits == 4 || n_ctas <= 0 || n_ctas > 0x7fffffffLL) return cudaErrorInvalidValue;
    cudaError_t e = cudaErrorInvalidValue;
#define PKV_LAUNCH_BLOCK(P, NT) if (a.geo.page == P && a.geo.rank_tiles == NT) e = launch_block<P, NT>(a, (int)n_ctas, st);
    PKV_FOR_EACH_SHAPE(PKV_LAUNCH_BLOCK)
#undef PKV_LAUNCH_BLOCK
    return e;
}

// Eq. 5 across caches: states [n_shards][n_rows][d + 2] as written by store_out; one warp per row.
__global__ void __launch_bounds__(128) merge_states_kernel(const float *states, int n_shards, long long n_rows,
                                                           __nv_bfloat16 *out, float *out_f32) {
    const long long row = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    const int d4 = (threadIdx.x & 31) * 4;
    const long long stride = n_rows * (kHeadDim + 2);
    const float *base = states + row * (kHeadDim + 2);
    float M = kNegInf;
    for (int k = 0; k < n_shards; ++k) M = fmaxf(M, base[k * stride + kHeadDim]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    for (int k = 0; k < n_shards; ++k) {                    // shard order: the result does not depend on who merges
        const float *pk = base + k * stride;
        const float w = exp2f(pk[kHeadDim] - M);
        const float2 a0 = *reinterpret_cast<const float2 *>(pk + d4), a1 = *reinterpret_cast<const float2 *>(pk + d4 + 2);
        acc.x += w * a0.x; acc.y += w * a0.y; acc.z += w * a1.x; acc.w += w * a1.y;
        L += w * pk[kHeadDim + 1];
    }
    const float inv = 1.f / L;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    const long long off = row * kHeadDim + d4;
    if (out) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 packed;
        packed.x = *reinterpret_cast<unsigned *>(&lo);
        packed.y = *reinterpret_cast<unsigned *>(&hi);
        *reinterpret_cast<uint2 *>(out + off) = packed;
    }
    if (out_f32) *reinterpret_cast<float4 *>(out_f32 + off) = acc;
}

cudaError_t launch_merge_states(const float *states, int n_shards, long long n_rows, void *out, float *out_f32,
                                cudaStream_t st) {
    if (n_rows <= 0) return cudaSuccess;
    merge_states_kernel<<<(unsigned)((n_rows + 3) / 4), 128, 0, st>>>(states, n_shards, n_rows,
                                                                      reinterpret_cast<__nv_bfloat16 *>(out), out_f32);
    return cudaGetLastError();
}

// Same launch as launch_decode(), with the partial states and tickets in g_static_scratch instead of
// the caller's workspace.  In host code the array's name is only a stand-in for the device symbol, so
// its device address is looked up (once per device, with that device current) and handed to the kernel.
cudaError_t launch_decode_static_scratch(const DecodeArgs &a, int n_segs, cudaStream_t st, const char **why) {
    static unsigned char *scratch_of_device[64] = {};
    *why = "";
    // per-CTA states, then the states of groups of CTAs; tickets per segment, then per group
    const long long n_flat = (long long)a.geo.n_ctas + n_segs, n_group = merge_group_slots(n_flat, n_segs);
    if (n_flat + n_group > kStaticPartialStates || n_segs + n_group > kStaticTickets) {
        *why = "call needs more split-K partial states than the static scratch holds "
               "(F + F / 8 + S + 2 must be <= 1024, with S = n_seqs * n_kv_heads and F = n_ctas + S)";
        return cudaErrorInvalidValue;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { *why = "cudaGetDevice failed"; return e; }
    if (dev < 0 || dev >= 64) { *why = "device ordinal above 63"; return cudaErrorInvalidDevice; }
    if (!scratch_of_device[dev]) {
        unsigned char *p = nullptr;
        e = cudaGetSymbolAddress((void **)&p, g_static_scratch);
        if (e != cudaSuccess || !p) { *why = "cudaGetSymbolAddress(g_static_scratch) failed"; return e != cudaSuccess ? e : cudaErrorUnknown; }
        scratch_of_device[dev] = p;
    }
    unsigned char *base = scratch_of_device[dev];
    DecodeArgs b = a;
    b.partials = reinterpret_cast<float *>(base);
    b.tickets = reinterpret_cast<int *>(base + kStaticTicketOffset);
    b.gpartials = b.partials + n_flat * kPartialFloats;
    b.gtickets = b.tickets + n_segs;
    // the array keeps whatever the previous call (or an aborted one) left: tickets must start at zero
    e = cudaMemsetAsync(b.tickets, 0, (size_t)(n_segs + n_group) * sizeof(int), st);
    if (e != cudaSuccess) { *why = "clearing the tickets failed"; return e; }
    e = launch_decode(b, n_segs, st);
    if (e != cudaSuccess) *why = "kernel launch failed";
    return e;
}

}  // namespace pkv
