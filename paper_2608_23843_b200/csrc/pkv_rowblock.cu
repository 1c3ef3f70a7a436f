// Row-block attention on the fifth-generation tensor cores (tcgen05.mma, accumulators and row operands in tensor
// memory).
//
// Same job as the mma.sync row-block kernel of pkv_decode.cu — many queries per sequence (a chunk of a prefill), a
// CTA per (sequence, KV head, block of query rows), Eq. 4 for factor pages and plain attention for dense ones, the
// pages in token order — but with 128 query rows per CTA as the M dimension of every product (and, where the row
// blocks alone would not fill the GPU, several CTAs per block with a range of the sequence each, whose softmax
// states rowblock_merge_kernel combines; pages of 32 tokens with ranks up to 16 are taken two to a unit):
//     G1: q~ [128 x r] = Q [128 x d] . B_k^T        G2: s [128 x P] = (q~_hi + q~_lo) . A_k^T
//     G3: w  [128 x r] = p [128 x P] . A_v          G4: o [128 x d] += w . B_v
//     dense pages:  Ga: s = Q . K^T                 Gb: o += p . V
// One thread owns one query row (= one lane of tensor memory): it reads its row of q~, s, w back from tensor memory,
// does the scaling, the two-term bf16 split, the masking and the online softmax alone (no shuffles), and writes the
// row of the next product's A operand over the columns it has just read (tcgen05.mma takes A from tensor memory).
// A^T factors are used where the bulk copy put them: the storage swizzle of an A^T row of 128, 64 or 32 bytes (P =
// 64, 32, 16) is the tensor core's swizzle for rows of that length (A_k^T as an MN-major B operand, A_v^T as a K-major
// one).  Rows of 256 bytes (B factors, dense K / V) arrive as two panels of 128-byte rows (tiled TMA copies, 64
// channels each), which is the 128-byte swizzle again.
//
// Warps 0-3: the 128 query rows.  Warp 4, one lane: copies into the ring.  Warp 5, one lane: issues every
// tcgen05.mma.  The four products of a factor page depend on one another through the row threads; the schedule
// keeps the row threads waiting for as few of them as it can.  Per unit u the rows hand over three times (an
// mbarrier of 128 arrivals each) and the issuer answers with tcgen05.commit on three mbarriers:
//     rows: wait "S"; softmax of s(u) -> p(u)               hand-over A -> issuer: G3(u) | Gb(u); commit "G3"
//     rows: wait "Q"; q~(u+1) to two bf16 terms             hand-over B -> issuer: G2(u+1) | Ga(u+1); commit "S";
//                                                                          first half of G1(u+2)
//     rows: wait "G3"; w(u) to bf16                         hand-over C -> issuer: G4(u); second half of G1(u+2); commit "Q"
// so the conversion of q~(u+1) runs while G3(u) does, s(u+1) is being computed while w(u) is converted, and G4 and
// G1 are off the rows' path: their commit is met one hand-over later, when it has long arrived (earlier only if o
// has to be rescaled).  The issuing lane also waits for each unit's copies and passes the unit's descriptor on to
// the row threads ahead of commit "Q".  Two CTAs per SM overlap one another's remaining waits; the blocks of a
// launch are taken longest first.  Every wait is bounded; tensor memory is released on every path out.
#include "pkv_device.cuh"

namespace pkv {

namespace {

constexpr int kURows = 128;
constexpr int kUThreads = 192;
constexpr int kUQBytes = 2 * kURows * 128;       // Q: two panels [128 rows][64 channels], 128-byte swizzle
constexpr uint32_t kColQt = 0, kColS = 32, kColW = 96, kColO = 128, kTmemCols = 256;

// A stage holds one unit the way the products read it, in parts of 128-byte rows (see StageLayout).  K side = B_k or
// a block of dense K, V side = B_v or a block of dense V; a side is two panels of 64 channels, written by tiled TMA
// copies (box = 64 channels x rows) straight from the pools' 256-byte rows: 16-byte chunk c of row j is stored at
// chunk c ^ (j & 7), so each half of a row is a 128-byte row in the tensor core's 128-byte swizzle.
// Pages of 32 or 16 tokens with ranks up to 16 are taken two to a unit: page j's B rows start
// at row 16 j of panels of 32 rows, so that q~ and w of the pair are one row of 32 columns and the products with the
// B factors are the same instructions as for a rank of 32; the products with the A factors are issued per page.
__host__ __device__ inline bool umma_pair(const Geometry &g) { return g.page <= 32 && g.rank_tiles <= 2; }
// Rows of a dense block: a whole page, or half a page of 64 tokens
__host__ __device__ inline int umma_part_rows(const Geometry &g) { return g.page < 32 ? g.page : 32; }
// Bytes kept free behind the last stage: a product that reads a rank padded to 16 or 32 rows may run past the last
// part of a stage (a pair's panels hold exactly the rows its products read).
__host__ __device__ inline int umma_stage_pad(const Geometry &g) { return umma_pair(g) ? 0 : 1024; }
// bytes of an A^T part of a stage: rows of 2 P bytes, the rank rounded up to 8 rows, the part to 1024 bytes (the parts
// behind it hold 128-byte-swizzled panels, whose pattern repeats every 1024 bytes)
__host__ __device__ inline int umma_a_bytes(const Geometry &g, int rank) { return ((((rank + 7) & ~7) * 2 * g.page) + 1023) & ~1023; }
__host__ __device__ inline int umma_stage_bytes(const Geometry &g) {
    const int factor = umma_pair(g) ? 2 * (umma_a_bytes(g, g.rank_k) + umma_a_bytes(g, g.rank_v)) + 4 * 32 * 128
                                    : umma_a_bytes(g, g.rank_k) + umma_a_bytes(g, g.rank_v) + 2 * 128 * (((g.rank_k + 7) & ~7) + ((g.rank_v + 7) & ~7));
    const int dense = 4 * umma_part_rows(g) * 128;
    return ((factor > dense ? factor : dense) + 1023) & ~1023;
}
// stages: the units u, u + 1 and u + 2 are in use at any time; the rest is the copies' lead
__host__ __device__ inline int umma_stages(const Geometry &g) {
    const int room = 113 * 1024 - kUQBytes - umma_stage_pad(g) - 512;
    return max(3, min(6, room / umma_stage_bytes(g)));
}

// ---- tcgen05 wrappers --------------------------------------------------------------------------------------
// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all in 16-byte units), descriptor
// version 1, layout 0 = no swizzle, 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo, uint32_t layout) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (uint64_t)((lbo >> 4) & 0x3FFF) << 16 | (uint64_t)((sbo >> 4) & 0x3FFF) << 32 |
           (uint64_t)1 << 46 | (uint64_t)layout << 61;
}
// The same descriptor `bytes` further on (a multiple of 16; the start-address field, in 16-byte units, is the lowest
// field and the sum stays inside the 256 KB the field covers): one 32-bit add on the low word.
__device__ __forceinline__ uint64_t umma_desc_step(uint64_t desc, uint32_t bytes) {
    uint32_t lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(desc));
    lo += bytes >> 4;
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M x N, B operand K-major (0) or MN-major (1); A always K-major.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// d (+)= a . b with a in shared memory / in tensor memory (row = lane, two bf16 per 32-bit column, 8 columns per
// step of 16 along the contraction)
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Tiled copy of one box (64 channels x the map's rows) starting at channel x of pool row y; completes on `bar`.
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

#define PKV_R8(r, o) "=r"(r[o]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define PKV_W8(r, o) "r"(r[o]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])
// consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t *r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : PKV_R8(r, 0), PKV_R8(r, 8), PKV_R8(r, 16), PKV_R8(r, 24) : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t *r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : PKV_R8(r, 0), PKV_R8(r, 8) : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t *r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), PKV_W8(r, 0), PKV_W8(r, 8), PKV_W8(r, 16), PKV_W8(r, 24) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t *r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), PKV_W8(r, 0), PKV_W8(r, 8) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t *r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), PKV_W8(r, 0) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tmem_ld_nowait(uint32_t taddr, uint32_t *r) {
    static_assert(N == 16 || N == 32, "16 or 32 columns");
    if (N == 16) tmem_ld16(taddr, r);
    else tmem_ld32(taddr, r);
}
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t *r) {
    static_assert(N == 16 || N == 32 || N == 64, "16, 32 or 64 columns");
    if (N == 16) tmem_ld16(taddr, r);
    else { tmem_ld32(taddr, r); if (N == 64) tmem_ld32(taddr + 32, r + 32); }
    tmem_ld_wait();
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t *r) {
    static_assert(N == 8 || N == 16 || N == 32, "8, 16 or 32 columns");
    if (N == 8) tmem_st8(taddr, r);
    else if (N == 16) tmem_st16(taddr, r);
    else tmem_st32(taddr, r);
}
// True in exactly one lane of a converged warp.  The single-lane roles are entered through this rather than through
// `lane == 0`: the compiler then knows that one lane runs the code, and issues tcgen05.mma (whose operands are
// warp-uniform registers) directly; behind a plain lane test each issue measured 230 clocks instead of 40.
__device__ __forceinline__ bool elect_one() {
    uint32_t leader;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
    return leader != 0;
}
// 2^x for x <= 0 (and the large negative stand-ins for -inf, which give 0)
__device__ __forceinline__ float exp2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Bounded waits.  One lane (producer, issuer): gives up when the clock limit passes or another role has given up.
__device__ __forceinline__ bool wait_lane(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit || *abort_flag) return false;
    }
    return true;
}
// A whole warp (the row threads run warp-collective tensor-memory loads right after): the outcome is the same for
// all 32 lanes.
__device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit) {
    if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
    const long long t0 = clock64();
    for (;;) {
        if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        if (__any_sync(0xffffffffu, clock64() - t0 > limit || *abort_flag)) return false;
    }
}

// Softmax state of this thread's row.  p and l are always taken against the true running maximum m, so the largest
// weight is exactly 1 and its bf16 rounding costs nothing.  o, which lives in tensor memory, is kept against an
// older maximum m_ref <= m instead of being rescaled every time m grows: a factor page's contribution enters o
// through w, an fp32 row that this thread rounds to bf16 itself, so it multiplies w by 2^(m - m_ref) first - the
// rounding is relative and does not care.  o is rescaled for real only when that factor would pass 2^kFrameLag, or
// before a dense block, whose p goes to the product as it is.
struct RowSoftmax {
    float m, l, m_ref;
};
constexpr float kFrameLag = 8.f;

// Byte offsets of a unit's parts inside its stage.  A factor unit is
//     [A_k^T: r_k rows of 2 P bytes][K side: 2 panels of r_k rows][A_v^T: r_v rows][V side: 2 panels of r_v rows]    (panels: 128-byte rows)
// with every part rounded up to a multiple of 8 rows, so a product that reads a rank padded to 16 or 32 rows reads
// rows no copy of this unit wrote (what an earlier unit left there, or the zeros of the start) and runs into the
// next part: finite data either way, multiplied by exact zeros (or producing columns that are replaced by exact
// zeros).  A dense unit is [K side: 2 x RB rows][V side: 2 x RB rows].
struct StageLayout {
    int ak, k, k_panel, av, v, v_panel;         // factor units
    int dk, dv, d_panel;                        // dense units
};
__host__ __device__ inline StageLayout umma_layout(const Geometry &g) {
    StageLayout L;
    const int rk = (g.rank_k + 7) & ~7, rv = (g.rank_v + 7) & ~7;        // parts start on 1024-byte boundaries
    L.ak = 0; L.k = umma_a_bytes(g, g.rank_k); L.k_panel = rk * 128;
    L.av = L.k + 2 * rk * 128; L.v = L.av + umma_a_bytes(g, g.rank_v); L.v_panel = rv * 128;
    if (umma_pair(g)) {          // [A_k^T x 2][K side: 2 panels of 32 rows][A_v^T x 2][V side: 2 panels of 32 rows]
        L.k = 2 * umma_a_bytes(g, g.rank_k); L.k_panel = 32 * 128;
        L.av = L.k + 2 * L.k_panel; L.v = L.av + 2 * umma_a_bytes(g, g.rank_v); L.v_panel = 32 * 128;
    }
    L.d_panel = umma_part_rows(g) * 128; L.dk = 0; L.dv = 2 * L.d_panel;
    return L;
}

// Two fp32 values in one 64-bit register, and the sm_100 instructions that work on both halves at once: the row
// threads' arithmetic is issue-bound (two row warps per scheduler), so halving the instruction count of the
// subtractions, sums and scalings shows.  Likewise the three-input maximum.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// RP fp32 values x (a row of q~ or w) times `scale`, as bf16 pairs; columns from `rank` on become exact zeros.  The
// kExact: the rank is KNOWN, a compile-time value (the ranks fill their tiles); otherwise KNOWN = RP and every column is
// tested against `rank`.
// (kHalves: the row is two ranks of 16 columns side by side - a pair of pages -, each with its own pad columns)
template <int RP, int KNOWN, bool kExact, bool kHalves = false>
__device__ __forceinline__ void scale_pack(const uint32_t *x, uint32_t *pk, float scale, int rank) {
    const uint64_t sc2 = f2_pack(scale, scale);
    constexpr int kMask = kHalves ? 15 : ~0;
#pragma unroll
    for (int k = 0; k < RP / 2; ++k) {
        if (kExact && ((2 * k + 1) & kMask) < KNOWN) {    // this pair lies below the rank
            float y0, y1;
            f2_unpack(f2_mul(f2_pack(__uint_as_float(x[2 * k]), __uint_as_float(x[2 * k + 1])), sc2), y0, y1);
            pk[k] = pack_bf16(y0, y1);
            continue;
        }
        const bool in0 = ((2 * k) & kMask) < KNOWN && ((2 * k) & kMask) < rank, in1 = ((2 * k + 1) & kMask) < KNOWN && ((2 * k + 1) & kMask) < rank;
        pk[k] = pack_bf16(in0 ? __uint_as_float(x[2 * k]) * scale : 0.f, in1 ? __uint_as_float(x[2 * k + 1]) * scale : 0.f);
    }
}
// The same with the rounding error of each pair as a second bf16 term (hi + lo carries about 16 bits).
template <int RP, int KNOWN, bool kExact, bool kHalves = false>
__device__ __forceinline__ void split_terms(const uint32_t *x, uint32_t *hi, uint32_t *lo, float scale, int rank) {
    const uint64_t sc2 = f2_pack(scale, scale);
    constexpr int kMask = kHalves ? 15 : ~0;
#pragma unroll
    for (int k = 0; k < RP / 2; ++k) {
        if (kExact && ((2 * k + 1) & kMask) < KNOWN) {    // this pair lies below the rank
            const uint64_t y = f2_mul(f2_pack(__uint_as_float(x[2 * k]), __uint_as_float(x[2 * k + 1])), sc2);
            float y0, y1, e0, e1;
            f2_unpack(y, y0, y1);
            hi[k] = pack_bf16(y0, y1);
            f2_unpack(f2_sub(y, f2_pack(bf16lo_f(hi[k]), bf16hi_f(hi[k]))), e0, e1);
            lo[k] = pack_bf16(e0, e1);
            continue;
        }
        const bool in0 = ((2 * k) & kMask) < KNOWN && ((2 * k) & kMask) < rank, in1 = ((2 * k + 1) & kMask) < KNOWN && ((2 * k + 1) & kMask) < rank;
        const float x0 = in0 ? __uint_as_float(x[2 * k]) * scale : 0.f, x1 = in1 ? __uint_as_float(x[2 * k + 1]) * scale : 0.f;
        hi[k] = pack_bf16(x0, x1);
        lo[k] = pack_bf16(x0 - bf16lo_f(hi[k]), x1 - bf16hi_f(hi[k]));
    }
}

// Online softmax of one row over N scores held in sv (already scaled and masked): updates (m, l), brings o to a
// frame it may stay in (see RowSoftmax) - which, when some row of the warp needs it, means waiting (once per unit:
// o_seen) for the product of the unit before that adds to o and rescaling o in tensor memory - and writes p as bf16
// pairs over the first N / 2 columns the scores were read from.  o_valid: some product has already written o.
// False if the wait ran out.
template <int N, bool kDense>
__device__ __forceinline__ bool softmax_row(float *sv, RowSoftmax &st, bool o_valid, uint32_t t_s, uint32_t t_o, uint32_t bar_Q,
                                            uint32_t &ph_Q, bool &o_seen, volatile int *abort_flag, long long limit) {
    float mx4[4] = {sv[0], sv[1], sv[2], sv[3]};           // four chains: a thread has no other work to hide latencies with
#pragma unroll
    for (int i = 4; i + 8 <= N; i += 8)
#pragma unroll
        for (int c = 0; c < 4; ++c) mx4[c] = max3(mx4[c], sv[i + c], sv[i + 4 + c]);
#pragma unroll
    for (int i = 4 + ((N - 4) / 8) * 8; i < N; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], sv[i]);
    const float mx = fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]);
    if (mx > st.m) { st.l *= exp2_fast(st.m - mx); st.m = mx; }
    if (!o_valid) {
        st.m_ref = st.m;
    } else if (__any_sync(0xffffffffu, kDense ? st.m != st.m_ref : st.m - st.m_ref > kFrameLag)) {
        if (!o_seen) {
            if (!wait_warp(bar_Q, ph_Q, abort_flag, limit)) return false;
            ph_Q ^= 1;
            o_seen = true;
            tc_fence_after();
        }
        const float f = exp2_fast(st.m_ref - st.m);
        st.m_ref = st.m;
        uint32_t r[32];
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            tmem_ld32(t_o + 32 * c, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
            tmem_st32(t_o + 32 * c, r);
        }
    }
    uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};         // (0.f, 0.f) each
    const uint64_t m2 = f2_pack(st.m, st.m);
    uint32_t pk[N / 2];
#pragma unroll
    for (int e = 0; e < N / 2; ++e) {
        float d0, d1;
        f2_unpack(f2_sub(f2_pack(sv[2 * e], sv[2 * e + 1]), m2), d0, d1);
        const float p0 = exp2_fast(d0), p1 = exp2_fast(d1);
        sum2[e & 3] = f2_add(sum2[e & 3], f2_pack(p0, p1));
        pk[e] = pack_bf16(p0, p1);
    }
    tmem_st<N / 2>(t_s, pk);
    tmem_st_wait();
    float s0, s1;
    f2_unpack(f2_add(f2_add(sum2[0], sum2[1]), f2_add(sum2[2], sum2[3])), s0, s1);
    st.l += s0 + s1;
    return true;
}

template <int P, int NT>
__global__ void __launch_bounds__(kUThreads, 2) block_umma_kernel(const __grid_constant__ DecodeArgs a,
                                                                  const __grid_constant__ RowBlockMaps maps) {
    // RP1: what a page's rank is padded to; RP: columns of q~ and w of a factor unit; PU: tokens of a factor unit
    // (kPair: two pages, see umma_pair()); kDB: rows of a dense block; bpp: blocks of a dense page
    constexpr bool kPair = P <= 32 && NT <= 2;
    constexpr int RP1 = NT <= 2 ? 16 : 32, RP = kPair ? 32 : RP1, PU = kPair ? 2 * P : P;
    constexpr int kDB = P < 32 ? P : 32, bpp = P / kDB;
    // A^T rows are 2 P bytes: the 128-byte swizzle for P = 64, the 64-byte one (8 rows = 512 bytes) for P = 32, the
    // 32-byte one for P = 16 - each time the XOR the pages are stored with
    constexpr uint32_t kASwizzle = P == 64 ? 2 : (P == 32 ? 4 : 6), kAGroup = 8 * 2 * P;
    static_assert(kDB <= 32 && RP <= 32, "a dense block's scores and a unit's q~ fit their columns of tensor memory");
    const Geometry &geo = a.geo;
    const StageLayout L = umma_layout(geo);
    const int S = umma_stages(geo), ustage = umma_stage_bytes(geo), H = geo.n_kv_heads, G = geo.group;
    const int n_rows = a.q_len * G, n_blk = (n_rows + kURows - 1) / kURows;
    // (the later a block's rows, the more of the sequence they see: the longest blocks of every head are started first,
    // so that what is left for the last wave of CTAs is the short ones)
    // With a.rb_splits = ns > 1 (few row blocks, long sequences) ns consecutive CTAs share a row block, each with its own
    // range of the block's units; they leave softmax states which rowblock_merge_kernel combines (Eq. 5).
    const int ns = a.rb_splits, blk_id = (int)blockIdx.x / ns, split = (int)blockIdx.x - blk_id * ns;
    const int n_he = (int)gridDim.x / ns / n_blk;         // (entry, head) pairs
    const int rb = n_blk - 1 - blk_id / n_he, head = (blk_id % n_he) % H, entry = (blk_id % n_he) / H;
    const PlanHeader hdr = *reinterpret_cast<const PlanHeader *>(a.plan);
    if (entry >= hdr.n_seqs) return;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sq = smem, *stages = smem + kUQBytes;
    // (one more KiB behind the last stage: a padded product of the last stage's last part reads it)
    const int stage_pad = umma_stage_pad(geo);
    unsigned long long *full_bar = reinterpret_cast<unsigned long long *>(stages + (size_t)S * ustage + stage_pad);
    unsigned long long *empty_bar = full_bar + S;
    unsigned long long *bars = empty_bar + S;          // rows -> issuer: A, B, C; issuer -> rows: G3, S, Q; drain
    StageDesc *descs = reinterpret_cast<StageDesc *>(bars + 8);
    StageDesc *info = descs + S;                       // [2]: the descriptor of a unit as the issuing lane read it, for the row threads
    volatile int *abort_flag = reinterpret_cast<volatile int *>(info + 2);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(const_cast<int *>(abort_flag) + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bar_A = smem_u32(bars + 0), bar_B = smem_u32(bars + 1), bar_C = smem_u32(bars + 2);
    const uint32_t bar_G3 = smem_u32(bars + 3), bar_S = smem_u32(bars + 4), bar_Q = smem_u32(bars + 5);
    const uint32_t bar_drain = smem_u32(bars + 6);
    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(full_bar + s), 1); mbar_init(smem_u32(empty_bar + s), 1); }
        mbar_init(bar_A, kURows); mbar_init(bar_B, kURows); mbar_init(bar_C, kURows);
        mbar_init(bar_G3, 1); mbar_init(bar_S, 1); mbar_init(bar_Q, 1); mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // What a padded product reads past a unit's own rows must be finite from the start.
    for (int i = tid; i < (S * ustage + stage_pad) / 16; i += kUThreads) reinterpret_cast<uint4 *>(stages)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_async_smem();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = *tmem_slot;
    const PlanEntry e = reinterpret_cast<const PlanEntry *>(a.plan + a.plan_entry)[entry];
    HeadUnits hu = head_units(geo, e);
    // this kernel's own units: dense pages in blocks of kDB rows; kPair: factor pages two to a unit (the last unit of an
    // odd number holds one)
    hu.d0 = hu.fb * bpp;
    if (kPair) hu.nf = (hu.nf + 1) >> 1;
    hu.units = hu.d0 + hu.nf + (e.n_pages - hu.fe) * bpp;
    const int T = a.n_tokens[(long long)e.seq * geo.n_layers + a.layer];
    // Units are in token order and the block's last row sees the most: units that start after what it sees are
    // hidden from every row of the block and are left out (all roles agree on the count).
    int n_units = hu.units;
    {
        const int last_row = min(n_rows, (rb + 1) * kURows) - 1;
        const int vis = T - (a.q_len - 1 - last_row / G);                 // tokens the last row sees (>= 1)
        const int page = (vis - 1) / P, blk = ((vis - 1) % P) / kDB;
        int need;
        if (page < hu.fb) need = page * bpp + blk + 1;
        else if (page < hu.fe) need = hu.d0 + hu.nf;
        else need = hu.d0 + hu.nf + (page - hu.fe) * bpp + blk + 1;
        n_units = max(1, min(need, hu.units));
    }
    int u_base = 0;                                       // first unit of this CTA's range
    if (ns > 1) {
        u_base = (int)((long long)n_units * split / ns);
        n_units = (int)((long long)n_units * (split + 1) / ns) - u_base;          // may be 0: a state without weight
    }
    const long long limit = a.wait_clocks;

    if (warp == 4) {
        // ------------------------------ copies (one lane) ------------------------------
        if (elect_one()) {
            const int *pt = a.page_table + ((long long)e.seq * geo.n_layers + a.layer) * geo.max_pages;
            bool ok = true;
            int u = 0;
            // (stage and use count of a unit are counted along: S is not known at compile time and a division per
            // unit is a hundred clocks of a single thread)
            for (int s = 0, round = 0; u < n_units; ++u, s = s + 1 == S ? 0 : s + 1, round += s == 0) {
                if (u >= S && !wait_lane(smem_u32(empty_bar + s), (round - 1) & 1, abort_flag, limit)) { ok = false; break; }
                int page, blk, kind;
                unit_to_page(bpp, hu, u_base + u, page, blk, kind);
                if (kPair && kind == kKindFactor) page = hu.fb + 2 * (page - hu.fb);
                const int slot = pt[page];
                const int n_pg = kPair && kind == kKindFactor && page + 1 < hu.fe ? 2 : 1;          // pages of this unit
                const int slot2 = n_pg == 2 ? pt[page + 1] : 0;
                int rows = 0, after = 0;
                const bool bad = slot < 0 || slot >= (kind == kKindFactor ? geo.n_factor_slots : geo.n_dense_slots) ||
                                 slot2 < 0 || slot2 >= geo.n_factor_slots;
                if (bad) {
                    atomicAdd(a.status + 2, 1);                  // corrupt page table: an empty unit, and a mark
                    kind = kKindDense;
                } else if (kind == kKindFactor) {
                    rows = P * n_pg;
                } else {
                    rows = max(0, min(kDB, T - page * P - blk * kDB));
                    after = max(0, T - page * P - blk * kDB - rows);
                }
                if (a.drop_unit == u && blockIdx.x == 0) continue;          // test hook: the unit is never armed, a wait must run out
                descs[s] = StageDesc{kind, rows, 0, after};
                const uint32_t bar = smem_u32(full_bar + s);
                const uint32_t dst = smem_u32(stages + (size_t)s * ustage);
                if (kind == kKindFactor) {
                    mbar_arrive_expect_tx(bar, geo.blob_bytes * n_pg);
                    for (int j = 0; j < n_pg; ++j) {
                        const long long off = (long long)(j ? slot2 : slot) * geo.factor_slot_bytes + (long long)head * geo.blob_bytes;
                        const unsigned char *src = a.factor_pool + off;
                        // B_k, B_v as rows of the pool seen in 256-byte rows; a part that starts 32 i bytes into such a row
                        // (A^T parts of 2 P r bytes come before it) goes through the map whose origin is that much further on
                        const long long ok_ = off + geo.bk_off, ov_ = off + geo.bv_off;
                        const CUtensorMap *mk = &maps.bk[(ok_ >> 5) & 7], *mv = &maps.bv[(ov_ >> 5) & 7];
                        const int yk = (int)(ok_ >> 8), yv = (int)(ov_ >> 8);
                        // (a pair: the second page's A^T parts follow the first's, its B rows start at row 16 of the panels)
                        const uint32_t dk = dst + L.k + j * (16 * 128), dv = dst + L.v + j * (16 * 128);
                        bulk_g2s_keep(dst + L.ak + j * umma_a_bytes(geo, geo.rank_k), src + geo.ak_off, geo.rank_k * 2 * P, bar);
                        bulk_g2s_keep(dst + L.av + j * umma_a_bytes(geo, geo.rank_v), src + geo.av_off, geo.rank_v * 2 * P, bar);
                        tma_box(dk, mk, 0, yk, bar);
                        tma_box(dk + L.k_panel, mk, 64, yk, bar);
                        tma_box(dv, mv, 0, yv, bar);
                        tma_box(dv + L.v_panel, mv, 64, yv, bar);
                    }
                } else if (rows > 0) {
                    // whole blocks: rows past the sequence's end hold whatever the pool holds; the scores there are
                    // masked and the row threads clear those rows
                    const int y = (int)(((long long)slot * geo.dense_slot_bytes + (long long)head * geo.dense_head_bytes) >> 8) + blk * kDB;
                    mbar_arrive_expect_tx(bar, 4 * L.d_panel);
                    tma_box(dst + L.dk, &maps.dense, 0, y, bar);
                    tma_box(dst + L.dk + L.d_panel, &maps.dense, 64, y, bar);
                    tma_box(dst + L.dv, &maps.dense, 0, y + P, bar);
                    tma_box(dst + L.dv + L.d_panel, &maps.dense, 64, y + P, bar);
                } else {
                    mbar_arrive(bar);
                }
            }
            if (!ok && !*abort_flag) { *abort_flag = 1; atomicAdd(a.status, 1); }
            // copies already in flight must land before the CTA retires: wait (bounded) for the stages armed last
            for (int back = 1; back <= min(u, S); ++back) {
                const int k = u - back;
                (void)mbar_wait(smem_u32(full_bar + k % S), (k / S) & 1, limit);
            }
        }
    } else if (warp == 5) {
        // ------------------------------ products (one lane) ------------------------------
        if (elect_one()) {
            const uint32_t sq_a = smem_u32(sq);
            const uint64_t dq0 = umma_desc(sq_a, 16, 1024, 2), dq1 = umma_desc(sq_a + kURows * 128, 16, 1024, 2);       // Q, channels 0-63 / 64-127
            const uint32_t t_qt = tm + kColQt, t_s = tm + kColS, t_w = tm + kColW, t_o = tm + kColO;
            uint32_t ph_A = 0, ph_B = 0, ph_C = 0;
            bool ok = true, o_valid = false;
            const uint32_t stages_a = smem_u32(stages);
            int s0 = 0, s1 = 0, s2 = 0, round2 = 0;          // stages of the units u, u + 1, u + 2; times the stage of u + 2 has been used before
            auto stage_at = [&](int s) { return stages_a + (uint32_t)(s * ustage); };
            // [128 x RP] = Q . (K side)^T: 8 steps of 16 channels; both operands K-major, 128-byte swizzle
            // (steps ks0 .. ks1 - 1: the eight steps of G1 are issued in two halves, so that they stand in the way of the
            // other CTA's products for half as long at a time)
            // (n: rows of the K side - RP for G1, the rows of a block for a dense unit)
            auto qk = [&](uint32_t t_dst, uint32_t kside, int panel, int ks0, int ks1, int n) {
                const uint32_t idesc = umma_idesc(128, n, 0);
                const uint64_t db0 = umma_desc(kside, 16, 1024, 2), db1 = umma_desc(kside + panel, 16, 1024, 2);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (ks >= ks0 && ks < ks1)
                        umma_ss(t_dst, umma_desc_step(ks < 4 ? dq0 : dq1, (ks & 3) * 32), umma_desc_step(ks < 4 ? db0 : db1, (ks & 3) * 32), idesc, ks > 0);
            };
            // o [128 x d] (+)= (rows of RP bf16 at t_src) . (V side): MN-major, two panels of 64 channels
            // (k: rows of the V side - RP for G4, the rows of a block for a dense unit)
            auto pv = [&](uint32_t t_src, uint32_t vside, int panel, int k) {
                const uint64_t dv = umma_desc(vside, panel, 1024, 2);
#pragma unroll
                for (int ks = 0; ks < 2; ++ks)
                    if (ks * 16 < k) umma_ts(t_o, t_src + ks * 8, umma_desc_step(dv, ks * 2048), umma_idesc(128, 128, 1), o_valid || ks > 0);
                o_valid = true;
            };
            // kind of a unit as the products see it: units without tokens run as dense units with every score masked
            // (the descriptor is passed on to the row threads, who meet it behind the next commit "Q": they need not wait
            // for the copies themselves)
            auto unit_kind = [&](int s, int round, bool &good, int unit) -> int {
                if (!wait_lane(smem_u32(full_bar + s), round & 1, abort_flag, limit)) { good = false; return kKindDense; }
                const StageDesc d = descs[s];
                info[unit & 1] = d;
                __threadfence_block();
                return d.kind == kKindFactor && d.rows > 0 ? kKindFactor : kKindDense;
            };
            int k0 = kKindDense, k1 = kKindDense, k2 = kKindDense;       // kinds of the units u, u + 1, u + 2
            for (int u = -2; u < n_units; ++u) {
                if (u >= 0) {
                    // hand-over A: p(u) is in tensor memory -> G3(u) | Gb(u)
                    if (!wait_lane(bar_A, ph_A, abort_flag, limit)) { ok = false; break; }
                    ph_A ^= 1;
                    tc_fence_after();
                    const uint32_t sb = stage_at(s0);
                    if (k0 == kKindFactor) {
#pragma unroll
                        for (int j = 0; j < (kPair ? 2 : 1); ++j) {        // (a pair: page j's tokens are columns 32 j .. of p, its ranks columns 16 j .. of w)
                            const uint64_t da = umma_desc(sb + L.av + j * umma_a_bytes(geo, geo.rank_v), 16, kAGroup, kASwizzle);
#pragma unroll
                            for (int ks = 0; ks < P / 16; ++ks)      // w = p . A_v, A_v^T in place (K-major)
                                umma_ts(t_w + j * RP1, t_s + (j * (P / 16) + ks) * 8, umma_desc_step(da, ks * 32), umma_idesc(128, RP1, 0), ks > 0);
                        }
                    } else {
                        pv(t_s, sb + L.dv, L.d_panel, kDB);
                        umma_commit(smem_u32(empty_bar + s0));         // a dense unit's stage is free after Gb
                    }
                    umma_commit(bar_G3);
                }
                if (u >= -1 && u + 1 < n_units) {
                    // hand-over B: q~(u+1) is in tensor memory -> G2(u+1) | Ga(u+1)
                    if (!wait_lane(bar_B, ph_B, abort_flag, limit)) { ok = false; break; }
                    ph_B ^= 1;
                    tc_fence_after();
                    const uint32_t sb = stage_at(s1);
                    if (k1 == kKindFactor) {
                        if (kPair) {
#pragma unroll
                            for (int j = 0; j < 2; ++j) {        // page j: its 16 columns of either term of q~ -> columns 32 j .. of s
                                const uint64_t dak = umma_desc(sb + L.ak + j * umma_a_bytes(geo, geo.rank_k), 16, kAGroup, kASwizzle);
#pragma unroll
                                for (int t = 0; t < 2; ++t)
                                    umma_ts(t_s + j * P, t_qt + t * (RP / 2) + j * 8, dak, umma_idesc(128, P, 1), t > 0);
                            }
                        } else {
                            const uint64_t dak = umma_desc(sb + L.ak, 16, kAGroup, kASwizzle);
#pragma unroll
                            for (int t = 0; t < 2; ++t)              // s = (q~_hi + q~_lo) . A_k^T, A_k^T in place (MN-major)
#pragma unroll
                                for (int ks = 0; ks < RP / 16; ++ks)
                                    umma_ts(t_s, t_qt + t * (RP / 2) + ks * 8, umma_desc_step(dak, ks * 2 * kAGroup),
                                            umma_idesc(128, P, 1), (t | ks) > 0);
                        }
                    } else {
                        qk(t_s, sb + L.dk, L.d_panel, 0, 8, kDB);
                    }
                    umma_commit(bar_S);
                    // behind it, off the rows' path: the first half of G1(u+2), over the q~ columns G2(u+1) has just read
                    if (u + 2 < n_units) {
                        k2 = unit_kind(s2, round2, ok, u + 2);
                        if (!ok) break;
                        if (k2 == kKindFactor) qk(t_qt, stage_at(s2) + L.k, L.k_panel, 0, 4, RP);
                    }
                }
                // hand-over C: w(u) is in tensor memory -> G4(u); then, off the rows' path, G1(u+2)
                if (!wait_lane(bar_C, ph_C, abort_flag, limit)) { ok = false; break; }
                ph_C ^= 1;
                tc_fence_after();
                if (u >= 0 && k0 == kKindFactor) {
                    pv(t_w, stage_at(s0) + L.v, L.v_panel, RP);
                    umma_commit(smem_u32(empty_bar + s0));             // a factor unit's stage is free after G4
                }
                if (u + 2 < n_units) {
                    if (u < -1) {                                  // (before the first unit there is no hand-over B)
                        k2 = unit_kind(s2, round2, ok, u + 2);
                        if (!ok) break;
                        if (k2 == kKindFactor) qk(t_qt, stage_at(s2) + L.k, L.k_panel, 0, 4, RP);
                    }
                    if (k2 == kKindFactor) qk(t_qt, stage_at(s2) + L.k, L.k_panel, 4, 8, RP);       // the second half of G1(u+2)
                }
                umma_commit(bar_Q);
                k0 = k1; k1 = k2;
                s0 = s1; s1 = s2;
                if (++s2 == S) { s2 = 0; ++round2; }
            }
            if (!ok && !*abort_flag) { *abort_flag = 1; atomicAdd(a.status, 1); }
            // nothing of this CTA's may still be running on the tensor cores when tensor memory is given back
            umma_commit(bar_drain);
            (void)mbar_wait(bar_drain, 0, limit);
        }
    } else {
        // ------------------------------ rows: one query row per thread ------------------------------
        const int row = rb * kURows + tid, j = row / G;
        const bool row_ok = row < n_rows;
        const long long qrow = ((long long)entry * a.q_len + j) * geo.n_q_heads + head * G + row % G;
        {
            const uint4 *qg = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(a.q) + qrow * kHeadDim);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint4 v = row_ok ? __ldg(qg + c) : make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(sq + (c >> 3) * (kURows * 128) + tid * 128 + (((c & 7) ^ (tid & 7)) << 4)) = v;
            }
            fence_async_smem();          // the products read Q through the async proxy
        }
        const int hid = row_ok ? a.q_len - 1 - j : 0;       // newest positions this row must not see
        const uint32_t t_lane = tm + ((uint32_t)(warp * 32) << 16);
        const uint32_t t_qt = t_lane + kColQt, t_s = t_lane + kColS, t_w = t_lane + kColW, t_o = t_lane + kColO;
        RowSoftmax st{kNegInf, 0.f, kNegInf};
        uint32_t ph_G3 = 0, ph_S = 0, ph_Q = 0;
        bool ok = true;
        const float scale = geo.scale_log2e;
        const bool full_tiles = geo.rank_k == 8 * NT && geo.rank_v == 8 * NT;     // then the rank bounds below are compile-time
        StageDesc cur{kKindDense, 0, 0, 0}, nxt{kKindDense, 0, 0, 0};
        int s_nxt = 0, round_nxt = 0;          // stage of the unit u + 1 and the times it has been used before
#define PKV_ROWS_WAIT(bar, ph) { if (!wait_warp(bar, ph, abort_flag, limit)) { ok = false; break; } ph ^= 1; tc_fence_after(); }
#define PKV_ROWS_ARRIVE(bar) { tc_fence_before(); mbar_arrive(bar); }
        for (int u = -2; u < n_units; ++u) {
            bool o_seen = false;          // whether this iteration has waited for the o of the unit before
            if (u >= 0) {
                // ---- softmax of s(u); p(u) -> hand-over A ----
                PKV_ROWS_WAIT(bar_S, ph_S)
                bool fine;
                if (cur.kind == kKindFactor) {
                    float sv[PU];
                    tmem_ld<PU>(t_s, reinterpret_cast<uint32_t *>(sv));
                    if (kPair && cur.rows < PU) {                 // the last page of an odd number: no second page
#pragma unroll
                        for (int i = P; i < PU; ++i) sv[i] = kMasked;
                    }
                    fine = softmax_row<PU, false>(sv, st, u > 0, t_s, t_o, bar_Q, ph_Q, o_seen, abort_flag, limit);
                } else {
                    float sv[kDB];
                    tmem_ld<kDB>(t_s, reinterpret_cast<uint32_t *>(sv));
                    const int lim = cur.rows - max(0, hid - cur.after);
#pragma unroll
                    for (int i = 0; i < kDB; ++i) sv[i] = i < lim ? sv[i] * scale : kMasked;
                    fine = softmax_row<kDB, true>(sv, st, u > 0, t_s, t_o, bar_Q, ph_Q, o_seen, abort_flag, limit);
                }
                if (!fine) { ok = false; break; }
                PKV_ROWS_ARRIVE(bar_A)
            }
            if (u >= -1 && !o_seen) PKV_ROWS_WAIT(bar_Q, ph_Q)   // G4(u-1) has added to o, G1(u+1) has written q~

            if (u >= -1 && u + 1 < n_units) {
                // ---- the next unit's descriptor; q~(u+1) as two bf16 terms -> hand-over B ----
                const int s = s_nxt, round = round_nxt;
                if (++s_nxt == S) { s_nxt = 0; ++round_nxt; }
                nxt = info[(u + 1) & 1];                        // written by the issuing lane ahead of the commit just met
                if (nxt.rows <= 0 || nxt.kind != kKindFactor) { nxt.kind = kKindDense; nxt.rows = max(0, min(nxt.rows, kDB)); }
                if (nxt.kind == kKindFactor) {      // columns past the rank are exact zeros
                    uint32_t rq[RP], hi[RP / 2], lo[RP / 2];
                    tmem_ld<RP>(t_qt, rq);
                    if (full_tiles) split_terms<RP, 8 * NT, true, kPair>(rq, hi, lo, scale, 8 * NT);
                    else split_terms<RP, RP, false, kPair>(rq, hi, lo, scale, geo.rank_k);
                    tmem_st<RP / 2>(t_qt, hi);
                    tmem_st<RP / 2>(t_qt + RP / 2, lo);
                    tmem_st_wait();
                } else if (nxt.rows < kDB) {
                    // rows past the sequence's end hold whatever the pool held: p is 0 there, but the rows must be
                    // finite (V), also for a padded product of the stage before this one (K).  (The copies have
                    // landed: the issuing lane has seen them; the wait costs nothing and orders these stores behind them.)
                    if (!wait_warp(smem_u32(full_bar + s), round & 1, abort_flag, limit)) { ok = false; break; }
                    unsigned char *st_base = stages + (size_t)s * ustage;
                    for (int i = tid; i < (kDB - nxt.rows) * 32; i += kURows) {
                        const int side = i & 1, panel = (i >> 1) & 1, chunk = (i >> 2) & 7, r = nxt.rows + (i >> 5);
                        *reinterpret_cast<uint4 *>(st_base + (side ? L.dv : L.dk) + panel * L.d_panel + r * 128 + chunk * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                    fence_async_smem();
                }
                PKV_ROWS_ARRIVE(bar_B)
            }
            if (u >= 0) {
                // ---- w(u) as bf16 -> hand-over C ----
                PKV_ROWS_WAIT(bar_G3, ph_G3)
                if (cur.kind == kKindFactor) {       // into the frame o is kept in; columns past the rank are exact zeros
                    uint32_t rw[RP], pk[RP / 2];
                    tmem_ld<RP>(t_w, rw);
                    const float c = exp2_fast(st.m - st.m_ref);
                    if (full_tiles) scale_pack<RP, 8 * NT, true, kPair>(rw, pk, c, 8 * NT);
                    else scale_pack<RP, RP, false, kPair>(rw, pk, c, geo.rank_v);
                    tmem_st<RP / 2>(t_w, pk);
                    tmem_st_wait();
                }
            }
            PKV_ROWS_ARRIVE(bar_C)
            cur = nxt;
        }
        if (ok) {                                                       // the last G4 | Gb
            ok = wait_warp(bar_Q, ph_Q, abort_flag, limit);
            tc_fence_after();
        }
#undef PKV_ROWS_WAIT
#undef PKV_ROWS_ARRIVE
        if (!ok && lane == 0 && !*abort_flag) { *abort_flag = 1; atomicAdd(a.status, 1); }
        if (ok && ns > 1) {
            // this range's state: o in the frame of its own maximum m, then m and l (rows of kRbStateFloats floats)
            const float f = st.l > 0.f ? exp2_fast(st.m_ref - st.m) : 0.f;
            float *dst = a.rb_partials + ((size_t)blockIdx.x * kURows + tid) * kRbStateFloats;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                if (n_units > 0) {                                      // (without units o was never written)
                    tmem_ld32(t_o + 32 * c, r);
                    tmem_ld_wait();
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = n_units > 0 ? __float_as_uint(__uint_as_float(r[i]) * f) : 0u;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    *reinterpret_cast<uint4 *>(dst + 32 * c + 4 * k) = make_uint4(r[4 * k], r[4 * k + 1], r[4 * k + 2], r[4 * k + 3]);
            }
            *reinterpret_cast<float2 *>(dst + kHeadDim) = make_float2(st.m, st.l);
        } else if (ok) {
            const float inv = st.l > 0.f ? exp2_fast(st.m_ref - st.m) / st.l : 0.f;          // o is in the frame of m_ref
            __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.out);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld32(t_o + 32 * c, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * inv);
                if (row_ok) {
                    if (out) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            *reinterpret_cast<uint4 *>(out + qrow * kHeadDim + 32 * c + 8 * k) =
                                make_uint4(pack_bf16(__uint_as_float(r[8 * k]), __uint_as_float(r[8 * k + 1])),
                                           pack_bf16(__uint_as_float(r[8 * k + 2]), __uint_as_float(r[8 * k + 3])),
                                           pack_bf16(__uint_as_float(r[8 * k + 4]), __uint_as_float(r[8 * k + 5])),
                                           pack_bf16(__uint_as_float(r[8 * k + 6]), __uint_as_float(r[8 * k + 7])));
                    }
                    if (a.out_f32) {
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            *reinterpret_cast<uint4 *>(a.out_f32 + qrow * kHeadDim + 32 * c + 4 * k) = make_uint4(r[4 * k], r[4 * k + 1], r[4 * k + 2], r[4 * k + 3]);
                    }
                }
            }
        }
    }
    // ------------------------------ every thread: give tensor memory back ------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(kTmemCols) : "memory");
}

// Eq. 5 over the ns ranges of a row block: one warp per query row, a lane per four channels; the ranges are taken in
// token order, so the result does not depend on which CTA finished first.
__global__ void __launch_bounds__(256) rowblock_merge_kernel(const __grid_constant__ DecodeArgs a) {
    const Geometry &geo = a.geo;
    const int ns = a.rb_splits, H = geo.n_kv_heads, G = geo.group;
    const int n_rows = a.q_len * G, n_blk = (n_rows + kURows - 1) / kURows;
    const int blk_id = (int)blockIdx.x / (kURows / 8), r = ((int)blockIdx.x % (kURows / 8)) * 8 + ((int)threadIdx.x >> 5);
    const int n_he = (int)gridDim.x / (kURows / 8) / n_blk;
    const int rb = n_blk - 1 - blk_id / n_he, head = (blk_id % n_he) % H, entry = (blk_id % n_he) / H;
    const int row = rb * kURows + r, lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    const long long qrow = ((long long)entry * a.q_len + row / G) * geo.n_q_heads + head * G + row % G;
    const float *src = a.rb_partials + ((size_t)blk_id * ns * kURows + r) * kRbStateFloats;
    const size_t stride = (size_t)kURows * kRbStateFloats;
    // lane k holds (m, l) of range k (at most 32 ranges) and works out the range's weight 2^(m_k - M); the sum over
    // the ranges then takes each weight by a shuffle, so that the loads of the o rows do not wait for one another
    static_assert(kRbMaxSplits <= 32, "one lane per range");
    float2 ml = make_float2(kNegInf, 0.f);
    if (lane < ns) ml = *reinterpret_cast<const float2 *>(src + lane * stride + kHeadDim);
    float M = ml.y > 0.f ? ml.x : kNegInf;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, d));
    const float wk = ml.y > 0.f ? exp2f(ml.x - M) : 0.f;          // weight of range `lane`
    float L = wk * ml.y;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int k = 0; k < ns; ++k) {                                  // token order: the sum is the same whoever ran first
        const float w = __shfl_sync(0xffffffffu, wk, k);
        const float4 o = *reinterpret_cast<const float4 *>(src + k * stride + 4 * lane);
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
    }
    // (l: summed in lane order by a fixed tree, the same for every launch)
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) L += __shfl_xor_sync(0xffffffffu, L, d);
    const float inv = L > 0.f ? 1.f / L : 0.f;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    if (a.out)
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + qrow * kHeadDim + 4 * lane) =
            make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    if (a.out_f32) *reinterpret_cast<float4 *>(a.out_f32 + qrow * kHeadDim + 4 * lane) = acc;
}

size_t umma_smem_bytes(const Geometry &g) {
    const int S = umma_stages(g);
    return (size_t)kUQBytes + (size_t)S * umma_stage_bytes(g) + umma_stage_pad(g) + (2 * S + 8) * 8 + (S + 2) * sizeof(StageDesc) + 64;
}

}  // namespace

bool row_block_umma_supported(const Geometry &g) {
    // A^T rows of 128, 64 or 32 bytes (P = 64, 32, 16: the swizzles the tensor cores know for such rows); every part of a blob
    // on a 32-byte boundary of the pool (the tiled copies address the pools in 256-byte rows, from one of eight origins
    // 32 bytes apart), which every rank gives
    return (g.page == 64 || g.page == 32 || g.page == 16) && g.factor_bits == 16 && g.global_rank == 0 &&
           g.rank_tiles >= 1 && g.rank_tiles <= 4 && g.bk_off % 32 == 0 && g.bv_off % 32 == 0 &&
           g.blob_bytes % 32 == 0 && g.factor_slot_bytes % 32 == 0 && umma_smem_bytes(g) <= (size_t)kSmemBudget / 2;
}

#define PKV_FOR_EACH_UMMA_SHAPE(X) X(64, 1) X(64, 2) X(64, 3) X(64, 4) X(32, 1) X(32, 2) X(32, 3) X(32, 4) X(16, 1) X(16, 2)

cudaError_t row_block_umma_setup() {
    cudaError_t e;
#define PKV_UMMA_SETUP(P, NT) \
    if ((e = cudaFuncSetAttribute(block_umma_kernel<P, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget / 2)) != cudaSuccess) return e;
    PKV_FOR_EACH_UMMA_SHAPE(PKV_UMMA_SETUP)
#undef PKV_UMMA_SETUP
    return cudaSuccess;
}

// Tensor maps of the two pools seen as matrices of 256-byte rows (128 bf16), box = 64 channels x `rows`; for the factor
// pool eight pairs with origins 32 bytes apart (see the copy lane).  The encoder is a driver entry
// point; it is looked up at run time so that the library does not link against the driver.
void row_block_make_maps(const Geometry &g, const void *factor_pool, const void *dense_pool, RowBlockMaps *maps) {
    typedef CUresult (*EncodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                    const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    maps->valid = 0;
    if (!row_block_umma_supported(g) || !dense_pool) return;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult found = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &found) != cudaSuccess || !fn ||
        found != cudaDriverEntryPointSuccess) {
        (void)cudaGetLastError();
        return;
    }
    const EncodeTiled encode = reinterpret_cast<EncodeTiled>(fn);
    auto make = [&](CUtensorMap *m, const void *base, long long bytes, int rows) -> bool {
        const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)(bytes / kRowBytes)};
        const cuuint64_t strides[1] = {(cuuint64_t)kRowBytes};
        const cuuint32_t box[2] = {64u, (cuuint32_t)rows}, elem[2] = {1u, 1u};
        return dims[1] > 0 && dims[1] < (1ull << 31) &&
               encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, elem,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    const int rb = umma_part_rows(g);
    if (!make(&maps->dense, dense_pool, (long long)g.n_dense_slots * g.dense_slot_bytes, rb)) return;
    if (factor_pool && g.n_factor_slots > 0) {
        const long long bytes = (long long)g.n_factor_slots * g.factor_slot_bytes;
        for (int i = 0; i < 8; ++i) {
            const unsigned char *origin = static_cast<const unsigned char *>(factor_pool) + 32 * i;
            if (i > 0 && bytes - 32 * i < 512) {          // (a pool of one or two rows: nothing can start there)
                maps->bk[i] = maps->bk[0];
                maps->bv[i] = maps->bv[0];
            } else if (!make(&maps->bk[i], origin, bytes - 32 * i, g.rank_k) || !make(&maps->bv[i], origin, bytes - 32 * i, g.rank_v)) {
                return;
            }
        }
    } else {
        for (int i = 0; i < 8; ++i) maps->bk[i] = maps->bv[i] = maps->dense;          // no factor pages: never used
    }
    maps->valid = 1;
}

// One CTA per (sequence, KV head, block of 128 query rows), or a.rb_splits CTAs with a range of the sequence each and
// a second launch that merges their states.
cudaError_t launch_decode_blocks_umma(const DecodeArgs &a, int n_seqs, const RowBlockMaps &maps, cudaStream_t st) {
    const int n_blk = (a.q_len * a.geo.group + kURows - 1) / kURows;
    const long long n_blocks = (long long)n_seqs * a.geo.n_kv_heads * n_blk, n_ctas = n_blocks * a.rb_splits;
    if (!maps.valid || !row_block_umma_supported(a.geo) || n_blocks <= 0 || n_ctas > 0x7fffffffLL || a.rb_splits < 1 ||
        (a.rb_splits > 1 && (!a.rb_partials || n_ctas > kRbSplitItems)))
        return cudaErrorInvalidValue;
    const size_t smem = umma_smem_bytes(a.geo);
    cudaError_t e = cudaErrorInvalidValue;
#define PKV_UMMA_LAUNCH(P, NT) \
    if (a.geo.page == P && a.geo.rank_tiles == NT) { block_umma_kernel<P, NT><<<(unsigned)n_ctas, kUThreads, smem, st>>>(a, maps); e = cudaGetLastError(); }
    PKV_FOR_EACH_UMMA_SHAPE(PKV_UMMA_LAUNCH)
#undef PKV_UMMA_LAUNCH
    if (e == cudaSuccess && a.rb_splits > 1) {
        rowblock_merge_kernel<<<(unsigned)(n_blocks * (kURows / 8)), 256, 0, st>>>(a);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace pkv
