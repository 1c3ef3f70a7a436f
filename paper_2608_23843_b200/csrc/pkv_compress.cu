// Batched per-page truncated SVD (paper: Eq. 2 and the Gram-matrix route that
// follows Eq. 3).  One CTA factorizes one P x d page X (K or V of one KV head):
//   G = X X^T (P x P, fp32, exact bf16 products)        -> shared memory
//   cyclic Jacobi eigen-solve of G with Q^T accumulating the rotations (fp32)
//   A = the r eigenvectors of largest eigenvalue, B = A^T X, both rounded to bf16
// Pages are independent, so the grid is simply (work-list entries) x (KV heads) x (K|V).
#include <cuda_bf16.h>

#include "pkv_internal.h"

namespace pkv {

namespace {

// Two fp32 values in one 64-bit register and the sm_100 instructions that multiply-add both halves at once.  Each half
// is an ordinary round-to-nearest FMA, so a sum written with them has the bits of the scalar version; what changes is
// the number of instructions (the dense 4 x 4 updates below are bound by instruction issue).
struct F2 { unsigned long long v; };
__device__ __forceinline__ F2 f2(float lo, float hi) { F2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void f2_get(F2 a, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v)); }
__device__ __forceinline__ F2 f2_mul(F2 a, F2 b) { F2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ F2 f2_fma(F2 a, F2 b, F2 c) { F2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r; }


constexpr int kXs = kHeadDim + 2;         // padded row stride of X (bf16): 65 words, odd

// Rotation pairs of every round of the pair ordering (P = 16), written once per device by the host.  A pair is
// stored as (first, second) = (smaller, larger index).
__constant__ uchar2 c_pairs[15 * 8];

// P = 64 and P = 32 use groups of four instead (see the quad ordering in the kernel).  A class partitions the P
// indices into P/4 quads; the classes of a sweep contain every pair of indices at least once.
//   P = 64: the indices are the points of the affine space AG(3, 4), a quad is a line, and the 21 parallel classes
//           of 16 lines contain every pair exactly once.  A line's members are stored in the order (A, B, A, B): an
//           index and its partner (index ^ 32, the one that shares its shared-memory bank) always get different
//           letters, so the 32 A-members of a class lie in 32 different banks, and so do the 32 B-members.
//   P = 32: no such design exists for 32 points.  Each half of 16 indices is an affine plane AG(2, 4): its 5
//           parallel classes of 4 lines give 5 classes of 8 quads with every pair inside a half once; the 256
//           pairs between the halves come from 8 more classes of quads {x, x ^ u, 16 + (x ^ a), 16 + (x ^ u ^ a)},
//           which hold the pairs of difference a and u ^ a (the 16 differences are split into 8 couples {a, a ^ u}),
//           and repeat two pairs inside the halves.  13 classes, 8 of them with two repeated pairs per quad.
template <int P> struct Quads {
    static constexpr int kQuads = P / 4;                       // per class
    static constexpr int kClasses = P == 64 ? 21 : 13;
    static constexpr int kDiag = 32 / kQuads;                  // wrapped diagonals of quad blocks per warp: 2 or 4
    static constexpr int kVarStep = 4 / kDiag;                 // lane group g takes its quads' members in the order j ^ (g * kVarStep)
    // off-diagonal quad blocks of G computed per class, one of every mirror-image couple (the diagonal blocks come
    // out of the rotation phase)
    static constexpr int kItems = kQuads * (kQuads / 2 - 1) + kQuads / 2;
    static constexpr int kGWarps = (kItems + 31) / 32;         // 4 or 1; the remaining warps update Q^T
    static constexpr int kQIters = kQuads * (P / 4) / 32;      // 8 or 2
    static constexpr int kCheck = (kClasses + 2) / 3;          // the energy rule is evaluated about three times per sweep
    // Where row k of quad q's 4 x 4 transform lives in M (variant g): quad-major with a stride of five float4.  The
    // eight lanes of a quarter warp that store rows (two quads x four rows: slots 5q + k) and the eight that load one
    // row of eight consecutive quads (slots 5q + k, q = 8j .. 8j+7) both cover all eight 16-byte bank groups.
    static constexpr int kMStride = 5;
    __host__ __device__ static constexpr int mslot(int g, int q, int k) { return (g * kQuads + q) * kMStride + k; }
};
__constant__ uchar4 c_quads64[Quads<64>::kClasses * Quads<64>::kQuads];
__constant__ uchar4 c_quads32[Quads<32>::kClasses * Quads<32>::kQuads];

template <int P>
struct Shape {
    static constexpr int kThreads = 4 * P;              // 256 / 128 / 64
    static constexpr int kWarps = kThreads / 32;
    // Row stride of G (floats).  Not padded on purpose: the bank of G[i][j] is then j mod 32 alone, which is what
    // makes the block update below conflict-free (see there).
    static constexpr int kGs = P;
    static constexpr int kPairs = P / 2;
    static constexpr int kMinBlocks = P == 64 ? 4 : (P == 32 ? 8 : 1);  // resident CTAs per SM the register allocation must allow
};

// The page X is needed for the Gram matrix and again for B = A^T X; in between its bytes hold Q^T, and it is
// fetched a second time (from L2, most likely) into the bytes of G once the eigenvalues are known: two P x P
// fp32 arrays per page instead of three let more pages share an SM.
template <int P>
struct CompressSmem {
    union {
        __nv_bfloat16 X[P * kXs];      // load and Gram phases (padded rows)
        float QT[P * P];               // Q^T: row j = eigenvector candidate j (16-byte aligned rows)
    };
    union {
        float G[P * P];
        __nv_bfloat16 X2[P * kHeadDim];    // the page again, rows unpadded (projection phase)
    };
    float2 cs[P / 2];
    uchar2 pairs[P >= 32 ? 1 : (P - 1) * (P / 2)];   // pair ordering: the rounds' pairs (lanes index it divergently)
    // quad ordering: the 4 x 4 transforms of a class's quads, [member order][row][quad] as float4, and the table
    using Qd = Quads<(P >= 32 ? P : 32)>;
    float4 M[P >= 32 ? Qd::kDiag * Qd::kMStride * Qd::kQuads : 1];
    uchar4 quads[P >= 32 ? Qd::kClasses * Qd::kQuads : 1];
    float lam[P];
    int order[P];
    float red[Shape<P>::kWarps];
};

// Extra shared memory of the INT4 epilogue (placed behind CompressSmem<P>).
struct QuantSmem {
    float B[32 * kHeadDim];        // B = A^T X in fp32, rank rows
    float root[32], inv[32];       // sqrt(sigma_j) and its inverse (0 for a zero row)
    float s_rank[32];              // stored (bf16-valued) scales: per rank column of A~ (keys)
    float s_tok[kMaxPage];         //                              per token of A~ (values)
    float s_ch[kHeadDim];          //                              per channel of B~
};

__device__ __forceinline__ float bf16_round(float v) {
    return __bfloat162float(__float2bfloat16_rn(v));
}
// symmetric INT4 code of x for a stored scale: round half to even, clipped to [-7, 7] (0 if the scale is 0),
// returned in its stored form code + 8
__device__ __forceinline__ unsigned int4_code(float x, float scale) {
    if (!(scale > 0.f)) return 8u;
    const float q = fminf(fmaxf(rintf(x / scale), -7.f), 7.f);
    return (unsigned)((int)q + 8);
}

// Round-robin tournament: in round rho (0..P-2) the P indices form P/2 disjoint
// pairs; over P-1 rounds every pair meets exactly once.
inline void pair_of(int P, int rho, int k, int &p, int &q) {
    const int m = P - 1;
    int a, b;
    if (k == 0) { a = m; b = rho; }
    else { a = rho + k; if (a >= m) a -= m; b = rho - k; if (b < 0) b += m; }
    p = a < b ? a : b; q = a < b ? b : a;
}

// Jacobi rotation (c, s) that zeroes g_pq: t = tan(angle) = 2 g_pq / (d + sign(d) sqrt(d^2 + 4 g_pq^2)), d = g_qq - g_pp
// (the smaller root, |t| <= 1), c = 1 / sqrt(1 + t^2), s = t c.  Skipped (c = 1, s = 0, returns false) when
// |g_pq| <= tol sqrt(|g_pp g_qq|) or |g_pq| <= floor_abs.  The reciprocal and the square roots are the hardware
// approximations (2 ulp): they set the angle, not the orthogonality, which rests on c^2 + s^2 = c^2 (1 + t^2).
__device__ __forceinline__ bool jacobi_rotation(float gpp, float gqq, float gpq, float tol, float floor_abs, float &c,
                                                float &s) {
    c = 1.f;
    s = 0.f;
    if (!(fabsf(gpq) > floor_abs && gpq * gpq > tol * tol * fabsf(gpp * gqq))) return false;
    const float d = gqq - gpp;
    const float h2 = fmaf(d, d, 4.f * gpq * gpq);
    const float h = h2 * rsqrtf(h2);
    const float t = __fdividef(2.f * gpq, d + copysignf(h, d));
    c = rsqrtf(fmaf(t, t, 1.f));
    s = t * c;
    return true;
}

// Early-stopping rule: the energy captured by the r largest diagonal entries of G is ||A^T X||_F^2 of the factors
// the current Q would give; when it stops growing (relative to the reconstruction error that is left) the
// remaining rotations only polish eigenvectors inside clusters.  Block-wide; every thread gets the answer.
template <int P>
__device__ __noinline__ bool energy_converged(CompressSmem<P> &S, int rank, float energy_tol, float trace,
                                              float &captured_prev, int tid, int lane, int warp) {
    constexpr int kWarps = Shape<P>::kWarps;
    // At full rank every orthogonal Q captures all of the energy, so the rule says nothing: keep rotating until Q
    // holds the eigenvectors (they give the factors the smallest entries, hence the least bf16 rounding error).
    if (rank >= P) return false;
    if (tid < P) S.lam[tid] = S.G[tid * Shape<P>::kGs + tid];
    __syncthreads();
    float mine = 0.f;
    if (tid < P) {
        const float li = S.lam[tid];
        int r = 0;
        for (int j = 0; j < P; ++j) {
            const float lj = S.lam[j];
            r += (lj > li) || (lj == li && j < tid);
        }
        if (r < rank) mine = li;
    }
    for (int o = 16; o; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if (lane == 0) S.red[warp] = mine;
    __syncthreads();
    float captured = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) captured += S.red[w];
    __syncthreads();
    const bool done = captured_prev >= 0.f && captured - captured_prev <= energy_tol * fmaxf(trace - captured, 0.f);
    captured_prev = captured;
    return done;
}

template <int P>
__global__ void __launch_bounds__(Shape<P>::kThreads, Shape<P>::kMinBlocks)
compress_kernel(Geometry geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                const int2 *worklist, int *status) {
    using Sh = Shape<P>;
    constexpr int kGs = Sh::kGs, kThreads = Sh::kThreads, kWarps = Sh::kWarps, kPairs = Sh::kPairs;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    CompressSmem<P> &S = *reinterpret_cast<CompressSmem<P> *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kv = blockIdx.x & 1;
    const int head = (blockIdx.x >> 1) % geo.n_kv_heads;
    const int entry = (blockIdx.x >> 1) / geo.n_kv_heads;
    const int2 wk = worklist[entry];
    if (wk.x < 0 || wk.x >= geo.n_dense_slots || wk.y < 0 || wk.y >= geo.n_factor_slots) {
        if (tid == 0) atomicAdd(&status[2], 1);       // corrupt work list: skip the page, leave a mark
        return;
    }
    const int rank = kv ? geo.rank_v : geo.rank_k;
    const unsigned char *src = dense_pool + (long long)wk.x * geo.dense_slot_bytes +
                               (long long)head * geo.dense_head_bytes + kv * (P * kRowBytes);
    unsigned char *blob = factor_pool + (long long)wk.y * geo.factor_slot_bytes + (long long)head * geo.blob_bytes;
    unsigned char *dstA = blob + (kv ? geo.av_off : geo.ak_off);
    unsigned char *dstB = blob + (kv ? geo.bv_off : geo.bk_off);

    // ---- load the page (undo the storage swizzle) ----
    for (int i = tid; i < P * 16; i += kThreads) {
        const int row = i >> 4, chunk = i & 15;
        const uint4 val = *reinterpret_cast<const uint4 *>(src + row * kRowBytes + swz_chunk(row, chunk) * 16);
        unsigned *dst = reinterpret_cast<unsigned *>(&S.X[row * kXs + chunk * 8]);
        dst[0] = val.x; dst[1] = val.y; dst[2] = val.z; dst[3] = val.w;
    }
    __syncthreads();

    // ---- Gram matrix: a 4 x 4 tile per thread ((P/4)^2 tiles) ----
    if (tid < (P / 4) * (P / 4)) {
        const int ti = tid / (P / 4), tj = tid % (P / 4);
        float acc[4][4] = {};
        for (int k = 0; k < kHeadDim; k += 2) {
            float2 a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                a[u] = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&S.X[(4 * ti + u) * kXs + k]));
                b[u] = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&S.X[(4 * tj + u) * kXs + k]));
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int w = 0; w < 4; ++w) acc[u][w] = fmaf(a[u].y, b[w].y, fmaf(a[u].x, b[w].x, acc[u][w]));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int w = 0; w < 4; ++w) S.G[(4 * ti + u) * kGs + 4 * tj + w] = acc[u][w];
    }
    __syncthreads();
    for (int i = tid; i < P * P / 4; i += kThreads) {          // Q^T = I, over the bytes of X
        const int r = i / (P / 4), c4 = (i % (P / 4)) * 4;
        reinterpret_cast<float4 *>(S.QT)[i] = make_float4(r == c4 ? 1.f : 0.f, r == c4 + 1 ? 1.f : 0.f,
                                                          r == c4 + 2 ? 1.f : 0.f, r == c4 + 3 ? 1.f : 0.f);
    }
    // G[i][j] and G[j][i] were accumulated from the same products in the same order: G is bitwise symmetric
    // absolute floor below which an off-diagonal entry is rounding noise of the Gram matrix
    float dmax = 0.f;
    if (tid < P) dmax = fabsf(S.G[tid * kGs + tid]);
    for (int o = 16; o; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
    if (lane == 0) S.red[warp] = dmax;
    __syncthreads();
    float gmax = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) gmax = fmaxf(gmax, S.red[w]);
    const float floor_abs = 2e-7f * gmax;
    const float tol = geo.jacobi_tol;
    // trace(G) = ||X||_F^2: with the energy captured by the r largest diagonal entries it gives the squared
    // reconstruction error the current Q would yield (used by the early-stopping rule below)
    float tr = tid < P ? S.G[tid * kGs + tid] : 0.f;
    for (int o = 16; o; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
    __syncthreads();
    if (lane == 0) S.red[warp] = tr;
    __syncthreads();
    float trace = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) trace += S.red[w];
    float captured_prev = -1.f;
    bool converged = false;
    int n_rounds = 0;                 // rotation rounds (classes of quads, or rounds of pairs) this page went through
    if constexpr (P >= 32) {
        using Qd = Quads<P>;
        constexpr int kQuads = Qd::kQuads;
        // ---- quad ordering ----
        // A class partitions the P indices into P/4 quads.  Inside a quad the six pairs are rotated in three layers,
        // (0,1)(2,3), (0,2)(1,3), (0,3)(1,2), which needs only the quad's own 4 x 4 diagonal block of G; the product
        // of the six rotations is a 4 x 4 orthogonal matrix M.  Then G' = M^T G M and Q^T' = M^T Q^T are applied
        // blockwise with dense 4 x 4 products: one pass over G and Q^T covers what takes three rounds of the pair
        // ordering, with a third of the shared-memory traffic and instructions; 21 classes (P = 64) or 13 (P = 32)
        // make a sweep in which every pair is rotated (see Quads).
        //   first P threads     four per quad: rotations and M                                   (between barriers)
        //   first kGWarps warps G: a thread owns the 4 x 4 block (quad a, quad b) of a mirror-image couple; a group
        //                       of P/4 lanes walks a wrapped diagonal (b = a + delta mod P/4, delta = 1 .. P/8), reads
        //                       16 entries, writes 16 and their mirror images
        //   the other warps     Q^T: a thread owns (quad, four tokens): four 128-bit loads, 64 FMAs, four stores
        // Banks: an entry's bank is its column index mod 32.  Lane group g of a warp takes its quads' members in
        // the order j ^ x (x = 0, 2 for the two groups at P = 64; x = 0 .. 3 for the four groups at P = 32) with M
        // permuted to match.  At P = 64 the warp then touches either all A-members or all B-members of the class at
        // any step, at P = 32 one member of each kind of every quad, i.e. all 32 indices: 32 different banks, for
        // the block accesses (columns of quad b) and for the mirrored stores (columns of quad a) alike.
        for (int i = tid; i < Qd::kClasses * kQuads; i += kThreads) S.quads[i] = P == 64 ? c_quads64[i] : c_quads32[i];
        __syncthreads();
        float4 *QT4 = reinterpret_cast<float4 *>(S.QT);
        for (int sweep = 0; sweep < geo.jacobi_max_sweeps && !converged; ++sweep) {
            int rotated = 0;
            for (int cls = 0; cls < Qd::kClasses && !converged; ++cls) {
                const uchar4 *quads = S.quads + cls * kQuads;
                ++n_rounds;
                if (tid < 4 * kQuads) {
                    // Four lanes per quad; lane t holds row t of the quad's diagonal block D and of M, stored
                    // "rotated": e[k] = D[t][t ^ k], f[k] = M[t][t ^ k], so that the partner of layer x (t ^ x), the
                    // pivot (e[x]) and the column pairs (k, k ^ x) have compile-time positions.
                    const int qd = tid >> 2, t = tid & 3;
                    const unsigned m4 = reinterpret_cast<const unsigned *>(quads)[qd];
                    const int mt = (m4 >> (8 * t)) & 0xff;
                    float e[4], f[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        e[k] = S.G[mt * kGs + ((m4 >> (8 * (t ^ k))) & 0xff)];
                        f[k] = k == 0 ? 1.f : 0.f;
                    }
#pragma unroll
                    for (int x = 1; x <= 3; ++x) {                      // layer x pairs t with t ^ x
                        const int y = x == 1 ? 2 : 1;                   // t ^ y lies in the layer's other pair
                        const bool low = t < (t ^ x);                   // this lane is the pair's lower index
                        const float d_mine = e[0], d_other = __shfl_xor_sync(0xffffffffu, e[0], x);
                        // both lanes of a pair must arrive at the same rotation: take the pivot from the lower one
                        const float g_other = __shfl_xor_sync(0xffffffffu, e[x], x), gpq = low ? e[x] : g_other;
                        const float gpp = low ? d_mine : d_other, gqq = low ? d_other : d_mine;
                        float c, sn;
                        if (jacobi_rotation(gpp, gqq, gpq, tol, floor_abs, c, sn)) rotated = 1;
                        const float c2 = __shfl_xor_sync(0xffffffffu, c, y), s2 = __shfl_xor_sync(0xffffffffu, sn, y);
                        // columns: positions (0, x) belong to this lane's pair, (y, y ^ x) to the other pair; the
                        // entry at position k is column t ^ k, the lower column of its pair iff (t ^ k) < (t ^ k ^ x)
                        const float sa = low ? sn : -sn;                                  // position 0 = column t
                        const float sb = ((t ^ y) < (t ^ y ^ x)) ? s2 : -s2;              // position y
                        const float e0 = c * e[0] - sa * e[x], ex = c * e[x] + sa * e[0];
                        const float ey = c2 * e[y] - sb * e[y ^ x], eyx = c2 * e[y ^ x] + sb * e[y];
                        const float f0 = c * f[0] - sa * f[x], fx = c * f[x] + sa * f[0];
                        const float fy = c2 * f[y] - sb * f[y ^ x], fyx = c2 * f[y ^ x] + sb * f[y];
                        f[0] = f0; f[x] = fx; f[y] = fy; f[y ^ x] = fyx;
                        // rows: new row t = c row t -/+ s row (t ^ x); the partner's entry of the same column sits
                        // at its position k ^ x
                        const float p0 = __shfl_xor_sync(0xffffffffu, ex, x), px = __shfl_xor_sync(0xffffffffu, e0, x);
                        const float py = __shfl_xor_sync(0xffffffffu, eyx, x), pyx = __shfl_xor_sync(0xffffffffu, ey, x);
                        e[0] = c * e0 - sa * p0; e[x] = c * ex - sa * px;
                        e[y] = c * ey - sa * py; e[y ^ x] = c * eyx - sa * pyx;
                    }
                    // e now holds row t of J^T D J over all six rotations = the quad's diagonal block of the new G:
                    // written here (upper triangle and its mirror image), so the block phase can leave it alone
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int cc = t ^ k;
                        if (cc >= t) {
                            const int mc = (m4 >> (8 * cc)) & 0xff;
                            S.G[mt * kGs + mc] = e[k];
                            S.G[mc * kGs + mt] = e[k];
                        }
                    }
                    // natural column order: M[t][c] = f[t ^ c]
                    float r0 = f[0], r1 = f[1], r2 = f[2], r3 = f[3];
                    if (t & 1) { float w = r0; r0 = r1; r1 = w; w = r2; r2 = r3; r3 = w; }
                    if (t & 2) { float w = r0; r0 = r2; r2 = w; w = r1; r1 = r3; r3 = w; }
                    const float r[4] = {r0, r1, r2, r3};
#pragma unroll
                    for (int g = 0; g < Qd::kDiag; ++g) {              // M'[k][j] = M[k ^ x][j ^ x] for member order j ^ x
                        constexpr int kStep = Qd::kVarStep;
                        const int x = g * kStep;
                        S.M[Qd::mslot(g, qd, t ^ x)] = make_float4(r[0 ^ x], r[1 ^ x], r[2 ^ x], r[3 ^ x]);
                    }
                }
                __syncthreads();
                if (warp < Qd::kGWarps) {
                    const int h = lane / kQuads, ia = lane % kQuads, delta = 1 + Qd::kDiag * warp + h;
                    if (delta < kQuads / 2 || (delta == kQuads / 2 && ia < kQuads / 2)) {
                        const int ib = (ia + delta) % kQuads;
                        // member order j ^ x: byte j of the permuted word is byte j ^ x of the table's
                        const unsigned sel = 0x3210u ^ (0x1111u * (unsigned)(h * Qd::kVarStep));
                        const unsigned ma4 = __byte_perm(reinterpret_cast<const unsigned *>(quads)[ia], 0u, sel);
                        const unsigned mb4 = __byte_perm(reinterpret_cast<const unsigned *>(quads)[ib], 0u, sel);
                        int ma[4], mb[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) { ma[i] = (ma4 >> (8 * i)) & 0xff; mb[i] = (mb4 >> (8 * i)) & 0xff; }
                        const float4 *Ma = S.M + Qd::mslot(h, ia, 0), *Mb = S.M + Qd::mslot(h, ib, 0);    // rows 0..3 of the quad
                        // (two values per instruction; per value the operations and their order are those of the scalar form)
                        F2 Tlo[4], Thi[4];                             // (T[0][j], T[1][j]) and (T[2][j], T[3][j])
#pragma unroll
                        for (int j = 0; j < 4; ++j) Tlo[j] = Thi[j] = f2(0.f, 0.f);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {                  // T = M_a^T X
                            const float4 mk = Ma[k];
                            const F2 mlo = f2(mk.x, mk.y), mhi = f2(mk.z, mk.w);
                            const float *row = S.G + ma[k] * kGs;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float x = row[mb[j]];
                                const F2 xx = f2(x, x);
                                Tlo[j] = f2_fma(mlo, xx, Tlo[j]);
                                Thi[j] = f2_fma(mhi, xx, Thi[j]);
                            }
                        }
                        float T[4][4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) { f2_get(Tlo[j], T[0][j], T[1][j]); f2_get(Thi[j], T[2][j], T[3][j]); }
                        const float4 b0 = Mb[0], b1 = Mb[1], b2 = Mb[2], b3 = Mb[3];
                        const F2 b0a = f2(b0.x, b0.y), b0b = f2(b0.z, b0.w), b1a = f2(b1.x, b1.y), b1b = f2(b1.z, b1.w);
                        const F2 b2a = f2(b2.x, b2.y), b2b = f2(b2.z, b2.w), b3a = f2(b3.x, b3.y), b3b = f2(b3.z, b3.w);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {                  // Y = T M_b, row i
                            float y[4];
                            const F2 t0 = f2(T[i][0], T[i][0]), t1 = f2(T[i][1], T[i][1]), t2 = f2(T[i][2], T[i][2]), t3 = f2(T[i][3], T[i][3]);
                            f2_get(f2_fma(t3, b3a, f2_fma(t2, b2a, f2_fma(t1, b1a, f2_mul(t0, b0a)))), y[0], y[1]);
                            f2_get(f2_fma(t3, b3b, f2_fma(t2, b2b, f2_fma(t1, b1b, f2_mul(t0, b0b)))), y[2], y[3]);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                S.G[ma[i] * kGs + mb[j]] = y[j];
                                S.G[mb[j] * kGs + ma[i]] = y[j];
                            }
                        }
                    }
                } else {
                    for (int itq = warp - Qd::kGWarps; itq < Qd::kQIters; itq += kWarps - Qd::kGWarps) {
                        const int v = itq * 32 + lane, k = v / (P / 4), ch = v % (P / 4);
                        const uchar4 m4 = quads[k];
                        float4 *r0 = QT4 + m4.x * (P / 4) + ch, *r1 = QT4 + m4.y * (P / 4) + ch;
                        float4 *r2 = QT4 + m4.z * (P / 4) + ch, *r3 = QT4 + m4.w * (P / 4) + ch;
                        const float4 x0 = *r0, x1 = *r1, x2 = *r2, x3 = *r3;
                        const float4 *Mk = S.M + Qd::mslot(0, k, 0);
                        const float4 c0 = Mk[0], c1 = Mk[1], c2 = Mk[2], c3 = Mk[3];
                        // row i' = sum_k M[k][i] row k, two channels per instruction (same order of operations per channel)
                        const F2 x0a = f2(x0.x, x0.y), x0b = f2(x0.z, x0.w), x1a = f2(x1.x, x1.y), x1b = f2(x1.z, x1.w);
                        const F2 x2a = f2(x2.x, x2.y), x2b = f2(x2.z, x2.w), x3a = f2(x3.x, x3.y), x3b = f2(x3.z, x3.w);
#define PKV_MIX(dst, comp) { const F2 k0 = f2(c0.comp, c0.comp), k1 = f2(c1.comp, c1.comp), k2 = f2(c2.comp, c2.comp), k3 = f2(c3.comp, c3.comp); \
                             float4 o; \
                             f2_get(f2_fma(k3, x3a, f2_fma(k2, x2a, f2_fma(k1, x1a, f2_mul(k0, x0a)))), o.x, o.y); \
                             f2_get(f2_fma(k3, x3b, f2_fma(k2, x2b, f2_fma(k1, x1b, f2_mul(k0, x0b)))), o.z, o.w); \
                             *dst = o; }
                        PKV_MIX(r0, x) PKV_MIX(r1, y) PKV_MIX(r2, z) PKV_MIX(r3, w)
#undef PKV_MIX
                    }
                }
                __syncthreads();
                // about three checks per sweep
                if (((cls + 1) % Qd::kCheck == 0 || cls == Qd::kClasses - 1) && geo.jacobi_energy_tol >= 0.f && energy_converged<P>(S, rank, geo.jacobi_energy_tol, trace, captured_prev, tid, lane, warp)) converged = true;
            }
            if (!__syncthreads_or(rotated)) converged = true;
        }
    } else {
        // ---- cyclic Jacobi sweeps, pair ordering (P = 16) ----
        // 2 x 2 blocks of G computed per round: one of each mirror-image couple, and the diagonal blocks
        constexpr int kBlocks = kPairs * (kPairs / 2) + kPairs / 2;
        constexpr int kChunks = P / 4;               // float4 chunks of a row of Q^T
        // The P/2 rotations of a round act on disjoint index pairs, so G' = J^T G J splits into (P/2)^2 independent
        // 2 x 2 blocks: block (a, b) = rows of pair a, columns of pair b, becomes J_a^T . block . J_b.  G is
        // symmetric, so one block of every mirror-image couple is computed: a thread reads its block's four entries
        // and writes them and their mirror images (G stays bitwise symmetric), so G passes through shared memory once
        // per round.  Lanes walk a wrapped diagonal, block (a, a + delta mod P/2) for lane a: delta = 0 .. P/4 covers
        // every couple once (delta = P/4 with a < P/4 only).  On a diagonal the lanes' row pairs are all different
        // and so are their column pairs; G's rows are unpadded, so the bank of an entry is its column index (all
        // below 32 here): neither the block accesses (bank = a member of the column pair) nor the mirrored stores
        // (bank = a member of the row pair) conflict inside a diagonal.  A warp holds several diagonals; every
        // other one takes its pairs in the opposite order, (q, p) with the rotation (c, -s), which is the same
        // rotation, so that it touches second members while its neighbour touches first members.
        // Q^T is stored instead of Q: rotating columns p, q of Q is rotating rows p, q of Q^T, four tokens at a time.
        for (int i = tid; i < (P - 1) * kPairs; i += kThreads) S.pairs[i] = c_pairs[i];
        __syncthreads();
        const uchar2 *pairs = S.pairs;
        for (int sweep = 0; sweep < geo.jacobi_max_sweeps && !converged; ++sweep) {
            int rotated = 0;
            for (int rho = 0; rho < P - 1; ++rho) {
                const uchar2 *pr = pairs + rho * kPairs;
                ++n_rounds;
                if (tid < kPairs) {
                    const int p = pr[tid].x, q = pr[tid].y;
                    const float gpp = S.G[p * kGs + p], gqq = S.G[q * kGs + q], gpq = S.G[p * kGs + q];
                    float c, s;
                    if (jacobi_rotation(gpp, gqq, gpq, tol, floor_abs, c, s)) rotated = 1;
                    S.cs[tid] = make_float2(c, s);
                }
                __syncthreads();
#pragma unroll
                for (int u0 = 0; u0 < kBlocks; u0 += kThreads) {
                    const int u = u0 + tid;
                    if (u < kBlocks) {
                        const int delta = u / kPairs, ia = u % kPairs, ib = (ia + delta) % kPairs;
                        float2 ca = S.cs[ia], cb = S.cs[ib];
                        if (ca.y != 0.f || cb.y != 0.f) {
                            uchar2 pa = pr[ia], pb = pr[ib];
                            if (delta & 1) {
                                pa = make_uchar2(pa.y, pa.x); ca.y = -ca.y;
                                pb = make_uchar2(pb.y, pb.x); cb.y = -cb.y;
                            }
                            float *g0 = S.G + pa.x * kGs, *g1 = S.G + pa.y * kGs;
                            const float x00 = g0[pb.x], x01 = g0[pb.y], x10 = g1[pb.x], x11 = g1[pb.y];
                            const float y00 = ca.x * x00 - ca.y * x10, y01 = ca.x * x01 - ca.y * x11;
                            const float y10 = ca.y * x00 + ca.x * x10, y11 = ca.y * x01 + ca.x * x11;
                            const float z00 = cb.x * y00 - cb.y * y01, z01 = cb.y * y00 + cb.x * y01;
                            const float z10 = cb.x * y10 - cb.y * y11, z11 = cb.y * y10 + cb.x * y11;
                            if (delta != 0) {
                                g0[pb.x] = z00; g0[pb.y] = z01; g1[pb.x] = z10; g1[pb.y] = z11;
                                float *h0 = S.G + pb.x * kGs, *h1 = S.G + pb.y * kGs;
                                h0[pa.x] = z00; h1[pa.x] = z01; h0[pa.y] = z10; h1[pa.y] = z11;
                            } else {                       // diagonal block: x01 = x10, and so are their images
                                g0[pb.x] = z00; g0[pb.y] = z01; g1[pb.x] = z01; g1[pb.y] = z11;
                            }
                        }
                    }
                }
                // rows p, q of Q^T:  x_p' = c x_p - s x_q,  x_q' = s x_p + c x_q
#pragma unroll
                for (int i0 = 0; i0 < kPairs * kChunks; i0 += kThreads) {
                    const int item = i0 + tid;
                    if (item < kPairs * kChunks) {
                        const int k = item / kChunks, ch = item % kChunks;
                        const float2 cs = S.cs[k];
                        if (cs.y != 0.f) {
                            const uchar2 pq = pr[k];
                            float4 *rp = reinterpret_cast<float4 *>(S.QT + pq.x * P) + ch;
                            float4 *rq = reinterpret_cast<float4 *>(S.QT + pq.y * P) + ch;
                            const float4 xp = *rp, xq = *rq;
                            *rp = make_float4(cs.x * xp.x - cs.y * xq.x, cs.x * xp.y - cs.y * xq.y,
                                              cs.x * xp.z - cs.y * xq.z, cs.x * xp.w - cs.y * xq.w);
                            *rq = make_float4(cs.y * xp.x + cs.x * xq.x, cs.y * xp.y + cs.x * xq.y,
                                              cs.y * xp.z + cs.x * xq.z, cs.y * xp.w + cs.x * xq.w);
                        }
                    }
                }
                __syncthreads();
            }
            converged = !__syncthreads_or(rotated);
            if (!converged && geo.jacobi_energy_tol >= 0.f && energy_converged<P>(S, rank, geo.jacobi_energy_tol, trace, captured_prev, tid, lane, warp)) converged = true;
        }
    }
    if (tid == 0) {
        if (!converged) atomicAdd(&status[1], 1);
        // 64-bit totals for the throughput report: rounds and page SVDs
        atomicAdd(reinterpret_cast<unsigned long long *>(status + 4), (unsigned long long)n_rounds);
        atomicAdd(reinterpret_cast<unsigned long long *>(status + 6), 1ull);
    }

    // ---- order eigenvalues: descending, ties by lower index ----
    if (tid < P) { S.lam[tid] = S.G[tid * kGs + tid]; S.order[tid] = tid; }
    __syncthreads();
    if (tid < P) {
        const float li = S.lam[tid];
        int r = 0;
        for (int j = 0; j < P; ++j) {
            const float lj = S.lam[j];
            r += (lj > li) || (lj == li && j < tid);
        }
        S.order[r] = tid;       // r < P always; NaN eigenvalues may collide (outputs then unspecified)
    }
    __syncthreads();
    // ---- the page again (G is no longer needed) ----
    for (int i = tid; i < P * 16; i += kThreads) {
        const int row = i >> 4, chunk = i & 15;
        reinterpret_cast<uint4 *>(S.X2)[i] =
            *reinterpret_cast<const uint4 *>(src + row * kRowBytes + swz_chunk(row, chunk) * 16);
    }
    __syncthreads();

    if (geo.factor_bits == 4) {
        // ---- INT4 factors (paper, Section 4.3): A~ = A Sigma^(1/2), B~ = Sigma^(-1/2) B, symmetric 4-bit codes ----
        QuantSmem &Z = *reinterpret_cast<QuantSmem *>(smem_raw + ((sizeof(CompressSmem<P>) + 15) / 16) * 16);
        for (int i = tid; i < rank * (kHeadDim / 2); i += kThreads) {
            const int j = i / (kHeadDim / 2), col = (i % (kHeadDim / 2)) * 2;
            const int oj = S.order[j];
            float b0 = 0.f, b1 = 0.f;
#pragma unroll 8
            for (int r = 0; r < P; ++r) {
                const float a = S.QT[oj * P + r];
                const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&S.X2[r * kHeadDim + col]));
                b0 = fmaf(a, x.x, b0);
                b1 = fmaf(a, x.y, b1);
            }
            Z.B[j * kHeadDim + col] = b0;
            Z.B[j * kHeadDim + col + 1] = b1;
        }
        __syncthreads();
        if (tid < rank) {                                   // sigma_j = ||B_j||
            float ss = 0.f;
            for (int c = 0; c < kHeadDim; ++c) ss = fmaf(Z.B[tid * kHeadDim + c], Z.B[tid * kHeadDim + c], ss);
            const float root = sqrtf(sqrtf(ss));
            Z.root[tid] = root;
            Z.inv[tid] = root > 0.f ? 1.f / root : 0.f;
        }
        __syncthreads();
        // scales = max|x| / 7, stored in bf16: keys per rank column of A~, values per token of A~; B~ per channel
        unsigned char *sc_base = blob + geo.codes_bytes;
        if (!kv) {
            if (tid < rank) {
                const int oj = S.order[tid];
                float m = 0.f;
                for (int i = 0; i < P; ++i) m = fmaxf(m, fabsf(S.QT[oj * P + i]));
                const float sc = bf16_round(m * Z.root[tid] / 7.f);
                Z.s_rank[tid] = sc;
                *reinterpret_cast<__nv_bfloat16 *>(sc_base + geo.sak_off + 2 * tid) = __float2bfloat16_rn(sc);
            } else if (tid < ((rank + 7) & ~7)) {           // padding entries of the rank-scale array
                *reinterpret_cast<__nv_bfloat16 *>(sc_base + geo.sak_off + 2 * tid) = __float2bfloat16_rn(0.f);
            }
        } else if (tid < P) {
            float m = 0.f;
            for (int j = 0; j < rank; ++j) m = fmaxf(m, fabsf(S.QT[S.order[j] * P + tid] * Z.root[j]));
            const float sc = bf16_round(m / 7.f);
            Z.s_tok[tid] = sc;
            *reinterpret_cast<__nv_bfloat16 *>(sc_base + geo.sav_off + 2 * tid) = __float2bfloat16_rn(sc);
        }
        for (int c = tid; c < kHeadDim; c += kThreads) {
            float m = 0.f;
            for (int j = 0; j < rank; ++j) m = fmaxf(m, fabsf(Z.B[j * kHeadDim + c] * Z.inv[j]));
            const float sc = bf16_round(m / 7.f);
            Z.s_ch[c] = sc;
            *reinterpret_cast<__nv_bfloat16 *>(sc_base + (kv ? geo.sbv_off : geo.sbk_off) + 2 * c) = __float2bfloat16_rn(sc);
        }
        __syncthreads();
        // code words in operand-register order (see int4_a_pos / int4_b_pos): A~ region, then B~ region of this
        // matrix pair; ranks past the true rank and registers past the last one hold zero codes
        const int NT = geo.rank_tiles;
        const int a_words = kv ? int4_b_words(P, NT) : int4_a_words(P, NT);
        const int b_words = kv ? int4_a_words(kHeadDim, NT) : int4_b_words(kHeadDim, NT);
        unsigned *wa = reinterpret_cast<unsigned *>(blob + (kv ? geo.cav_off : geo.cak_off));
        unsigned *wb = reinterpret_cast<unsigned *>(blob + (kv ? geo.cbv_off : geo.cbk_off));
        for (int w = tid; w < a_words + b_words; w += kThreads) {
            const bool is_a = w < a_words;
            const int wl = is_a ? w : w - a_words, ln = wl & 31, wq = wl >> 5;
            unsigned word = 0u;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int t = e >> 1, h = e & 1, n = 4 * wq + t;
                int x = 0, j = 0;                  // x: token (A~) or channel (B~); j: rank
                unsigned code = 8u;
                if (is_a) {
                    const bool ok = kv ? int4_b_elem(P, NT, ln, n, h, x, j) : int4_a_elem(P, NT, ln, n, h, x, j);
                    if (ok && j < rank)
                        code = int4_code(S.QT[S.order[j] * P + x] * Z.root[j], kv ? Z.s_tok[x] : Z.s_rank[j]);
                } else {
                    const bool ok = kv ? int4_a_elem(kHeadDim, NT, ln, n, h, x, j) : int4_b_elem(kHeadDim, NT, ln, n, h, x, j);
                    if (ok && j < rank) code = int4_code(Z.B[j * kHeadDim + x] * Z.inv[j], Z.s_ch[x]);
                }
                word |= code << (4 * (t + 4 * h));
            }
            (is_a ? wa : wb)[wl] = word;
        }
        return;
    }
    // ---- A^T [r][P] = Q[:, order[:r]]^T as bf16, chunk-swizzled rows ----
    for (int i = tid; i < rank * (P / 2); i += kThreads) {
        const int j = i / (P / 2), tok = (i % (P / 2)) * 2;
        const int oj = S.order[j];
        const float a0 = S.QT[oj * P + tok], a1 = S.QT[oj * P + tok + 1];
        *reinterpret_cast<__nv_bfloat162 *>(dstA + a_t_offset(P, j, tok)) = __floats2bfloat162_rn(a0, a1);
    }
    // ---- B = A^T X (fp32 eigenvectors, exact page), rows swizzled like dense rows ----
    for (int i = tid; i < rank * (kHeadDim / 2); i += kThreads) {
        const int j = i / (kHeadDim / 2), col = (i % (kHeadDim / 2)) * 2;
        const int oj = S.order[j];
        float b0 = 0.f, b1 = 0.f;
#pragma unroll 8
        for (int r = 0; r < P; ++r) {
            const float a = S.QT[oj * P + r];
            const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&S.X2[r * kHeadDim + col]));
            b0 = fmaf(a, x.x, b0);
            b1 = fmaf(a, x.y, b1);
        }
        *reinterpret_cast<__nv_bfloat162 *>(dstB + j * kRowBytes + swz_chunk(j, col >> 3) * 16 + (col & 7) * 2) =
            __floats2bfloat162_rn(b0, b1);
    }
}

// Round-robin pairs of every round (P = 16).
void fill_pair_table(int P, uchar2 *out) {
    const int B = P / 2;
    for (int rho = 0; rho < P - 1; ++rho)
        for (int k = 0; k < B; ++k) {
            int p, q;
            pair_of(P, rho, k, p, q);
            out[rho * B + k] = make_uchar2((unsigned char)p, (unsigned char)q);
        }
}

// The 21 parallel classes of lines of AG(3, 4) over the indices 0..63 (index = x0 + 4 x1 + 16 x2, coordinates in
// GF(4) = {0, 1, w, w^2} with addition = xor), members ordered (A, B, A, B) as Quads describes.
void fill_quad_table64(uchar4 *out) {
    constexpr int kQuadClasses = Quads<64>::kClasses, kQuadsPerClass = Quads<64>::kQuads;
    static const int mul[4][4] = {{0, 0, 0, 0}, {0, 1, 2, 3}, {0, 2, 3, 1}, {0, 3, 1, 2}};
    int dirs[kQuadClasses][3], nd = 0;
    for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) { dirs[nd][0] = 1; dirs[nd][1] = a; dirs[nd][2] = b; ++nd; }
    for (int a = 0; a < 4; ++a) { dirs[nd][0] = 0; dirs[nd][1] = 1; dirs[nd][2] = a; ++nd; }
    dirs[nd][0] = 0; dirs[nd][1] = 0; dirs[nd][2] = 1; ++nd;
    for (int c = 0; c < kQuadClasses; ++c) {
        int line[kQuadsPerClass][4], n_lines = 0, mate[64], colour[64];
        bool seen[64] = {};
        for (int x = 0; x < 64; ++x) {
            if (seen[x]) continue;
            for (int t = 0; t < 4; ++t) {
                const int y = (x & 3) ^ mul[t][dirs[c][0]] | (((x >> 2) & 3) ^ mul[t][dirs[c][1]]) << 2 |
                              (((x >> 4) & 3) ^ mul[t][dirs[c][2]]) << 4;
                line[n_lines][t] = y;
                seen[y] = true;
            }
            ++n_lines;
        }
        // Two-colour the indices so that mates inside a line (members 0-1 and 2-3) differ and so do x and x ^ 32:
        // the two perfect matchings form even cycles, walked alternately.
        for (int l = 0; l < kQuadsPerClass; ++l) {
            mate[line[l][0]] = line[l][1]; mate[line[l][1]] = line[l][0];
            mate[line[l][2]] = line[l][3]; mate[line[l][3]] = line[l][2];
        }
        for (int x = 0; x < 64; ++x) colour[x] = -1;
        for (int start = 0; start < 64; ++start) {
            int x = start;
            while (colour[x] < 0) {
                colour[x] = 0;
                const int y = mate[x];
                colour[y] = 1;
                x = y ^ 32;
            }
        }
        for (int l = 0; l < kQuadsPerClass; ++l) {
            int m[4];
            for (int half = 0; half < 2; ++half) {
                const int u = line[l][2 * half], v = line[l][2 * half + 1];
                m[2 * half] = colour[u] == 0 ? u : v;
                m[2 * half + 1] = colour[u] == 0 ? v : u;
            }
            out[c * kQuadsPerClass + l] = make_uchar4((unsigned char)m[0], (unsigned char)m[1], (unsigned char)m[2],
                                                      (unsigned char)m[3]);
        }
    }
}

// The 13 classes of 8 quads for 32 indices (see Quads): GF(4)^2 lines inside each half of 16, then the classes that
// pair the halves.  Index inside a half = x0 + 4 x1.
void fill_quad_table32(uchar4 *out) {
    static const int mul[4][4] = {{0, 0, 0, 0}, {0, 1, 2, 3}, {0, 2, 3, 1}, {0, 3, 1, 2}};
    static const int dirs[5][2] = {{1, 0}, {1, 1}, {1, 2}, {1, 3}, {0, 1}};
    int n = 0;
    for (int c = 0; c < 5; ++c) {
        bool seen[16] = {};
        for (int x = 0; x < 16; ++x) {
            if (seen[x]) continue;
            int m[4];
            for (int t = 0; t < 4; ++t) {
                m[t] = ((x & 3) ^ mul[t][dirs[c][0]]) | (((x >> 2) & 3) ^ mul[t][dirs[c][1]]) << 2;
                seen[m[t]] = true;
            }
            out[n++] = make_uchar4((unsigned char)m[0], (unsigned char)m[1], (unsigned char)m[2], (unsigned char)m[3]);
        }
        for (int l = 0; l < 4; ++l) {                       // the same four lines in the other half
            const uchar4 q = out[n - 4];
            out[n++] = make_uchar4((unsigned char)(q.x + 16), (unsigned char)(q.y + 16), (unsigned char)(q.z + 16),
                                   (unsigned char)(q.w + 16));
        }
    }
    // differences 0..15 in couples {a, a ^ u}; u varies so that the repeated pairs inside the halves vary too
    static const int couple[8][2] = {{0, 1}, {2, 6}, {3, 11}, {4, 5}, {7, 15}, {8, 10}, {9, 13}, {12, 14}};
    for (int c = 0; c < 8; ++c) {
        const int a = couple[c][0], u = couple[c][0] ^ couple[c][1];
        bool seen[16] = {};
        for (int x = 0; x < 16; ++x) {
            if (seen[x]) continue;
            seen[x] = seen[x ^ u] = true;
            out[n++] = make_uchar4((unsigned char)x, (unsigned char)(16 + (x ^ a)), (unsigned char)(x ^ u),
                                   (unsigned char)(16 + (x ^ u ^ a)));
        }
    }
}

cudaError_t upload_pair_tables() {
    static uchar2 host[15 * 8];
    fill_pair_table(16, host);
    cudaError_t e = cudaMemcpyToSymbol(c_pairs, host, sizeof host);
    if (e != cudaSuccess) return e;
    static uchar4 quads64[Quads<64>::kClasses * Quads<64>::kQuads], quads32[Quads<32>::kClasses * Quads<32>::kQuads];
    fill_quad_table64(quads64);
    fill_quad_table32(quads32);
    if ((e = cudaMemcpyToSymbol(c_quads64, quads64, sizeof quads64)) != cudaSuccess) return e;
    return cudaMemcpyToSymbol(c_quads32, quads32, sizeof quads32);
}

template <int P>
cudaError_t launch_p(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                     const int2 *worklist, int n_entries, int *status, cudaStream_t st) {
    static bool configured[64] = {};         // attribute and constant table are per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(compress_kernel<P>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(sizeof(CompressSmem<P>) + 16 + sizeof(QuantSmem)));
        if (e != cudaSuccess) return e;
        if ((e = upload_pair_tables()) != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const unsigned grid = (unsigned)n_entries * geo.n_kv_heads * 2;
    const size_t smem = sizeof(CompressSmem<P>) + (geo.factor_bits == 4 ? 16 + sizeof(QuantSmem) : 0);
    compress_kernel<P><<<grid, Shape<P>::kThreads, smem, st>>>(geo, dense_pool, factor_pool, worklist, status);
    return cudaGetLastError();
}

}  // namespace

bool rotation_schedule(int P, unsigned char *out, long long cap, int *n_rounds, int *groups, int *group_size) {
    if (!out || !n_rounds || !groups || !group_size) return false;
    if (P == 64 || P == 32) {
        const int nr = P == 64 ? Quads<64>::kClasses : Quads<32>::kClasses, ng = P / 4;
        if (cap < (long long)nr * ng * 4) return false;
        static uchar4 table[Quads<64>::kClasses * Quads<64>::kQuads];
        if (P == 64) fill_quad_table64(table); else fill_quad_table32(table);
        for (int i = 0; i < nr * ng; ++i) {
            out[4 * i] = table[i].x; out[4 * i + 1] = table[i].y; out[4 * i + 2] = table[i].z; out[4 * i + 3] = table[i].w;
        }
        *n_rounds = nr; *groups = ng; *group_size = 4;
        return true;
    }
    if (P == 16) {
        if (cap < 15 * 8 * 2) return false;
        uchar2 table[15 * 8];
        fill_pair_table(16, table);
        for (int i = 0; i < 15 * 8; ++i) { out[2 * i] = table[i].x; out[2 * i + 1] = table[i].y; }
        *n_rounds = 15; *groups = 8; *group_size = 2;
        return true;
    }
    return false;
}

cudaError_t launch_compress(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                            const int2 *worklist, int n_entries, int *status, cudaStream_t st) {
    switch (geo.page) {
        case 16: return launch_p<16>(geo, dense_pool, factor_pool, worklist, n_entries, status, st);
        case 32: return launch_p<32>(geo, dense_pool, factor_pool, worklist, n_entries, status, st);
        case 64: return launch_p<64>(geo, dense_pool, factor_pool, worklist, n_entries, status, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace pkv
