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

constexpr int kXs = kHeadDim + 2;         // padded row stride of X (bf16): 65 words, odd

// Rotation pairs of every round for P = 16, 32, 64 (offsets 0, 15*8, 15*8 + 31*16), written once per device by
// the host.  A pair is stored as (first, second); for P = 64 the orientation is chosen so that the 32 first
// members of a round fall into 32 different shared-memory banks (index mod 32), and so do the second members.
__constant__ uchar2 c_pairs[15 * 8 + 31 * 16 + 63 * 32];
__host__ __device__ constexpr int pair_table_offset(int P) { return P == 16 ? 0 : (P == 32 ? 15 * 8 : 15 * 8 + 31 * 16); }

template <int P>
struct Shape {
    static constexpr int kThreads = 4 * P;              // 256 / 128 / 64
    static constexpr int kWarps = kThreads / 32;
    // Row stride of G (floats).  Not padded on purpose: the bank of G[i][j] is then j mod 32 alone, which is what
    // makes the block update below conflict-free (see there).
    static constexpr int kGs = P;
    static constexpr int kPairs = P / 2;
    // 2 x 2 blocks of G computed per round: one of each mirror-image couple, and the diagonal blocks
    static constexpr int kBlocks = kPairs * (kPairs / 2) + kPairs / 2;
    static constexpr int kChunks = P / 4;               // float4 chunks of a row of Q^T
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
    uchar2 pairs[(P - 1) * (P / 2)];   // this page size's rows of c_pairs (lanes index it divergently)
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

template <int P>
__global__ void __launch_bounds__(Shape<P>::kThreads)
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

    // ---- cyclic Jacobi sweeps ----
    // The P/2 rotations of a round act on disjoint index pairs, so G' = J^T G J splits into (P/2)^2 independent
    // 2 x 2 blocks: block (a, b) = rows of pair a, columns of pair b, becomes J_a^T . block . J_b.  G is
    // symmetric, so one block of every mirror-image couple is computed: a thread reads its block's four entries
    // and writes them and their mirror images (G stays bitwise symmetric), so G passes through shared memory once
    // per round.  Lanes walk a wrapped diagonal, block (a, a + delta mod P/2) for lane a: delta = 0 .. P/4 covers
    // every couple once (delta = P/4 with a < P/4 only).  On a diagonal the lanes' row pairs are all different
    // and so are their column pairs; the bank of an entry is its column index mod 32 and the oriented pair table
    // keeps a round's first members (and its second members) in different banks, so neither the block accesses
    // (bank = a member of the column pair) nor the mirrored stores (bank = a member of the row pair) conflict.
    // For P < 64 a warp holds several diagonals; every other one takes its pairs in the opposite order, (q, p)
    // with the rotation (c, -s), which is the same rotation, so that it touches second members while its
    // neighbour touches first members.
    // Q^T is stored instead of Q: rotating columns p, q of Q is rotating rows p, q of Q^T, four tokens at a time.
    for (int i = tid; i < (P - 1) * kPairs; i += kThreads) S.pairs[i] = c_pairs[pair_table_offset(P) + i];
    __syncthreads();
    const uchar2 *pairs = S.pairs;
    bool converged = false;
    for (int sweep = 0; sweep < geo.jacobi_max_sweeps && !converged; ++sweep) {
        int rotated = 0;
        for (int rho = 0; rho < P - 1; ++rho) {
            const uchar2 *pr = pairs + rho * kPairs;
            if (tid < kPairs) {
                const int p = pr[tid].x, q = pr[tid].y;
                const float gpp = S.G[p * kGs + p], gqq = S.G[q * kGs + q], gpq = S.G[p * kGs + q];
                float c = 1.f, s = 0.f;
                if (fabsf(gpq) > fmaxf(tol * sqrtf(fabsf(gpp * gqq)), floor_abs)) {
                    const float theta = (gqq - gpp) / (2.f * gpq);
                    const float t = copysignf(1.f, theta) / (fabsf(theta) + sqrtf(1.f + theta * theta));
                    c = rsqrtf(1.f + t * t);
                    s = t * c;
                    rotated = 1;
                }
                S.cs[tid] = make_float2(c, s);
            }
            __syncthreads();
#pragma unroll
            for (int u0 = 0; u0 < Sh::kBlocks; u0 += kThreads) {
                const int u = u0 + tid;
                if (u < Sh::kBlocks) {
                    const int delta = u / kPairs, ia = u % kPairs, ib = (ia + delta) % kPairs;
                    float2 ca = S.cs[ia], cb = S.cs[ib];
                    if (ca.y != 0.f || cb.y != 0.f) {
                        uchar2 pa = pr[ia], pb = pr[ib];
                        if (kPairs < 32 && (delta & 1)) {
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
            for (int i0 = 0; i0 < kPairs * Sh::kChunks; i0 += kThreads) {
                const int item = i0 + tid;
                if (item < kPairs * Sh::kChunks) {
                    const int k = item / Sh::kChunks, ch = item % Sh::kChunks;
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
        if (!converged && geo.jacobi_energy_tol >= 0.f) {
            // energy captured by the r largest diagonal entries after this sweep
            if (tid < P) S.lam[tid] = S.G[tid * kGs + tid];
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
            if (captured_prev >= 0.f && captured - captured_prev <= geo.jacobi_energy_tol * fmaxf(trace - captured, 0.f))
                converged = true;
            captured_prev = captured;
        }
    }
    if (!converged && tid == 0) atomicAdd(&status[1], 1);

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

// Round-robin pairs of every round.  For P = 64 each pair is oriented (first, second) so that the first members
// of a round have distinct indices mod 32 (and hence so do the second members): mark x first and its partner y
// second; y ^ 32 shares y's bank, so it must be a first member; continue from there until the cycle closes.
void fill_pair_table(int P, uchar2 *out) {
    const int B = P / 2;
    for (int rho = 0; rho < P - 1; ++rho) {
        int partner[kMaxPage], role[kMaxPage];      // role: 0 unknown, 1 first, 2 second
        for (int k = 0; k < B; ++k) {
            int p, q;
            pair_of(P, rho, k, p, q);
            partner[p] = q; partner[q] = p;
            role[p] = P == 64 ? 0 : 1; role[q] = P == 64 ? 0 : 2;
        }
        if (P == 64) {
            for (int start = 0; start < P; ++start) {
                int x = start;
                while (role[x] == 0) {
                    role[x] = 1;
                    const int y = partner[x];
                    role[y] = 2;
                    x = y ^ 32;
                }
            }
        }
        int k = 0;
        for (int x = 0; x < P; ++x)
            if (role[x] == 1) out[rho * B + k++] = make_uchar2((unsigned char)x, (unsigned char)partner[x]);
    }
}

cudaError_t upload_pair_tables() {
    static uchar2 host[15 * 8 + 31 * 16 + 63 * 32];
    fill_pair_table(16, host + pair_table_offset(16));
    fill_pair_table(32, host + pair_table_offset(32));
    fill_pair_table(64, host + pair_table_offset(64));
    return cudaMemcpyToSymbol(c_pairs, host, sizeof host);
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
