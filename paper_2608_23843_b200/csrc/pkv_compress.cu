// Batched per-page truncated SVD (paper: Eq. 2 and the Gram-matrix route that
// follows Eq. 3).  One CTA factorizes one P x d page X (K or V of one KV head):
//   G = X X^T (P x P, fp32, exact bf16 products)        -> shared memory
//   cyclic Jacobi eigen-solve of G with Q accumulating the rotations (fp32)
//   A = the r eigenvectors of largest eigenvalue, B = A^T X, both rounded to bf16
// Pages are independent, so the grid is simply (work-list entries) x (KV heads) x (K|V).
#include <cuda_bf16.h>

#include "pkv_internal.h"

namespace pkv {

namespace {

constexpr int kXs = kHeadDim + 2;         // padded row stride of X (bf16): 65 words, odd

template <int P>
struct Shape {
    static constexpr int kThreads = 4 * P;              // 256 / 128 / 64
    static constexpr int kWarps = kThreads / 32;
    static constexpr int kGs = P + 1;                   // padded row stride of G and Q (floats)
    static constexpr int kPairsPerWarp = (P / 2) / kWarps;   // = 4 for every P
    static constexpr int kHalves = (P + 31) / 32;       // 32-row groups a warp walks in the column phase
};

template <int P>
struct CompressSmem {
    float G[P * (P + 1)];
    float Q[P * (P + 1)];
    __nv_bfloat16 X[P * kXs];
    float2 cs[P / 2];
    float lam[P];
    int order[P];
    float red[Shape<P>::kWarps];
};

// Round-robin tournament: in round rho (0..P-2) the P indices form P/2 disjoint
// pairs; over P-1 rounds every pair meets exactly once.
template <int P>
__device__ __forceinline__ void pair_of(int rho, int k, int &p, int &q) {
    constexpr int m = P - 1;
    int a, b;
    if (k == 0) { a = m; b = rho; }
    else { a = rho + k; if (a >= m) a -= m; b = rho - k; if (b < 0) b += m; }
    p = min(a, b); q = max(a, b);
}

template <int P>
__global__ void __launch_bounds__(Shape<P>::kThreads)
compress_kernel(Geometry geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                const int2 *worklist, int *status) {
    using Sh = Shape<P>;
    constexpr int kGs = Sh::kGs, kThreads = Sh::kThreads, kWarps = Sh::kWarps;
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
            for (int w = 0; w < 4; ++w) {
                S.G[(4 * ti + u) * kGs + 4 * tj + w] = acc[u][w];
                S.Q[(4 * ti + u) * kGs + 4 * tj + w] = (4 * ti + u == 4 * tj + w) ? 1.f : 0.f;
            }
    }
    __syncthreads();
    // the upper triangle was computed in a different summation order than the lower: symmetrise exactly
    for (int i = tid; i < P * P; i += kThreads) {
        const int r = i / P, c = i % P;
        if (r > c) S.G[r * kGs + c] = S.G[c * kGs + r];
    }
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

    // ---- cyclic Jacobi sweeps ----
    bool converged = false;
    for (int sweep = 0; sweep < geo.jacobi_max_sweeps && !converged; ++sweep) {
        int rotated = 0;
        for (int rho = 0; rho < P - 1; ++rho) {
            if (tid < P / 2) {
                int p, q;
                pair_of<P>(rho, tid, p, q);
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
            // columns p, q of G and Q:  x_p' = c x_p - s x_q,  x_q' = s x_p + c x_q
#pragma unroll
            for (int kk = 0; kk < Sh::kPairsPerWarp; ++kk) {
                const int k = warp + kk * kWarps;
                int p, q;
                pair_of<P>(rho, k, p, q);
                const float2 cs = S.cs[k];
                if (cs.y != 0.f) {
#pragma unroll
                    for (int half = 0; half < Sh::kHalves; ++half) {
                        const int i = lane + 32 * half;
                        if (i < P) {
                            float gp = S.G[i * kGs + p], gq = S.G[i * kGs + q];
                            S.G[i * kGs + p] = cs.x * gp - cs.y * gq;
                            S.G[i * kGs + q] = cs.y * gp + cs.x * gq;
                            float qp = S.Q[i * kGs + p], qq = S.Q[i * kGs + q];
                            S.Q[i * kGs + p] = cs.x * qp - cs.y * qq;
                            S.Q[i * kGs + q] = cs.y * qp + cs.x * qq;
                        }
                    }
                }
            }
            __syncthreads();
            // rows p, q of G
#pragma unroll
            for (int kk = 0; kk < Sh::kPairsPerWarp; ++kk) {
                const int k = warp + kk * kWarps;
                int p, q;
                pair_of<P>(rho, k, p, q);
                const float2 cs = S.cs[k];
                if (cs.y != 0.f) {
#pragma unroll
                    for (int half = 0; half < Sh::kHalves; ++half) {
                        const int j = lane + 32 * half;
                        if (j < P) {
                            float gp = S.G[p * kGs + j], gq = S.G[q * kGs + j];
                            S.G[p * kGs + j] = cs.x * gp - cs.y * gq;
                            S.G[q * kGs + j] = cs.y * gp + cs.x * gq;
                        }
                    }
                }
            }
            __syncthreads();
        }
        converged = !__syncthreads_or(rotated);
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

    // ---- A^T [r][P] = Q[:, order[:r]]^T as bf16, chunk-swizzled rows ----
    for (int i = tid; i < rank * (P / 2); i += kThreads) {
        const int j = i / (P / 2), tok = (i % (P / 2)) * 2;
        const int oj = S.order[j];
        const float a0 = S.Q[tok * kGs + oj], a1 = S.Q[(tok + 1) * kGs + oj];
        *reinterpret_cast<__nv_bfloat162 *>(dstA + a_t_offset(P, j, tok)) = __floats2bfloat162_rn(a0, a1);
    }
    // ---- B = A^T X (fp32 eigenvectors, exact page), rows swizzled like dense rows ----
    for (int i = tid; i < rank * (kHeadDim / 2); i += kThreads) {
        const int j = i / (kHeadDim / 2), col = (i % (kHeadDim / 2)) * 2;
        const int oj = S.order[j];
        float b0 = 0.f, b1 = 0.f;
#pragma unroll 8
        for (int r = 0; r < P; ++r) {
            const float a = S.Q[r * kGs + oj];
            const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&S.X[r * kXs + col]));
            b0 = fmaf(a, x.x, b0);
            b1 = fmaf(a, x.y, b1);
        }
        *reinterpret_cast<__nv_bfloat162 *>(dstB + j * kRowBytes + swz_chunk(j, col >> 3) * 16 + (col & 7) * 2) =
            __floats2bfloat162_rn(b0, b1);
    }
}

template <int P>
cudaError_t launch_p(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                     const int2 *worklist, int n_entries, int *status, cudaStream_t st) {
    static bool configured[64] = {};         // the attribute is per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(compress_kernel<P>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(CompressSmem<P>));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const unsigned grid = (unsigned)n_entries * geo.n_kv_heads * 2;
    compress_kernel<P><<<grid, Shape<P>::kThreads, sizeof(CompressSmem<P>), st>>>(geo, dense_pool, factor_pool,
                                                                                   worklist, status);
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
