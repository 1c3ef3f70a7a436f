// The Global SVD form (paper: Section 4.1 "Baselines", Section 4.2): one truncated SVD per region - the pages of a
// (sequence, layer, KV head) converted together - instead of one per page.  Three kernels:
//   region_gram_kernel    G = X^T X (d x d, fp32, exact bf16 products) over the rows of the region's pages, in page order
//   region_eig_kernel     cyclic Jacobi eigen-solve of G in shared memory; B = the r eigenvectors of largest eigenvalue
//                         (r x d, orthonormal rows), rounded to bf16, written with the dense-row swizzle
//   project_pages_kernel  A = X_page B^T (P x r) per page, with the stored (rounded) B, written as A^T with the A swizzle
// The region is small work done once per sequence and layer; these kernels are plain and deterministic (no atomics:
// a region is summed by one CTA in page order), not tuned.
#include <cuda_bf16.h>

#include "pkv_internal.h"

namespace pkv {

namespace {

constexpr int kD = kHeadDim;                 // 128
constexpr int kEigThreads = 512;

// One CTA per (KV head, K|V): 512 threads, thread t owns the 4 x 8 tile (rows 4 (t / 16), columns 8 (t % 16)) of G.
__global__ void __launch_bounds__(512) region_gram_kernel(Geometry geo, const unsigned char *dense_pool,
                                                          const int2 *worklist, int n_pages, float *gram, int *status) {
    __shared__ float X[kMaxPage][kD + 1];
    const int head = blockIdx.x >> 1, kv = blockIdx.x & 1, tid = threadIdx.x, P = geo.page;
    const int i0 = 4 * (tid >> 4), j0 = 8 * (tid & 15);
    float acc[4][8] = {};
    for (int pg = 0; pg < n_pages; ++pg) {
        const int slot = worklist[pg].x;
        __syncthreads();
        if (slot < 0 || slot >= geo.n_dense_slots) {                   // corrupt work list: skip the page, leave a mark
            if (tid == 0) atomicAdd(status + 2, 1);
            continue;
        }
        const unsigned char *src = dense_pool + (long long)slot * geo.dense_slot_bytes +
                                   (long long)head * geo.dense_head_bytes + kv * (P * kRowBytes);
        for (int i = tid; i < P * 16; i += 512) {                      // undo the storage swizzle
            const int row = i >> 4, chunk = i & 15;
            const uint4 val = *reinterpret_cast<const uint4 *>(src + row * kRowBytes + swz_chunk(row, chunk) * 16);
            const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&val);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float2 f = __bfloat1622float2(h[u]);
                X[row][chunk * 8 + 2 * u] = f.x;
                X[row][chunk * 8 + 2 * u + 1] = f.y;
            }
        }
        __syncthreads();
        for (int p = 0; p < P; ++p) {
            float a[4], b[8];
#pragma unroll
            for (int u = 0; u < 4; ++u) a[u] = X[p][i0 + u];
#pragma unroll
            for (int w = 0; w < 8; ++w) b[w] = X[p][j0 + w];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int w = 0; w < 8; ++w) acc[u][w] = fmaf(a[u], b[w], acc[u][w]);
        }
    }
    float *G = gram + (long long)blockIdx.x * kD * kD;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int w = 0; w < 8; ++w) G[(i0 + u) * kD + j0 + w] = acc[u][w];
}

// Round-robin tournament over n = 128 indices: round rho (0 .. n-2), pair k (0 .. n/2-1) -> (p, q), p < q.
__device__ __forceinline__ void tournament_pair(int n, int rho, int k, int &p, int &q) {
    const int m = n - 1;
    int a, b;
    if (k == 0) { a = m; b = rho; }
    else { a = rho + k; if (a >= m) a -= m; b = rho - k; if (b < 0) b += m; }
    p = min(a, b); q = max(a, b);
}

// One CTA per (KV head, K|V).  Shared memory: G (d x d) and Q^T (d x d) in fp32, rows padded by one float.
// Every round rotates d/2 disjoint pairs: rows p, q of G and of Q^T first, then columns p, q of G.
__global__ void __launch_bounds__(kEigThreads) region_eig_kernel(Geometry geo, const float *gram, unsigned char *basis,
                                                                 int *status) {
    extern __shared__ __align__(16) float sm[];
    constexpr int kS = kD + 1;
    float *G = sm, *QT = sm + kD * kS;
    float2 *cs = reinterpret_cast<float2 *>(QT + kD * kS);       // [d/2]
    float *lam = reinterpret_cast<float *>(cs + kD / 2);          // [d]
    int *order = reinterpret_cast<int *>(lam + kD);               // [d]
    __shared__ int rotated;
    const int tid = threadIdx.x, r = geo.global_rank;
    const float *Gin = gram + (long long)blockIdx.x * kD * kD;
    for (int i = tid; i < kD * kD; i += kEigThreads) {
        const int row = i / kD, col = i % kD;
        // symmetrise: the two triangles were accumulated in different orders
        G[row * kS + col] = 0.5f * (Gin[row * kD + col] + Gin[col * kD + row]);
        QT[row * kS + col] = row == col ? 1.f : 0.f;
    }
    __syncthreads();
    const float tol = geo.jacobi_tol;
    bool converged = false;
    const int max_sweeps = 2 * geo.jacobi_max_sweeps;            // a 128 x 128 problem needs a few sweeps more than a page
    for (int sweep = 0; sweep < max_sweeps && !converged; ++sweep) {
        if (tid == 0) rotated = 0;
        __syncthreads();
        for (int rho = 0; rho < kD - 1; ++rho) {
            if (tid < kD / 2) {
                int p, q;
                tournament_pair(kD, rho, tid, p, q);
                const float gpp = G[p * kS + p], gqq = G[q * kS + q], gpq = G[p * kS + q];
                float c = 1.f, s = 0.f;
                // A rotation is skipped below the relative threshold, or below the rounding noise of the two rows
                // (2e-7 of the larger diagonal entry; a floor tied to the largest eigenvalue of all, as the page
                // kernel uses, is too coarse here: a region's spectrum spans four decades and the directions next
                // to the rank cut would be left turned by a few hundredths of a radian)
                if (fabsf(gpq) > 2e-7f * fmaxf(fabsf(gpp), fabsf(gqq)) && gpq * gpq > tol * tol * fabsf(gpp * gqq)) {
                    const float d = gqq - gpp;
                    const float h = sqrtf(fmaf(d, d, 4.f * gpq * gpq));
                    const float t = 2.f * gpq / (d + copysignf(h, d));
                    c = rsqrtf(fmaf(t, t, 1.f));
                    s = t * c;
                    rotated = 1;
                }
                cs[tid] = make_float2(c, s);
            }
            __syncthreads();
            // rows p, q of G and of Q^T:  x_p' = c x_p - s x_q,  x_q' = s x_p + c x_q
            for (int it = tid; it < (kD / 2) * kD; it += kEigThreads) {
                const int k = it / kD, col = it % kD;
                const float2 r2 = cs[k];
                if (r2.y == 0.f) continue;
                int p, q;
                tournament_pair(kD, rho, k, p, q);
                const float gp = G[p * kS + col], gq = G[q * kS + col];
                G[p * kS + col] = r2.x * gp - r2.y * gq;
                G[q * kS + col] = r2.y * gp + r2.x * gq;
                const float tp = QT[p * kS + col], tq = QT[q * kS + col];
                QT[p * kS + col] = r2.x * tp - r2.y * tq;
                QT[q * kS + col] = r2.y * tp + r2.x * tq;
            }
            __syncthreads();
            // columns p, q of G
            for (int it = tid; it < (kD / 2) * kD; it += kEigThreads) {
                const int k = it / kD, row = it % kD;
                const float2 r2 = cs[k];
                if (r2.y == 0.f) continue;
                int p, q;
                tournament_pair(kD, rho, k, p, q);
                const float gp = G[row * kS + p], gq = G[row * kS + q];
                G[row * kS + p] = r2.x * gp - r2.y * gq;
                G[row * kS + q] = r2.y * gp + r2.x * gq;
            }
            __syncthreads();
        }
        converged = rotated == 0;
        __syncthreads();
    }
    if (!converged && tid == 0) atomicAdd(status + 1, 1);
    // eigenvalues descending, ties by lower index
    if (tid < kD) lam[tid] = G[tid * kS + tid];
    __syncthreads();
    if (tid < kD) {
        const float li = lam[tid];
        int rank = 0;
        for (int j = 0; j < kD; ++j) rank += (lam[j] > li) || (lam[j] == li && j < tid);
        order[rank] = tid;
    }
    __syncthreads();
    // B rows = the leading eigenvectors (rows of Q^T), bf16, dense-row swizzle; this CTA's matrix is B_k or B_v
    unsigned char *dst = basis + (long long)(blockIdx.x >> 1) * geo.basis_head_bytes + (blockIdx.x & 1) * r * kRowBytes;
    for (int i = tid; i < r * (kD / 2); i += kEigThreads) {
        const int j = i / (kD / 2), col = (i % (kD / 2)) * 2;
        const float *row = QT + order[j] * kS;
        *reinterpret_cast<__nv_bfloat162 *>(dst + j * kRowBytes + swz_chunk(j, col >> 3) * 16 + (col & 7) * 2) =
            __floats2bfloat162_rn(row[col], row[col + 1]);
    }
}

// One CTA per (page of the work list, KV head, K|V): A = X B^T with the stored basis.
__global__ void __launch_bounds__(256) project_pages_kernel(Geometry geo, const unsigned char *dense_pool,
                                                            unsigned char *factor_pool, const int2 *worklist,
                                                            const unsigned char *basis, int *status) {
    extern __shared__ __align__(16) float sm[];
    const int P = geo.page, r = geo.global_rank, tid = threadIdx.x;
    float *X = sm;                                   // [P][d + 1]
    float *B = sm + P * (kD + 1);                    // [r][d + 1]
    const int kv = blockIdx.x & 1, head = (blockIdx.x >> 1) % geo.n_kv_heads, entry = (blockIdx.x >> 1) / geo.n_kv_heads;
    const int2 wk = worklist[entry];
    if (wk.x < 0 || wk.x >= geo.n_dense_slots || wk.y < 0 || wk.y >= geo.n_factor_slots) {
        if (tid == 0) atomicAdd(status + 2, 1);
        return;
    }
    const unsigned char *src = dense_pool + (long long)wk.x * geo.dense_slot_bytes + (long long)head * geo.dense_head_bytes +
                               kv * (P * kRowBytes);
    const unsigned char *bsrc = basis + (long long)head * geo.basis_head_bytes + kv * r * kRowBytes;
    for (int i = tid; i < (P + r) * 16; i += 256) {
        const bool is_x = i < P * 16;
        const int row = (is_x ? i : i - P * 16) >> 4, chunk = i & 15;
        const uint4 val = *reinterpret_cast<const uint4 *>((is_x ? src : bsrc) + row * kRowBytes + swz_chunk(row, chunk) * 16);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&val);
        float *dst = (is_x ? X : B) + row * (kD + 1) + chunk * 8;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 f = __bfloat1622float2(h[u]);
            dst[2 * u] = f.x;
            dst[2 * u + 1] = f.y;
        }
    }
    __syncthreads();
    unsigned char *blob = factor_pool + (long long)wk.y * geo.factor_slot_bytes + (long long)head * geo.blob_bytes +
                          (kv ? geo.av_off : geo.ak_off);
    for (int i = tid; i < r * (P / 2); i += 256) {
        const int j = i / (P / 2), tok = (i % (P / 2)) * 2;
        float a0 = 0.f, a1 = 0.f;
        const float *b = B + j * (kD + 1), *x0 = X + tok * (kD + 1), *x1 = x0 + (kD + 1);
#pragma unroll 8
        for (int c = 0; c < kD; ++c) { a0 = fmaf(x0[c], b[c], a0); a1 = fmaf(x1[c], b[c], a1); }
        *reinterpret_cast<__nv_bfloat162 *>(blob + a_t_offset(P, j, tok)) = __floats2bfloat162_rn(a0, a1);
    }
}

__global__ void read_basis_kernel(Geometry geo, const unsigned char *b, unsigned short *B_k, unsigned short *B_v) {
    const int r = geo.global_rank;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 2 * r * kD; i += gridDim.x * blockDim.x) {
        const int m = i / (r * kD), j = (i % (r * kD)) / kD, col = i % kD;
        const unsigned short raw = *reinterpret_cast<const unsigned short *>(b + m * r * kRowBytes + j * kRowBytes +
                                                                               swz_chunk(j, col >> 3) * 16 + (col & 7) * 2);
        (m ? B_v : B_k)[j * kD + col] = raw;
    }
}

size_t eig_smem_bytes() { return sizeof(float) * (2 * kD * (kD + 1) + kD + kD) + sizeof(int) * kD; }

}  // namespace

cudaError_t launch_region_basis(const Geometry &geo, const unsigned char *dense_pool, const int2 *worklist, int n_pages,
                                float *gram, unsigned char *basis_seq_layer, int *status, cudaStream_t st) {
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(region_eig_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)eig_smem_bytes());
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(project_pages_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(sizeof(float) * (kMaxPage + 96) * (kD + 1)));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    region_gram_kernel<<<geo.n_kv_heads * 2, 512, 0, st>>>(geo, dense_pool, worklist, n_pages, gram, status);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    region_eig_kernel<<<geo.n_kv_heads * 2, kEigThreads, eig_smem_bytes(), st>>>(geo, gram, basis_seq_layer, status);
    return cudaGetLastError();
}

cudaError_t launch_project_pages(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                                 const int2 *worklist, int n_pages, const unsigned char *basis_seq_layer, int *status,
                                 cudaStream_t st) {
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(project_pages_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(sizeof(float) * (kMaxPage + 96) * (kD + 1)));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const size_t smem = sizeof(float) * (geo.page + geo.global_rank) * (kD + 1);
    project_pages_kernel<<<(unsigned)n_pages * geo.n_kv_heads * 2, 256, smem, st>>>(geo, dense_pool, factor_pool, worklist,
                                                                                 basis_seq_layer, status);
    return cudaGetLastError();
}

cudaError_t launch_read_basis(const Geometry &geo, const unsigned char *basis_head, void *B_k, void *B_v, cudaStream_t st) {
    read_basis_kernel<<<16, 256, 0, st>>>(geo, basis_head, reinterpret_cast<unsigned short *>(B_k),
                                          reinterpret_cast<unsigned short *>(B_v));
    return cudaGetLastError();
}

}  // namespace pkv
