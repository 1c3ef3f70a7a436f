// Row scatter for pkv_append_kv and the format translators behind
// pkv_read_factors / pkv_write_factors / pkv_read_dense.
#include "pkv_internal.h"

namespace pkv {

namespace {

// One thread moves one 16-byte chunk of one (token, KV head, K|V) row into the
// swizzled dense page.  Block 0 also publishes the new token counts.
// The descriptors come either from device memory (`desc_mem`) or, for small batches, inside the kernel's own
// parameters (`inl`), which saves the host-to-device copy that would otherwise precede every decode step's append.
struct AppendInline { AppendDesc d[kAppendInline]; };

__global__ void append_kernel(Geometry geo, unsigned char *dense_pool, const int *page_table, int *n_tokens,
                              const AppendDesc *desc_mem, const __grid_constant__ AppendInline inl, int n_seqs,
                              long long n_tok, int layer, const uint4 *k, const uint4 *v, int *status) {
    const AppendDesc *desc = desc_mem ? desc_mem : inl.d;
    const int H = geo.n_kv_heads;
    const long long total = n_tok * H * 2 * 16;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int chunk = (int)(idx & 15);
        long long rest = idx >> 4;
        const int kv = (int)(rest & 1);
        rest >>= 1;
        const int h = (int)(rest % H);
        const long long tok = rest / H;
        // entry whose token range holds `tok`
        int lo = 0, hi = n_seqs - 1;
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (desc[mid].tok_begin <= tok) lo = mid; else hi = mid - 1;
        }
        const AppendDesc e = desc[lo];
        const int t = e.t_start + (int)(tok - e.tok_begin);
        const int page = t / geo.page, row = t % geo.page;
        // a corrupt descriptor or page table: skip the row, leave a mark (checked before the table is indexed)
        const bool in_table = t >= 0 && page < geo.max_pages && e.seq >= 0 && e.seq < geo.max_seqs;
        const int slot = in_table ? page_table[((long long)e.seq * geo.n_layers + layer) * geo.max_pages + page] : -1;
        if (slot < 0 || slot >= geo.n_dense_slots) {
            if (chunk == 0 && kv == 0 && h == 0) atomicAdd(status + 2, 1);
            continue;
        }
        const uint4 val = (kv ? v : k)[(tok * H + h) * 16 + chunk];
        unsigned char *dst = dense_pool + (long long)slot * geo.dense_slot_bytes + (long long)h * geo.dense_head_bytes +
                             kv * (geo.page * kRowBytes) + row * kRowBytes + swz_chunk(row, chunk) * 16;
        *reinterpret_cast<uint4 *>(dst) = val;
    }
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < n_seqs; i += blockDim.x) {
            n_tokens[(long long)desc[i].seq * geo.n_layers + layer] = desc[i].t_start + desc[i].n_new;
        }
    }
}

// blob <-> row-major factors.  dir = 0: blob -> arrays (INT4 blobs are dequantised), 1: arrays -> blob (bf16
// blobs only).  The caller's A is [P][r] row-major; the blob holds A^T with swizzled chunks, and B rows with
// the dense-row swizzle.
__global__ void factor_io_kernel(Geometry geo, unsigned char *blob, unsigned short *A_k, unsigned short *B_k,
                                 unsigned short *A_v, unsigned short *B_v, int dir) {
    const int P = geo.page, rk = geo.rank_k, rv = geo.rank_v;
    // (Global SVD form: a page stores only its A rows)
    const int nAk = P * rk, nBk = geo.global_rank ? 0 : rk * kHeadDim, nAv = P * rv, nBv = geo.global_rank ? 0 : rv * kHeadDim;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nAk + nBk + nAv + nBv; i += gridDim.x * blockDim.x) {
        unsigned short *plain;
        int which, r, e, off;
        if (i < nAk) {
            which = 0; r = i % rk; e = i / rk; plain = A_k + i;
            off = geo.ak_off + a_t_offset(P, r, e);
        } else if (i < nAk + nBk) {
            const int j = i - nAk;
            which = 1; r = j / kHeadDim; e = j % kHeadDim; plain = B_k + j;
            off = geo.bk_off + r * kRowBytes + swz_chunk(r, e >> 3) * 16 + (e & 7) * 2;
        } else if (i < nAk + nBk + nAv) {
            const int j = i - nAk - nBk;
            which = 2; r = j % rv; e = j / rv; plain = A_v + j;
            off = geo.av_off + a_t_offset(P, r, e);
        } else {
            const int j = i - nAk - nBk - nAv;
            which = 3; r = j / kHeadDim; e = j % kHeadDim; plain = B_v + j;
            off = geo.bv_off + r * kRowBytes + swz_chunk(r, e >> 3) * 16 + (e & 7) * 2;
        }
        if (dir == 0) *plain = (unsigned short)(__float_as_uint(blob_value(geo, blob, which, r, e)) >> 16);
        else *reinterpret_cast<unsigned short *>(blob + off) = *plain;
    }
}

__global__ void dense_read_kernel(int P, const unsigned char *head_base, unsigned short *K, unsigned short *V) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 2 * P * kHeadDim; i += gridDim.x * blockDim.x) {
        int kv = i / (P * kHeadDim), j = i % (P * kHeadDim), row = j / kHeadDim, col = j % kHeadDim;
        const unsigned short *src = reinterpret_cast<const unsigned short *>(
                                        head_base + kv * (P * kRowBytes) + row * kRowBytes +
                                        swz_chunk(row, col >> 3) * 16) + (col & 7);
        (kv ? V : K)[j] = *src;
    }
}

}  // namespace

cudaError_t launch_append(const Geometry &geo, unsigned char *dense_pool, const int *page_table,
                          int *n_tokens, const AppendDesc *desc, const AppendDesc *host_desc, int n_seqs,
                          long long n_tok, int layer, const void *k, const void *v, int *status, cudaStream_t st) {
    const long long total = n_tok * geo.n_kv_heads * 2 * 16;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    if (blocks < 1) blocks = 1;
    AppendInline inl = {};
    if (host_desc) {
        for (int i = 0; i < n_seqs; ++i) inl.d[i] = host_desc[i];
    }
    append_kernel<<<(unsigned)blocks, threads, 0, st>>>(geo, dense_pool, page_table, n_tokens, host_desc ? nullptr : desc,
                                                        inl, n_seqs, n_tok, layer, (const uint4 *)k, (const uint4 *)v,
                                                        status);
    return cudaGetLastError();
}

cudaError_t launch_read_factors(const Geometry &geo, const unsigned char *blob, void *A_k, void *B_k,
                                void *A_v, void *B_v, cudaStream_t st) {
    factor_io_kernel<<<8, 256, 0, st>>>(geo, const_cast<unsigned char *>(blob), (unsigned short *)A_k,
                                        (unsigned short *)B_k, (unsigned short *)A_v, (unsigned short *)B_v, 0);
    return cudaGetLastError();
}

cudaError_t launch_write_factors(const Geometry &geo, unsigned char *blob, const void *A_k, const void *B_k,
                                 const void *A_v, const void *B_v, cudaStream_t st) {
    factor_io_kernel<<<8, 256, 0, st>>>(geo, blob, (unsigned short *)const_cast<void *>(A_k),
                                        (unsigned short *)const_cast<void *>(B_k),
                                        (unsigned short *)const_cast<void *>(A_v),
                                        (unsigned short *)const_cast<void *>(B_v), 1);
    return cudaGetLastError();
}

cudaError_t launch_read_dense(const Geometry &geo, const unsigned char *head_base, void *K, void *V,
                              cudaStream_t st) {
    dense_read_kernel<<<16, 256, 0, st>>>(geo.page, head_base, (unsigned short *)K, (unsigned short *)V);
    return cudaGetLastError();
}

}  // namespace pkv
