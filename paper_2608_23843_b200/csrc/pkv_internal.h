// Internal declarations shared by the host cache manager and the CUDA kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "pkv.h"

namespace pkv {

constexpr int kHeadDim = 128;          // d (only supported value)
constexpr int kMaxPage = 64;           // P is 16, 32 or 64
constexpr int kRowBytes = kHeadDim * 2;
constexpr int kMaxGroup = 8;           // query heads per KV head handled by the tensor-core kernel
constexpr int kConsumerWarps = 5;      // decode kernel: warps that compute (two CTAs share an SM; 6 warps x 168 regs x 2 fit the register file)
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;
constexpr int kPartialFloats = kMaxGroup * (kHeadDim + 2);   // o[8][128], m[8], l[8]
constexpr int kStatusWords = 8;        // [0] device timeouts, [1] page SVDs not converged, [2] slot indices out of range
constexpr int kCompressChunk = 8192;   // work-list entries per compression launch
constexpr int kDecodeBuffers = 16;     // decode_overlap = 2: rotating sets of split-K scratch (see pkv_decode_attention)
constexpr int kSmemBudget = 227 * 1024;

// Sizes derived from a validated pkv_config.  Plain data: passed to kernels by value.
struct Geometry {
    int n_layers, n_kv_heads, n_q_heads, group;   // group = H_q / H_kv
    int page;                          // P
    int rank_k, rank_v;
    int rank_tiles;                    // ceil(rank / 8), the same for K and V
    int max_seqs, max_pages;
    int n_dense_slots, n_factor_slots;
    int sink_pages, recent_pages;
    // factor blob of one (slot, KV head): [A_k^T r_k x P][B_k r_k x d][A_v^T r_v x P][B_v r_v x d], bf16
    int ak_off, bk_off, av_off, bv_off, blob_bytes;
    int dense_head_bytes;              // [K P x d][V P x d] of one KV head = 2*P*d*2
    long long dense_slot_bytes, factor_slot_bytes;
    // decode work units: a factor page, or a block of `block_tokens` rows of a dense page
    int block_tokens, blocks_per_page, stage_bytes, n_stages;
    int n_ctas;
    float scale_log2e;                 // softmax_scale * log2(e)
    int jacobi_max_sweeps;
    float jacobi_tol;
    float jacobi_energy_tol;           // < 0: off
};

// Device-resident decode plan of one layer (written by the host when the batch
// or a page table changes, read by every decode launch).
struct PlanHeader { int n_seqs, n_used_ctas, n_segs, total_units; };
struct PlanCta    { int entry, head, unit, pad; };          // first unit of a CTA's range
struct PlanEntry  { int seq, n_pages, f_begin, f_end; };    // pages [f_begin, f_end) are factor pages
struct PlanSeg    { int cta_first, n_parts; };              // CTAs holding partial states of (entry, head)

struct MetaLayout {                    // byte offsets inside the caller's `meta` buffer
    long long page_table;              // int32 [max_seqs][n_layers][max_pages]
    long long n_tokens;                // int32 [max_seqs][n_layers]
    long long plans;                   // n_layers * plan_stride
    long long plan_stride;
    long long plan_cta, plan_entry, plan_seg;   // offsets inside one plan
    long long append_desc;             // int4 [max_seqs]
    long long status;                  // int32 [kStatusWords]
    long long total;
};

struct WorkspaceLayout {
    long long partials;                // float [kDecodeBuffers][n_partials][kPartialFloats]
    long long n_partials;
    long long partials_stride;         // bytes of one buffer
    long long tickets_stride;

    long long worklist;                // int2 [kCompressChunk]
    long long tickets;                 // int [max_seqs * n_kv_heads]
    long long trace;                   // long long [n_ctas][8]
    long long total;
};

struct AppendDesc { int seq, t_start, tok_begin, n_new; };

struct DecodeArgs {
    Geometry geo;
    const unsigned char *dense_pool, *factor_pool;
    const int *page_table;             // whole table
    const int *n_tokens;               // whole array
    const unsigned char *plan;         // this layer's plan
    long long plan_cta, plan_entry, plan_seg;
    const void *q;
    void *out;
    float *out_f32;
    float *partials;
    int *tickets;                      // one per segment, zero between launches

    int *status;
    int layer;
    int variant;                       // 0 = tensor-core pipeline, 1 = scalar reference kernel
    int overlap;                       // 0 wait at entry, 1 wait before the first partial state is written, 2 never wait
    int plain_launch;                  // launch without programmatic serialization (drains the stream first)
    long long *trace;                  // NULL, or [n_ctas][8] time stamps written by each CTA (debugging)
};

// Launchers (defined in the .cu files); all return the launch error.
cudaError_t launch_append(const Geometry &geo, unsigned char *dense_pool, const int *page_table,
                          int *n_tokens, const AppendDesc *desc, int n_seqs, long long n_tok, int layer,
                          const void *k, const void *v, int *status, cudaStream_t st);
cudaError_t launch_compress(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                            const int2 *worklist, int n_entries, int *status, cudaStream_t st);
cudaError_t launch_decode(const DecodeArgs &a, int n_segs, cudaStream_t st);
cudaError_t launch_decode_static_scratch(const DecodeArgs &a, int n_segs, cudaStream_t st, const char **why);
cudaError_t launch_read_factors(const Geometry &geo, const unsigned char *blob, void *A_k, void *B_k,
                                void *A_v, void *B_v, cudaStream_t st);
cudaError_t launch_write_factors(const Geometry &geo, unsigned char *blob, const void *A_k, const void *B_k,
                                 const void *A_v, const void *B_v, cudaStream_t st);
cudaError_t launch_read_dense(const Geometry &geo, const unsigned char *head_base, void *K, void *V,
                              cudaStream_t st);
cudaError_t decode_kernel_setup();     // raises the dynamic shared-memory limit once per device

// Storage swizzle of a 256-byte row: 16-byte chunk c of row `row` lives at
// chunk position c ^ (row & 7).  Applied to dense K/V rows and to B factors.
__host__ __device__ inline int swz_chunk(int row, int chunk) { return chunk ^ (row & 7); }

// A factors are stored transposed, [r][P]: rows of 2P bytes = P/8 chunks.  Eight consecutive rows must
// land in eight different 16-byte bank groups of a 128-byte window, so the chunk index is XORed with
// the row's position inside that window: P = 64 -> row & 7, P = 32 -> (row >> 1) & 3, P = 16 -> (row >> 2) & 1.
__host__ __device__ inline int swz_a_chunk(int P, int row, int chunk) {
    const int nch = P >> 3;
    return chunk ^ (((row * nch) >> 3) & (nch - 1));
}
// byte offset of element (row r, token i) inside an A^T matrix
__host__ __device__ inline int a_t_offset(int P, int r, int i) {
    return r * 2 * P + swz_a_chunk(P, r, i >> 3) * 16 + (i & 7) * 2;
}

}  // namespace pkv
