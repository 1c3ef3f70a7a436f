// Internal declarations shared by the host cache manager and the CUDA kernels.
#pragma once

#include <cuda.h>            // CUtensorMap (the type only: no driver call is linked)
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
constexpr int kStatusWords = 8;        // [0] device timeouts, [1] page SVDs not converged, [2] slot indices out of range,
                                       // [4..5] Jacobi rounds executed (64-bit), [6..7] page SVDs run (64-bit)
constexpr int kCompressChunk = 8192;   // work-list entries per compression launch
constexpr int kMaxDecodeBuffers = 64;  // decode_overlap = 2: at most this many rotating sets of split-K scratch
constexpr long long kDecodeBufferBudget = 128LL << 20;   // ... and at most this many bytes of them (but at least 4 sets)
constexpr int kSmemBudget = 227 * 1024;
constexpr int kMergeFan = 8;           // partial states summed at a time by the cross-CTA merge (see flush_segment)
// Group states and tickets a launch with `n_flat` per-CTA state slots and `n_segs` segments may index.
inline long long merge_group_slots(long long n_flat, long long n_segs) { return n_flat / kMergeFan + n_segs + 2; }
constexpr int kTraceSlots = 16;        // 64-bit time stamps per CTA of a traced decode launch

// Sizes derived from a validated pkv_config.  Plain data: passed to kernels by value.
struct Geometry {
    int n_layers, n_kv_heads, n_q_heads, group;   // group = H_q / H_kv
    int page;                          // P
    int rank_k, rank_v;
    int rank_tiles;                    // ceil(rank / 8), the same for K and V
    int max_seqs, max_pages;
    int n_dense_slots, n_factor_slots;
    int sink_pages, recent_pages;
    // bf16 factor blob of one (slot, KV head): [A_k^T r_k x P][B_k r_k x d][A_v^T r_v x P][B_v r_v x d]
    int ak_off, bk_off, av_off, bv_off;
    int blob16_bytes;                  // size of the bf16 form
    int blob_bytes;                    // stored size of a blob in the factor pool (= blob16_bytes for bf16 factors)
    int factor_bits;                   // 16 or 4
    // Global SVD form (global_rank > 0): rank_k = rank_v = global_rank; a page's blob is [A_k^T r x P][A_v^T r x P]
    // (bk_off, bv_off unused); the basis of a (sequence, layer, KV head) is [B_k r x d][B_v r x d] bf16 with the
    // dense-row swizzle, basis_head_bytes in all, kept in the meta buffer.
    int global_rank, basis_head_bytes;
    // INT4 blobs: [codes of A~_K][codes of B~_K][codes of A~_V][codes of B~_V][bf16 scales: A~_K per rank column
    // (padded to 8), B~_K per channel, A~_V per token, B~_V per channel].  Codes are stored in the register order
    // of the mma operand each matrix is read as (see int4_a_pos / int4_b_pos).
    int cak_off, cbk_off, cav_off, cbv_off;                  // byte offsets of the four code regions
    int codes_bytes, sak_off, sbk_off, sav_off, sbv_off;     // scale offsets are relative to the scales' start
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
    long long plan_cta_entry;          // PlanEntry [n_ctas]: a copy of the entry each CTA's range starts in (saves a dependent load)
    long long append_desc;             // int4 [max_seqs]
    long long status;                  // int32 [kStatusWords]
    long long basis;                   // Global SVD form: bytes [max_seqs][n_layers][H_kv][basis_head_bytes]
    long long total;
};

struct WorkspaceLayout {
    int n_sets;                        // rotating sets of split-K scratch: 1 unless decode_overlap = 2
    long long partials;                // float [n_sets][n_partials][kPartialFloats]: per-CTA states, then group states
    long long n_partials;              // = n_flat + n_group
    long long n_flat, n_group, n_seg_tickets;
    long long partials_stride;         // bytes of one buffer
    long long tickets_stride;

    long long worklist;                // int2 [kCompressChunk]
    long long tickets;                 // int [n_sets][n_seg_tickets + n_group]: per segment, then per group
    long long gram;                    // Global SVD form: float [H_kv][2][d][d], the region Gram matrices of one (sequence, layer)
    long long trace;                   // long long [n_ctas][kTraceSlots]
    long long rb_partials;             // float [kRbSplitItems][128][kRbStateFloats]: states of row blocks split by token range (0 bytes if the tcgen05 kernel does not cover the shape)
    long long total;
};

struct AppendDesc { int seq, t_start, tok_begin, n_new; };
constexpr int kAppendInline = 64;      // descriptors of up to this many sequences are passed as kernel parameters

struct DecodeArgs {
    Geometry geo;
    const unsigned char *dense_pool, *factor_pool;
    const int *page_table;             // whole table
    const int *n_tokens;               // whole array
    const unsigned char *basis;        // Global SVD form: all bases (see MetaLayout::basis)
    const unsigned char *plan;         // this layer's plan
    long long plan_cta, plan_entry, plan_seg, plan_cta_entry;
    const void *q;
    void *out;
    float *out_f32;
    float *state;                      // not NULL: write (o unnormalised, m, l) rows of d + 2 floats instead of out / out_f32
    float *partials;
    int *tickets;                      // one per segment, zero between launches
    float *gpartials;                  // states of groups of kMergeFan CTAs (segments split over more CTAs than that)
    int *gtickets;                     // one per group, zero between launches

    // Queries per sequence (1 = decoding).  A score tile has eight query columns: q_tpt = min(q_len, 8 / group)
    // consecutive query tokens fill q_cols = q_tpt * group of them, so a sequence has b = ceil(q_len / q_tpt) blocks of
    // query tokens.  The CTAs of a launch work in groups of q_group siblings on one plan range, one block each; a
    // sequence has ceil(b / q_group) plan entries (more than one only if b exceeds the grid), so block numbers run
    // over q_nblk = entries x q_group per sequence (those past b are empty).
    int q_len, q_tpt, q_nblk, q_group, q_cols;
    int *status;
    int layer;
    int variant;                       // 0 = tensor-core pipeline, 1 = scalar reference kernel
    int overlap;                       // 0 wait at entry, 1 wait before the first partial state is written, 2 never wait
    int plain_launch;                  // launch without programmatic serialization (drains the stream first)
    long long wait_clocks;             // limit of every in-kernel wait of the decode kernel (SM clocks)
    int drop_unit;                     // -1; test hook: CTA 0's producer never arms this unit (a wait must run out)
    long long *trace;                  // NULL, or [n_ctas][kTraceSlots] time stamps written by each CTA (debugging)
    // tcgen05 row-block kernel: CTAs per row block (each with its own range of the sequence; 1 = no split) and where
    // their states go
    int rb_splits;
    float *rb_partials;
};

// Launchers (defined in the .cu files); all return the launch error.
// desc: device copy of the descriptors; host_desc: if not NULL (and n_seqs <= kAppendInline) the descriptors travel in
// the kernel's parameters instead and `desc` is not read
cudaError_t launch_append(const Geometry &geo, unsigned char *dense_pool, const int *page_table,
                          int *n_tokens, const AppendDesc *desc, const AppendDesc *host_desc, int n_seqs,
                          long long n_tok, int layer, const void *k, const void *v, int *status, cudaStream_t st);
cudaError_t launch_compress(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                            const int2 *worklist, int n_entries, int *status, cudaStream_t st);
cudaError_t launch_decode(const DecodeArgs &a, int n_segs, cudaStream_t st);
// Row blocks split by token range: a state is d channels of o, then m and l, padded to 16-byte rows; at most
// kRbSplitItems CTAs per launch when split, at most kRbMaxSplits per row block, at least kRbMinPages pages per range.
constexpr int kRbStateFloats = kHeadDim + 4, kRbSplitItems = 512, kRbMaxSplits = 32, kRbMinPages = 8;
constexpr int kRowBlock = 64;          // query rows (token x query head) per CTA of the mma.sync row-block kernel
// tcgen05 row-block kernel (pkv_rowblock.cu): 128 query rows per CTA; bf16 page-wise factors
bool row_block_umma_supported(const Geometry &geo);
cudaError_t row_block_umma_setup();
// TMA descriptors of the pools for that kernel (B factors; dense K / V); valid = 0 where the shape is not covered or
// the driver offers no encoder, and the mma.sync kernel is used instead
// (bk[i], bv[i]: the factor pool from an origin 32 i bytes in - a B matrix may start on any 32-byte boundary of a 256-byte row)
struct RowBlockMaps { CUtensorMap bk[8], bv[8], dense; int valid; };
void row_block_make_maps(const Geometry &geo, const void *factor_pool, const void *dense_pool, RowBlockMaps *maps);
cudaError_t launch_decode_blocks_umma(const DecodeArgs &a, int n_seqs, const RowBlockMaps &maps, cudaStream_t st);
cudaError_t launch_decode_blocks(const DecodeArgs &a, int n_seqs, const RowBlockMaps &maps, cudaStream_t st);
cudaError_t launch_merge_states(const float *states, int n_shards, long long n_rows, void *out, float *out_f32,
                                cudaStream_t st);
cudaError_t launch_decode_static_scratch(const DecodeArgs &a, int n_segs, cudaStream_t st, const char **why);
cudaError_t launch_read_factors(const Geometry &geo, const unsigned char *blob, void *A_k, void *B_k,
                                void *A_v, void *B_v, cudaStream_t st);
cudaError_t launch_write_factors(const Geometry &geo, unsigned char *blob, const void *A_k, const void *B_k,
                                 const void *A_v, const void *B_v, cudaStream_t st);
cudaError_t launch_read_dense(const Geometry &geo, const unsigned char *head_base, void *K, void *V,
                              cudaStream_t st);
// Global SVD form (pkv_global.cu).  worklist: (dense slot, factor slot) of the pages of ONE (sequence, layer).
cudaError_t launch_region_basis(const Geometry &geo, const unsigned char *dense_pool, const int2 *worklist, int n_pages,
                                float *gram, unsigned char *basis_seq_layer, int *status, cudaStream_t st);
cudaError_t launch_project_pages(const Geometry &geo, const unsigned char *dense_pool, unsigned char *factor_pool,
                                 const int2 *worklist, int n_pages, const unsigned char *basis_seq_layer, int *status,
                                 cudaStream_t st);
cudaError_t launch_read_basis(const Geometry &geo, const unsigned char *basis_head, void *B_k, void *B_v, cudaStream_t st);
cudaError_t decode_kernel_setup();     // raises the dynamic shared-memory limit once per device
// Rotation order of the compression kernel for page size P (see pkv_get_rotation_schedule); false if P is unsupported
// or `cap` bytes are too few.
bool rotation_schedule(int P, unsigned char *out, long long cap, int *n_rounds, int *groups, int *group_size);

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

// ---- INT4 code layout -------------------------------------------------------------------------------------
// Codes are stored as code + 8 (1..15; 8 = zero) in the order in which the decode kernel's tensor-core
// instructions want their operands, so that a lane turns one 32-bit word into four operand registers without a
// shared-memory round trip.  An operand register holds two bf16 values; a lane (g = lane >> 2, c = lane & 3)
// numbers the registers it needs from one matrix n = 0, 1, ...; register n lives in the lane's word n >> 2 at
// nibbles t and t + 4 (t = n & 3, low and high half), so that (word >> 4t) & 0x000F000F is the pair.  Word w
// of lane l sits at 32-bit index 32 w + l of the matrix's code region.  NT = ceil(rank / 8); ranks up to 8 NT
// are stored, the ones past the true rank as zeros.
//   "A-type" (m16 x k16 row operand; rows m = tokens of A~_K or channels of B~_V, contraction over ranks):
//       16-row tile i = m >> 4 owns registers i * 2NT ...: per 16-rank step four, (rows g, g+8) x (ranks 2c, 2c+8),
//       then two for a last 8-rank step.
//   "B-type" (k16 x n8 col operand; contraction index k = channels of B~_K or tokens of A~_V, columns = ranks):
//       rank tile j owns registers j * (K/8) ...: register 2 kk + b holds k = 16 kk + 8 b + 2c (+1), rank 8 j + g.
__host__ __device__ inline int int4_a_words(int M, int NT) { return (((M / 16) * 2 * NT + 3) / 4) * 32; }
__host__ __device__ inline int int4_b_words(int K, int NT) { return ((NT * (K / 8) + 3) / 4) * 32; }
// element (row m, rank r) -> 32-bit word index and bit shift of its nibble
__host__ __device__ inline void int4_a_pos(int NT, int m, int r, int &word, int &shift) {
    const int i = m >> 4, q0 = (m >> 3) & 1, g = m & 7, full = NT / 2;
    int e, c;
    if (r < 16 * full) { e = 4 * (r >> 4) + 2 * ((r >> 3) & 1) + q0; c = (r & 7) >> 1; }
    else               { e = 4 * full + q0; c = (r - 16 * full) >> 1; }
    const int n = i * 2 * NT + e;
    word = (n >> 2) * 32 + 4 * g + c;
    shift = 4 * ((n & 3) + 4 * (r & 1));
}
__host__ __device__ inline void int4_b_pos(int K, int k, int r, int &word, int &shift) {
    const int n = (r >> 3) * (K / 8) + 2 * (k >> 4) + ((k >> 3) & 1);
    word = (n >> 2) * 32 + 4 * (r & 7) + ((k & 7) >> 1);
    shift = 4 * ((n & 3) + 4 * (k & 1));
}
// the inverse: half h of register n of `lane` -> (m, r) / (k, r); false past the last register
__host__ __device__ inline bool int4_a_elem(int M, int NT, int lane, int n, int h, int &m, int &r) {
    if (n >= (M / 16) * 2 * NT) return false;
    const int i = n / (2 * NT), e = n % (2 * NT), g = lane >> 2, c = lane & 3, full = NT / 2;
    if (e < 4 * full) { m = 16 * i + 8 * (e & 1) + g; r = 16 * (e >> 2) + 8 * ((e >> 1) & 1) + 2 * c + h; }
    else              { m = 16 * i + 8 * (e - 4 * full) + g; r = 16 * full + 2 * c + h; }
    return true;
}
__host__ __device__ inline bool int4_b_elem(int K, int NT, int lane, int n, int h, int &k, int &r) {
    if (n >= NT * (K / 8)) return false;
    const int j = n / (K / 8), rem = n % (K / 8), g = lane >> 2, c = lane & 3;
    r = 8 * j + g;
    k = 16 * (rem >> 1) + 8 * (rem & 1) + 2 * c + h;
    return true;
}

#ifdef __CUDACC__
// Value of one factor element as attention reads it.  which: 0 = A_k(r, token i), 1 = B_k(r, channel i),
// 2 = A_v(r, token i), 3 = B_v(r, channel i).  bf16 factors are read as stored; INT4 factors are
// bf16(code * scale) with the scale of the element's column or row (see Geometry).
__device__ inline float blob_value(const Geometry &g, const unsigned char *blob, int which, int r, int i) {
    const int P = g.page;
    if (g.factor_bits != 4) {
        int off;
        if (which == 0) off = g.ak_off + a_t_offset(P, r, i);
        else if (which == 2) off = g.av_off + a_t_offset(P, r, i);
        else off = (which == 1 ? g.bk_off : g.bv_off) + r * kRowBytes + swz_chunk(r, i >> 3) * 16 + (i & 7) * 2;
        const unsigned short raw = *reinterpret_cast<const unsigned short *>(blob + off);
        return __uint_as_float((unsigned)raw << 16);
    }
    int w, shift, region;
    if (which == 0)      { int4_a_pos(g.rank_tiles, i, r, w, shift); region = g.cak_off; }
    else if (which == 1) { int4_b_pos(kHeadDim, i, r, w, shift);     region = g.cbk_off; }
    else if (which == 2) { int4_b_pos(P, i, r, w, shift);            region = g.cav_off; }
    else                 { int4_a_pos(g.rank_tiles, i, r, w, shift); region = g.cbv_off; }
    const unsigned word = reinterpret_cast<const unsigned *>(blob + region)[w];
    const int code = (int)((word >> shift) & 0xFu) - 8;
    const int soff = which == 0 ? g.sak_off + 2 * r : which == 1 ? g.sbk_off + 2 * i
                   : which == 2 ? g.sav_off + 2 * i : g.sbv_off + 2 * i;
    const unsigned short sraw = *reinterpret_cast<const unsigned short *>(blob + g.codes_bytes + soff);
    const float v = (float)code * __uint_as_float((unsigned)sraw << 16);
    unsigned u = __float_as_uint(v);           // round to bf16, ties to even (v is finite)
    u += 0x7fffu + ((u >> 16) & 1u);
    return __uint_as_float(u & 0xffff0000u);
}
#endif

}  // namespace pkv
