/*
 * pkv.h — C ABI of the PuzzleKV decode hot path for NVIDIA B200 (sm_100a).
 *
 * What the library does (paper: Section 3.3).  Each (layer, KV head) of a
 * sequence is split into pages of P tokens.  The sink pages and a moving window
 * of recent pages are kept as dense bf16 rows; every other completed page is
 * replaced, once, by its rank-r truncated-SVD factors (Eq. 2)
 *        K_page ~= A_k B_k,  V_page ~= A_v B_v,   A: P x r,  B: r x d,
 * (A is the paper's L, B the paper's R).  Decode attention (Eq. 4, Eq. 5)
 * evaluates factor pages straight from the factors and merges all pages with an
 * online softmax; historical K/V is never rebuilt.
 *
 * Entry points: the paper's path is pkv_init_cache, pkv_append_kv,
 * pkv_compress_eligible_pages, pkv_decode_attention.  Around it: the same attention
 * for several new positions per sequence (pkv_decode_attention_multi), from host
 * buffers (pkv_decode_attention_host), without a workspace
 * (pkv_decode_attention_static_scratch), as a softmax state for sequences sharded
 * over caches (pkv_decode_attention_partial, pkv_merge_attention_states); the
 * compression in two steps on a side stream (pkv_compress_begin,
 * pkv_compress_commit); inspection and test access (pkv_get_*, pkv_read_*,
 * pkv_write_factors).
 *
 * Conventions
 *  - Every function returns a pkv_status (0 = PKV_OK, negative = error).  No
 *    exception or abort crosses this boundary.  pkv_last_error() gives a
 *    message for the most recent failure on that cache.
 *  - Ownership: the caller allocates every device buffer and passes raw device
 *    pointers; pkv_query_sizes() says how large each must be.  The library owns
 *    only host-side metadata (page tables, free lists, a pinned staging ring)
 *    and never allocates or frees device memory.  Buffers must stay valid until
 *    pkv_destroy_cache().
 *  - Pointers marked [device] are device addresses on the current CUDA device,
 *    [host] are ordinary host addresses.  bf16 = IEEE bfloat16 bit pattern.
 *  - Alignment of caller buffers (checked on the host; PKV_ERR_INVALID_ARG, nothing
 *    launched): k and v 16 bytes, q 4, out 8, out_f32 16, state 8.  Contiguous
 *    tensors from any allocator satisfy this; a view at an odd element offset may not.
 *  - All device work is enqueued on the `stream` argument (a cudaStream_t passed
 *    as void*); calls are asynchronous unless stated.  Operations on one cache
 *    must be issued on one stream (or the caller orders the streams); the one
 *    exception is pkv_compress_begin(), which takes a second stream by design.
 *  - One cache object is not thread-safe; use one host thread per cache.
 *  - Supported shapes: head_dim = 128; page_size 16, 32 or 64; 1 <= rank_k,
 *    rank_v <= min(32, page_size) with ceil(rank_k / 8) == ceil(rank_v / 8)
 *    (e.g. the paper's default P = 32, (r_K, r_V) = (16, 14)); 1 <= n_q_heads /
 *    n_kv_heads <= 8.  Anything else returns PKV_ERR_UNSUPPORTED from
 *    pkv_init_cache().
 *  - Dry-run mode: if dense_pool, factor_pool, meta and workspace are all NULL
 *    in pkv_init_cache(), no CUDA call is ever made; append / compress /
 *    free_seq update the page tables exactly as they would with device buffers
 *    (k, v, q, out may then be NULL) and pkv_decode_attention() only validates
 *    its arguments.  Useful for capacity planning.
 */
#ifndef PKV_H
#define PKV_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pkv_cache pkv_cache;
typedef int32_t pkv_status;

#define PKV_OK                   0
#define PKV_ERR_INVALID_ARG     (-1)  /* bad pointer, size, layer, count, or an empty sequence in attention */
#define PKV_ERR_POOL_EXHAUSTED  (-2)  /* no free dense / factor slot, or a sequence exceeds max_pages_per_seq; state unchanged */
#define PKV_ERR_BAD_SEQ         (-3)  /* sequence id outside [0, max_seqs) or repeated within one call */
#define PKV_ERR_CUDA            (-4)  /* a CUDA runtime call failed; message holds cudaGetErrorString */
#define PKV_ERR_NOT_CONVERGED   (-5)  /* reported by pkv_get_stats users: some page hit the Jacobi sweep cap (factors still written) */
#define PKV_ERR_UNSUPPORTED     (-6)  /* shape outside the supported set; a call that cannot be recorded while its stream is capturing a CUDA graph; or a call that would interfere with a compression begun and not yet committed */
#define PKV_ERR_DEVICE_TIMEOUT  (-7)  /* a bounded in-kernel wait gave up (seen via pkv_get_stats); results of that call are invalid */

#define PKV_KIND_DENSE  0
#define PKV_KIND_FACTOR 1

typedef struct pkv_config {
    int32_t n_layers;
    int32_t n_kv_heads;         /* H_kv */
    int32_t n_q_heads;          /* H_q, a multiple of H_kv; query head h reads KV head h / (H_q/H_kv) */
    int32_t head_dim;           /* d */
    int32_t page_size;          /* P tokens per page */
    int32_t rank_k, rank_v;     /* r_K, r_V of Eq. 2 */
    int32_t sink_tokens;        /* S, multiple of P: the first S tokens stay dense for ever */
    int32_t recent_tokens;      /* W, multiple of P: the W/P most recently completed pages and the incomplete page stay dense */
    int32_t max_seqs;           /* sequence ids are 0 .. max_seqs-1 */
    int32_t max_pages_per_seq;  /* ceil(max context / P) */
    int64_t n_dense_slots;      /* pool capacities; one slot = one logical page of one layer, all KV heads */
    int64_t n_factor_slots;
    float   softmax_scale;      /* 0 => 1/sqrt(head_dim)  (Eq. 1) */
    int32_t jacobi_max_sweeps;  /* 0 => default (16) */
    float   jacobi_tol;         /* 0 => default; rotation skipped when |g_pq| <= tol*sqrt(g_pp*g_qq) */
    int32_t n_ctas;             /* decode grid size; 0 => SM count of the current device (148 in dry-run), doubled unless decode_overlap */
    int32_t decode_variant;     /* 0 = tensor-core kernels (the product path); 1 = scalar fp32 kernel that evaluates
                                   the same equations one unit at a time, kept as a debugging reference; 2 = as 0 but
                                   pkv_decode_attention_multi never uses its row-block kernels; 3 = as 0 but the
                                   row-block kernel is the mma.sync one for every shape (2, 3: for comparisons) */
    float   jacobi_energy_tol;  /* the sweeps also stop once the energy captured by the r largest diagonal entries
                                   (= ||A^T X||_F^2 of the factors they would give) has grown, since the previous
                                   check, by less than this fraction of the energy left outside them (= the squared
                                   reconstruction error): the remaining rotations only polish eigenvectors inside
                                   near-degenerate clusters and cannot improve A B measurably.  Checked about three
                                   times per sweep for page sizes 32 and 64, once per sweep for 16; not applied at
                                   full rank (r = P), where it would say nothing.  0 => default 1e-4 (3e-3 would save 16 % of
                                   the rotation rounds and moves typical pages by 0.2 % of the optimum, but rank-8 pages
                                   with outlier rows then miss the factor gate by up to 16 %); negative => off
                                   (iterate until no rotation exceeds jacobi_tol) */
    int32_t factor_bits;        /* 0 or 16: factors stored in bf16.  4: INT4 factors (Section 4.3): the singular
                                   values are split evenly, A~ = A Sigma^(1/2), B~ = Sigma^(-1/2) B, and each matrix is
                                   quantized symmetrically to 4 bits with one bf16 scale per column of A~_K, B~_K and
                                   B~_V and per row (token) of A~_V; scale = max|x|/7, codes in [-7, 7].  Attention
                                   reads bf16(code * scale).  pkv_read_factors returns those dequantised values;
                                   pkv_write_factors is not available in this mode. */
    int32_t decode_overlap;     /* pkv_decode_attention is launched with programmatic stream serialization, so its
                                   CTAs start as SMs free up.
                                   0 (default): the kernel waits for the preceding kernel on the stream to finish
                                      before it reads q or writes anything.  Pages of the cache are already
                                      streamed into shared memory while that kernel finishes: only this library's
                                      own calls write the pools, and a decode call that follows one of them is
                                      launched the ordinary way (see the last paragraph).
                                   1: the caller promises that the kernel enqueued just before each
                                      pkv_decode_attention call writes neither this cache's pools nor q (typical:
                                      the previous layer's decode with queries prepared in advance).  The kernel
                                      streams pages at once and waits for the preceding kernel only before it
                                      touches its shared workspace and `out`; launches complete in order.
                                   2: the same promise for ALL decode launches that may be in flight, and `out`
                                      buffers of consecutive calls must be distinct (or hold the same values).
                                      Launches never wait for one another and may complete out of order; the
                                      library rotates the split-K scratch over n sets (n = 64, fewer where 64 sets
                                      would exceed 128 MiB of workspace, at least 4) and makes every (n-1)-th
                                      launch an ordinary one, which starts only after all earlier work on the
                                      stream has finished.  May be recorded into CUDA graphs (see
                                      pkv_decode_attention).
                                   Work enqueued after a decode call by any other means (another kernel, a copy)
                                   still starts only after that call has completed, in every mode, and a decode
                                   call that follows a pkv_append_kv, pkv_compress_eligible_pages,
                                   pkv_compress_commit or pkv_write_factors call on this cache always waits for
                                   it, in every mode: the promise concerns other writers (of q, or of the pools
                                   through their raw pointers, which no mode allows while decode calls are in
                                   flight) only. */
    int32_t global_rank;        /* 0: the paper's page-wise factors.  64, 80 or 96: the Global SVD form the paper
                                   compares with (Section 4.1 "Baselines", Section 4.2), as a second workload of
                                   the same decode kernel: each (sequence, layer, KV head) gets ONE basis B_k and
                                   one B_v (global_rank x d, orthonormal rows: the leading right singular vectors
                                   of the rows of all pages converted by the first compression of that sequence
                                   and layer - its region), and every factor page stores only its token rows
                                   A = X_page B^T (P x global_rank, for K and for V); pages converted later are
                                   projected on the same basis.  Attention computes q~ = B_k q once per (sequence,
                                   KV head) and CTA instead of once per page, streams only the A rows, keeps the
                                   weighted sum in rank space and applies B_v once at the end.  rank_k and rank_v
                                   are ignored (the paper's 76-78 rounds up to 80).  Needs page_size 32 or 64,
                                   bf16 factors, decode_variant 0; pkv_decode_attention_multi,
                                   pkv_compress_begin and pkv_write_factors return PKV_ERR_UNSUPPORTED. */
} pkv_config;

typedef struct pkv_sizes {
    int64_t dense_slot_bytes;   /* H_kv * 2 * P * d * 2 */
    int64_t factor_slot_bytes;  /* bf16 factors: H_kv * 2 * (r_k + r_v) * (P + d) bytes, so that Eq. 3 is
                                   factor_slot_bytes / dense_slot_bytes; INT4 factors, with R_k, R_v = the ranks
                                   rounded up to multiples of 8 (zero codes fill the rest):
                                   H_kv * ((R_k + R_v)(P + d)/2 + 2 * (R_k + 2d + P)) bytes, each KV head's part
                                   rounded up to 16 */
    int64_t dense_pool_bytes;   /* n_dense_slots * dense_slot_bytes */
    int64_t factor_pool_bytes;
    int64_t meta_bytes;         /* device page tables, token counts, decode plans, status words; with global_rank
                                   also the bases: max_seqs * n_layers * H_kv * 2 * global_rank * d * 2 bytes */
    int64_t workspace_bytes;    /* split-K partial states, merge tickets, compression work list; where the tcgen05
                                   row-block kernel applies (see pkv_decode_attention_multi), 34.6 MB for the states of
                                   row blocks cut into token ranges */
} pkv_sizes;

typedef struct pkv_stats {
    int64_t dense_slots_in_use;
    int64_t factor_slots_in_use;
    int64_t pages_compressed;        /* logical pages (one layer, all KV heads) converted so far */
    int64_t page_svds_not_converged; /* K or V pages whose Jacobi iteration hit the sweep cap */
    int64_t device_timeouts;         /* bounded in-kernel waits that gave up (must be 0) */
    int64_t bad_slot_indices;        /* page-table entries outside the pools met by a kernel (skipped; must be 0) */
    int64_t last_decode_bytes;       /* algorithmic HBM bytes of the most recent pkv_decode_attention call:
                                        factor blobs + valid dense rows + q + out */
    int64_t last_decode_units;       /* work units (factor pages + dense blocks) of that call */
    int64_t page_svds;               /* K or V pages of one KV head factorized so far (Eq. 2, one SVD each) */
    int64_t jacobi_rounds;           /* rotation rounds those SVDs took in total.  A round rotates P/2 disjoint pairs
                                        (page size 16: P - 1 rounds per sweep) or P/4 disjoint groups of four indices,
                                        six pairs each (page size 64: 21 rounds per sweep, 32: 13); see
                                        pkv_get_rotation_schedule() */
} pkv_stats;

/* Sizes of the caller-allocated buffers for a configuration.  Validates cfg. */
pkv_status pkv_query_sizes(const pkv_config *cfg, pkv_sizes *out);

/*
 * Section 3.3 "Page-Wise Low-Rank KV Cache Construction": creates an empty
 * hybrid cache over caller-owned storage.
 *   dense_pool, factor_pool, meta, workspace  [device] buffers of at least the
 *       sizes from pkv_query_sizes(), 256-byte aligned.  Contents need not be
 *       initialised; meta and workspace are initialised here (synchronously).
 *   dense_slot_order, factor_slot_order  [host] permutations of
 *       0..n_*_slots-1 giving the order in which physical slots are handed out
 *       (a shuffled physical pool); NULL = identity.  A released slot is reused
 *       (last released first) before the order array is consumed further.
 *   out  receives the cache handle.
 * The storage format inside the pools is private (A factors are stored
 * transposed, and all rows carry a 16-byte-chunk XOR swizzle, so that a page can
 * be copied linearly into shared memory and read without bank conflicts); use
 * pkv_read_* / pkv_write_factors to look inside.
 */
pkv_status pkv_init_cache(const pkv_config *cfg, void *dense_pool, void *factor_pool,
                          void *meta, void *workspace,
                          const int32_t *dense_slot_order, const int32_t *factor_slot_order,
                          pkv_cache **out);

/*
 * Section 3.3 "Incremental Cache Update": appends new key/value rows to the
 * current dense page of each listed sequence in one layer; a new dense slot is
 * taken at each page boundary.  The rows take part in the next attention call.
 *   seq_ids [host] n_seqs distinct ids;  n_new [host] tokens per sequence (>= 0)
 *   k, v    [device] bf16 [sum(n_new), H_kv, d], tokens of seq_ids[0] first.
 * Token counts are kept per (sequence, layer); this call advances `layer` only.
 * On PKV_ERR_POOL_EXHAUSTED nothing has been appended.
 */
pkv_status pkv_append_kv(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                         const int32_t *n_new, const void *k, const void *v, void *stream);

/*
 * Section 3.3, Eq. 2 and the Gram-matrix route described after Eq. 3: converts
 * every eligible page of `layer` (-1 = all layers) to factors.  A page p of a
 * sequence with T tokens is eligible iff S/P <= p < floor(T/P) - W/P and it is
 * still dense.  Pages are taken in ascending (sequence, layer, page) order; for
 * each, a factor slot is allocated, the K and V page of every KV head are
 * factorized on the GPU (G = X X^T in fp32, cyclic Jacobi eigen-solve in shared
 * memory, A = top-r eigenvectors, B = A^T X, both rounded to bf16), then the
 * dense slot is released.  Factor pages are never revisited.
 *   n_pages_compressed [host, may be NULL] logical pages converted by this call.
 * If the factor pool runs out, the pages converted so far stay converted and
 * PKV_ERR_POOL_EXHAUSTED is returned.
 */
pkv_status pkv_compress_eligible_pages(pkv_cache *c, int32_t layer, int64_t *n_pages_compressed,
                                       void *stream);

/*
 * The same conversion in two steps, so that the factorization can run on a second stream while the caller's main
 * stream goes on with other work (the next layer's projections, appends and attention during a chunked prefill).
 * Not in the paper, which compresses synchronously; the result is the one pkv_compress_eligible_pages() would
 * give for the same pages.
 *
 * pkv_compress_begin(): picks the pages of `layer` (0 <= layer < n_layers) that are eligible now, in ascending
 * (sequence, page) order, allocates their factor slots, and enqueues the factorization on `side_stream`, ordered
 * behind everything enqueued on `main_stream` so far (the appends that wrote the pages).  Nothing else changes:
 * until the commit the pages stay dense pages for every other call - attention keeps reading their rows, appends
 * and compressions of other layers proceed - and their dense slots stay allocated.
 *   n_pages_begun [host, may be NULL] pages picked.  PKV_ERR_POOL_EXHAUSTED: the factor pool ran out; the pages
 *   picked so far are begun and must still be committed.
 * pkv_compress_commit(): for `layer` (-1 = every layer with a begun compression, ascending) makes `main_stream`
 * wait for that factorization, then does what pkv_compress_eligible_pages() does per page, in the same order:
 * the page becomes a factor page, its dense slot is released (so slot reuse stays deterministic: it depends on
 * the order of calls, never on timing), the page table is updated on `main_stream`.  A layer without a begun
 * compression is skipped.   n_pages_compressed [host, may be NULL].
 * Between the two calls, for the layer concerned: pkv_compress_begin and pkv_compress_eligible_pages (also with
 * layer = -1) return PKV_ERR_UNSUPPORTED, and so does pkv_free_seq for a sequence that has pages in flight.
 * Neither call can be captured into a CUDA graph.  pkv_destroy_cache waits for factorizations still running.
 */
pkv_status pkv_compress_begin(pkv_cache *c, int32_t layer, void *main_stream, void *side_stream,
                              int64_t *n_pages_begun);
pkv_status pkv_compress_commit(pkv_cache *c, int32_t layer, void *main_stream, int64_t *n_pages_compressed);

/*
 * Section 3.3 "Attention over Mixed KV Pages", Eq. 4 and Eq. 5: one query per
 * sequence and query head attends over all tokens of that sequence in `layer`.
 *   seq_ids [host] n_seqs distinct ids, each with at least one token in `layer`
 *   q       [device] bf16 [n_seqs, H_q, d]
 *   out     [device] bf16 [n_seqs, H_q, d]
 *   out_f32 [device, may be NULL] the same result before rounding, fp32
 * Scores use softmax_scale; accumulation is fp32.  The result does not depend
 * on physical slot placement and is bit-identical from run to run.
 *
 * CUDA graphs: the call may be recorded into a graph (any decode_overlap), provided this layer's plan for
 * this batch is current, i.e. the same call has been made once outside the capture since the last change of the
 * batch's page tables (otherwise PKV_ERR_UNSUPPORTED: the plan cannot be uploaded from inside a capture).  A
 * replay reads token counts, page tables and the plan from device memory when it runs: appends that stay inside a
 * sequence's current page need nothing; after an append that opens a page, a compression or a free, one such call
 * outside a capture brings the plan up to date and existing graphs for the same batch are valid again.
 * pkv_append_kv and pkv_compress_eligible_pages update host-side state and cannot be captured (PKV_ERR_UNSUPPORTED
 * while the stream is capturing).  With decode_overlap = 2 a recorded launch keeps its scratch set in every replay:
 * launches inside a graph overlap as they do outside, consecutive graph launches are ordered by the stream, and
 * from the first capture on, this cache's launches outside a graph are ordinary (non-overlapping) ones.
 */
pkv_status pkv_decode_attention(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                const void *q, void *out, float *out_f32, void *stream);

/*
 * Mixed attention for the q_len newest positions of each sequence at once (a speculative-decoding step, or a
 * chunk of a prefill after its rows were appended).  The paper's Eq. 4 carries one query; this is the same
 * operation under the causal rule of Eq. 1: query j (0 <= j < q_len) of a sequence with T tokens in `layer`
 * belongs to position T - q_len + j and attends over tokens 0 .. T - q_len + j, itself included, factor pages
 * through their factors and dense pages through their rows exactly as in pkv_decode_attention(); partial states
 * merge by Eq. 5.  q_len = 1 is pkv_decode_attention().
 *   q, out  [device] bf16 [n_seqs, q_len, H_q, d];  out_f32 [device, may be NULL] fp32, same shape
 * Requirements (else PKV_ERR_INVALID_ARG, nothing launched): 1 <= q_len <= T for every listed sequence; no listed
 * sequence has a factor page that reaches past token T - q_len (so every query sees every factor page whole:
 * holds whenever q_len <= recent_tokens and compression ran no later than the append of these positions, and it is
 * checked per call); n_seqs * b <= max_seqs with b = ceil(q_len / max(1, 8 / (H_q / H_kv))) blocks of query tokens
 * per sequence, b rounded up to a multiple of the grid size if it exceeds it (split-K partial states and tickets
 * are kept per sequence and block).
 * Two kinds of kernel serve this call.  A row-block kernel - CTAs per (sequence, KV head, block of query rows),
 * which read the sequence's pages once for the block, the query rows being the row operand of every product of
 * Eq. 4 - runs when q_len * (H_q / H_kv) >= 64 and the factors are bf16.  It is the tcgen05 kernel (any page
 * size and ranks; 128 rows per CTA, accumulators and row
 * operands in tensor memory, pages brought in by TMA in the layout the tensor cores read); where the blocks alone
 * would not fill the GPU it cuts each block's sequence into up to 32 token ranges, one CTA each, and a second
 * launch merges their softmax states by Eq. 5 in token order.  With decode_variant 3 (or a driver without the
 * tensor-map encoder) it is the mma.sync kernel (64 rows per CTA, never split), and then only if the call makes at least 128 blocks
 * (enough to fill the GPU) or would exceed the limit above, which does not apply to row blocks.  Otherwise
 * the decode kernel runs
 * with its CTAs in groups of b = ceil(q_len / max(1, 8 / (H_q / H_kv))): the CTAs of a group walk the same pages at
 * the same time, one block of 8 / (H_q / H_kv) query tokens each, so HBM delivers a page once and L2 delivers it b
 * times (q_len = 2 at H_q / H_kv = 8 costs 1.3 single-query launches, q_len = 2 at H_q / H_kv = 4 costs one).
 * All of them give the same result up to fp32 summation order.
 * Needs decode_variant 0, 2 or 3 (PKV_ERR_UNSUPPORTED with 1).  CUDA-graph and overlap semantics as for
 * pkv_decode_attention(); a layer keeps one plan, that of its most recent (batch, q_len), so calls that
 * alternate between shapes on one layer rebuild it each time (host work and a small upload; not capturable).
 */
pkv_status pkv_decode_attention_multi(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                      int32_t q_len, const void *q, void *out, float *out_f32, void *stream);

/*
 * One sequence spread over several caches (sequence sharding: each cache, e.g. one per GPU, holds a contiguous
 * range of the sequence's tokens with its own pages and factors).  Eq. 5 merges per-page softmax states; the same
 * rule merges per-cache states, so each cache returns its state instead of a normalised output and one more
 * application of Eq. 5 gives the attention over all tokens.  The paper runs on one GPU; this is the exchange step
 * its page-wise formulation allows.
 *
 * pkv_decode_attention_partial(): as pkv_decode_attention(), but writes
 *   state [device] fp32 [n_seqs, H_q, d + 2]: per query head o (d values, not divided by l), then m, then l, where
 *   with s_t = (q . k_t) * softmax_scale * log2(e) over this cache's tokens: m = max_t s_t, l = sum_t 2^(s_t - m),
 *   o = sum_t 2^(s_t - m) v_t  (factor pages contribute through their factors as in Eq. 4).
 * pkv_merge_attention_states(): Eq. 5 over n_shards such arrays stored back to back,
 *   states [device] fp32 [n_shards, n_rows, d + 2] (n_rows = n_seqs * H_q; e.g. the result of an all-gather),
 *   out [device, may be NULL] bf16 [n_rows, d];  out_f32 [device, may be NULL] fp32 [n_rows, d]; not both NULL.
 * Shards are summed in index order, so every holder of the same gathered array computes the same bits.  Needs no
 * cache handle; returns PKV_ERR_INVALID_ARG for NULL / misaligned pointers (states and out 8 bytes, out_f32 16),
 * PKV_ERR_CUDA if the launch fails.
 */
pkv_status pkv_decode_attention_partial(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                        const void *q, float *state, void *stream);
pkv_status pkv_merge_attention_states(const float *states, int32_t n_shards, int64_t n_rows, void *out,
                                      float *out_f32, void *stream);

/*
 * The same call for callers whose queries and results live in host memory.
 *   q_host, out_host [host] bf16 [n_seqs, H_q, d];  q_stage, out_stage [device]
 *   caller-owned staging buffers of the same size.
 * If both host buffers are pinned and device-mapped (cudaHostAlloc / cudaHostRegister), the kernel
 * reads q_host and writes out_host across the bus directly and the staging buffers are not used;
 * otherwise q_host is copied to q_stage, the kernel runs, and out_stage is copied to out_host, all on
 * `stream`.  Either way out_host is valid once the work enqueued on `stream` has completed.
 */
pkv_status pkv_decode_attention_host(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                     const void *q_host, void *out_host, void *q_stage, void *out_stage,
                                     void *stream);

/*
 * No counterpart in the paper: this entry point exists for deployment reasons only.
 *
 * pkv_decode_attention() keeps its split-K scratch (one partial softmax state per CTA and segment,
 * plus the merge tickets) in the `workspace` buffer that the caller allocated.  Some callers cannot
 * provide such a buffer when they decode: code that runs inside a serving process whose device
 * memory is fully handed out at start-up and where a later cudaMalloc is forbidden (it would stall
 * every stream of the device), plug-ins that are given fixed input/output tensors by a host
 * framework and have no allocator of their own, and hosts that let another component reuse or
 * release the workspace between steps.  This variant computes exactly what pkv_decode_attention()
 * computes, with the same kernels, arguments and results, but keeps that scratch in a fixed array
 * inside the library itself.  It calls no cudaMalloc, cudaFree or other allocating routine; the
 * cache's own workspace buffer is not touched.
 *
 * Limits and rules
 *  - Capacity: 1024 partial states: F + F / 8 + S + 2 <= 1024 with S = n_seqs * n_kv_heads and
 *    F = n_ctas + S (one state per CTA and segment, plus the states of groups of eight CTAs that a
 *    segment spread over many CTAs is summed through).  The default grid (296 CTAs) leaves room for
 *    about 280 (sequence, KV head) pairs.  A larger call is rejected with PKV_ERR_INVALID_ARG and a
 *    message; nothing is launched.
 *  - Cost: the array (about 4.1 MiB) is part of the library image, so every GPU on which the
 *    library is loaded holds it until the process exits, whether or not this function is called.
 *  - The first call on each device looks up the array's device address (the device must be
 *    current).  Make that first call outside any CUDA stream capture.  As with
 *    pkv_decode_attention(), a call whose plan must be rebuilt (new batch, or a page table
 *    changed) returns PKV_ERR_UNSUPPORTED while `stream` is capturing.
 *  - All calls on a device share the one array, which keeps the previous call's contents; the
 *    function clears the part that must start at zero (the tickets) on `stream` before each
 *    launch.  Two calls that may run on the GPU at the same time (different streams without an
 *    ordering between them, or different caches) would overwrite each other's partial states:
 *    the caller must order them.  For the same reason consecutive calls do not overlap on the
 *    GPU even when decode_overlap is set.
 */
pkv_status pkv_decode_attention_static_scratch(pkv_cache *c, int32_t layer, int32_t n_seqs,
                                               const int32_t *seq_ids, const void *q, void *out,
                                               float *out_f32, void *stream);

/* Page table of one (sequence, layer) from the host mirror: kinds[i] in
 * {PKV_KIND_DENSE, PKV_KIND_FACTOR}, slots[i] the physical slot, for i <
 * *n_pages (arrays [host] of capacity max_pages_per_seq; may be NULL). */
pkv_status pkv_get_page_table(const pkv_cache *c, int32_t seq, int32_t layer, int32_t *kinds,
                              int32_t *slots, int32_t *n_pages, int32_t *n_tokens);

/*
 * The split of the most recent pkv_decode_attention() call on `layer` over CTAs
 * (host mirror; for tests and tuning).  Work units are ordered by (position in
 * seq_ids, KV head, unit); a unit is one factor page or one block of 16 or 32
 * rows of a dense page.  CTA j owns the units from cta_starts[3j..3j+2] =
 * (position, KV head, unit) up to the start of CTA j+1; entry n_used_ctas is the
 * end sentinel (n_seqs, 0, 0).  seg_parts[2s], seg_parts[2s+1] = first CTA and
 * number of CTAs that hold a partial softmax state of segment s = position *
 * H_kv + KV head.  Arrays [host]: cta_starts 3*(n_ctas+1) ints, seg_parts
 * 2*n_seqs*H_kv ints; any pointer may be NULL.
 */
pkv_status pkv_get_decode_plan(const pkv_cache *c, int32_t layer, int32_t *n_used_ctas, int32_t *cta_starts,
                               int32_t *n_segs, int32_t *seg_parts);

/*
 * Debugging aid.  When the environment variable PKV_DECODE_TRACE=1 is set at pkv_init_cache() time, every
 * CTA of a decode launch records sixteen 64-bit values in the workspace: [0] globaltimer (ns) at entry,
 * [1] at exit, then SM clock counts: [2] entry, [3] first copy issued, [4] first unit's data arrived,
 * [5] last unit of the CTA consumed, [6] exit, [7] units processed (a count), [8] consumers released (mode 0:
 * the preceding kernel has finished), and for the CTA's last segment [9] flush begun, [10] partial state and
 * ticket done, [11] cross-CTA merge: copies issued, [12] first round landed, [13] result stored ([11]-[13] are 0
 * unless this CTA merged); [14], [15] unused.  This call synchronises `stream` and copies the stamps of the most
 * recent launch to out [host, n_ctas * 16 values].
 */
pkv_status pkv_get_decode_trace(pkv_cache *c, int64_t *out, int32_t n_ctas, void *stream);

/* Counters; synchronises `stream` to read the device status words. */
pkv_status pkv_get_stats(pkv_cache *c, pkv_stats *out, void *stream);

/* Releases every slot of a sequence (layers ascending, pages ascending). */
pkv_status pkv_free_seq(pkv_cache *c, int32_t seq);

/* Frees host metadata only; the caller's device buffers are untouched. */
pkv_status pkv_destroy_cache(pkv_cache *c);

const char *pkv_last_error(const pkv_cache *c);

/*
 * Inspection helpers (asynchronous on `stream`).  They translate the private
 * pool format to plain row-major bf16 in caller-owned [device] buffers:
 *   pkv_read_factors : A_k [P, r_k], B_k [r_k, d], A_v [P, r_v], B_v [r_v, d]
 *   pkv_write_factors: the reverse (overwrites one KV head of a factor slot)
 *   pkv_read_dense   : K [P, d], V [P, d] of one KV head of a dense slot
 */
pkv_status pkv_read_factors(pkv_cache *c, int64_t factor_slot, int32_t kv_head, void *A_k, void *B_k,
                            void *A_v, void *B_v, void *stream);
pkv_status pkv_write_factors(pkv_cache *c, int64_t factor_slot, int32_t kv_head, const void *A_k,
                             const void *B_k, const void *A_v, const void *B_v, void *stream);
pkv_status pkv_read_dense(pkv_cache *c, int64_t dense_slot, int32_t kv_head, void *K, void *V,
                          void *stream);
/*
 * Global SVD form only (global_rank > 0; Section 4.2): the shared basis of one (sequence, layer, KV head) as plain
 * row-major bf16, B_k [global_rank, d] and B_v [global_rank, d] ([device], caller-owned).  In that form
 * pkv_read_factors() returns A_k [P, global_rank] and A_v [P, global_rank] only (its B_k, B_v may be NULL), and a
 * page's K^ is A_k B_k with this B_k.  PKV_ERR_INVALID_ARG if the sequence has no basis yet (nothing compressed).
 */
pkv_status pkv_read_basis(pkv_cache *c, int32_t seq, int32_t layer, int32_t kv_head, void *B_k, void *B_v,
                          void *stream);

/*
 * The order in which the page-SVD kernel (pkv_compress_eligible_pages) rotates index pairs during one Jacobi sweep,
 * for inspection and tests.  Host only: no cache, no GPU work.  (The paper fixes the decomposition, Eq. 2, not how the
 * eigen-solve orders its rotations; this describes this library's kernel.)
 *   page_size 64 or 32: the indices 0..P-1 are rotated in groups of four.  *n_rounds = 21 (13) classes,
 *     *groups_per_round = P/4, *group_size = 4; inside a group the six pairs are rotated in the layers
 *     (0,1)(2,3), (0,2)(1,3), (0,3)(1,2) of the group's member positions.
 *   page_size 16: pairs.  *n_rounds = 15, *groups_per_round = 8, *group_size = 2.
 * members [host, out]: n_rounds * groups_per_round * group_size bytes, round-major; `capacity` = its size in bytes.
 * Returns PKV_ERR_INVALID_ARG for another page size, a NULL pointer or a buffer that is too small (nothing written).
 */
pkv_status pkv_get_rotation_schedule(int32_t page_size, uint8_t *members, int64_t capacity, int32_t *n_rounds,
                                     int32_t *groups_per_round, int32_t *group_size);

/*
 * How many token ranges pkv_decode_attention_multi() cuts each row block's sequence into when its tcgen05 row-block
 * kernel serves a call (see there; Eq. 5 merges the ranges), for inspection and tests.  Host only: no cache, no GPU
 * work.  (The paper fixes the merge rule, not how work is spread over a GPU; this describes this library's launch.)
 *   n_row_blocks    blocks of 128 query rows in the call: n_seqs * H_kv * ceil(q_len * (H_q / H_kv) / 128)
 *   longest_tokens  tokens of the longest listed sequence;  page_size as in the configuration
 *   n_sms           multiprocessors of the GPU (two CTAs of the kernel fit one)
 * *n_ranges = min(32, min(2 n_sms, 512) / n_row_blocks, ceil(longest_tokens / page_size) / 8) (integer divisions) if
 * that is at least 2, else 1: ranges only when the row blocks alone leave half the GPU idle, at least eight pages
 * per range, at most 512 states in the workspace.
 * Returns PKV_ERR_INVALID_ARG for a NULL pointer or an argument below 1 (nothing written).
 */
pkv_status pkv_get_row_block_ranges(int64_t n_row_blocks, int32_t longest_tokens, int32_t page_size, int32_t n_sms,
                                    int32_t *n_ranges);

#ifdef __cplusplus
}
#endif
#endif /* PKV_H */
