// Host side of the library: configuration, page tables, free lists, eligibility,
// decode planning (split of the page list over CTAs) and the C ABI.  All device
// work is delegated to the launchers declared in pkv_internal.h.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "pkv_internal.h"

using namespace pkv;

namespace {

struct FreeList {
    // Slots are handed out in the caller's order; a released slot is reused
    // (last released first) before the order array is consumed further.
    std::vector<int32_t> order, stack;
    size_t next = 0;
    int64_t available() const { return (int64_t)(order.size() - next + stack.size()); }
    int32_t alloc() {
        if (!stack.empty()) { int32_t s = stack.back(); stack.pop_back(); return s; }
        return order[next++];
    }
    void release(int32_t s) { stack.push_back(s); }
    int64_t in_use() const { return (int64_t)next - (int64_t)stack.size(); }
};

struct SeqLayer {
    int32_t n_tokens = 0;
    int32_t f_end = 0;                 // pages [sink_pages, f_end) are factor pages
    uint64_t version = 0;              // bumped whenever the page list changes
    bool has_basis = false;            // Global SVD form: the region's basis has been computed
    std::vector<int32_t> slots;
};

struct PlanCache {
    bool valid = false;
    std::vector<int32_t> seq_ids;
    std::vector<uint64_t> versions;
    int q_len = 1;                     // query tokens per sequence the plan was built for
    int n_segs = 0;
    int max_parts = 0;                 // most CTAs any segment is split over
    int64_t units = 0;
    std::vector<PlanCta> ctas;         // n_used + 1 entries (last = end sentinel)
    std::vector<PlanSeg> segs;
};

// Pages whose factorization was started by pkv_compress_begin() and not yet committed: they are still dense pages
// for every other call (slots, f_end and the device page table are untouched until pkv_compress_commit()).
struct PendingPage { int32_t seq, page, dense_slot, factor_slot; };
struct PendingCompress {
    bool active = false;
    std::vector<PendingPage> pages;    // ascending (seq, page)
    cudaEvent_t done = nullptr;        // recorded behind the layer's compression kernels
};

// Pinned staging ring for host -> device metadata uploads.
struct Stager {
    static constexpr int kChunks = 32;
    static constexpr size_t kChunkBytes = 128 * 1024;
    unsigned char *base = nullptr;
    cudaEvent_t ev[kChunks];
    bool pending[kChunks];
    int cur = 0;
    size_t used = 0;
    bool dirty = false;
};

}  // namespace

struct pkv_cache {
    pkv_config cfg;
    Geometry geo;
    MetaLayout ml;
    WorkspaceLayout wl;
    bool dry = false;
    int n_sms = 148;                   // of the device the cache was created on
    bool trace = false;                // PKV_DECODE_TRACE=1: CTAs write time stamps into the workspace
    unsigned char *dense_pool = nullptr, *factor_pool = nullptr, *meta = nullptr, *workspace = nullptr;
    RowBlockMaps row_maps = {};        // TMA descriptors of the pools (tcgen05 row-block kernel)
    FreeList dense_free, factor_free;
    std::vector<SeqLayer> sl;          // [max_seqs * n_layers]
    std::vector<PlanCache> plans;      // [n_layers]
    std::vector<int32_t> stamp;        // duplicate detection
    int32_t stamp_gen = 0;
    Stager stg;
    std::string err;
    int64_t pages_compressed = 0;
    int64_t last_decode_bytes = 0, last_decode_units = 0;
    uint64_t decode_seq = 0;           // decode launches so far (decode_overlap = 2: picks the scratch buffer)
    bool cache_written = true;         // an append or compression kernel was enqueued since the last decode launch
    bool captured_mode2 = false;       // a decode_overlap = 2 launch has been recorded into a CUDA graph
    std::vector<PendingCompress> pending;   // [n_layers]
    int n_pending = 0;                 // layers with a begun, uncommitted compression
    cudaEvent_t order_ev = nullptr;    // scratch event: orders a side stream behind the caller's main stream
    cudaEvent_t worklist_ev = nullptr; // recorded behind the last kernel that reads the device work list
    bool worklist_busy = false;
    // Test hooks (environment, read once per cache): PKV_TEST_WAIT_CLOCKS shortens the decode kernel's bounded
    // waits, PKV_TEST_DROP_UNIT makes the first decode launch leave one unit unarmed, so that a wait runs out.
    long long wait_clocks = 2000000000LL;
    int drop_unit = -1;
    int64_t timeouts_seen = 0;         // device_timeouts at the last pkv_get_stats()
    bool tickets_dirty = false;        // a launch gave up: merge tickets may be left non-zero

    SeqLayer &at(int seq, int layer) { return sl[(size_t)seq * cfg.n_layers + layer]; }
    const SeqLayer &at(int seq, int layer) const { return sl[(size_t)seq * cfg.n_layers + layer]; }
};

namespace {

pkv_status fail(pkv_cache *c, pkv_status code, const char *fmt, ...) {
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return code;
}

#define PKV_CUDA(c, call)                                                                         \
    do {                                                                                          \
        cudaError_t e_ = (call);                                                                  \
        if (e_ != cudaSuccess)                                                                    \
            return fail((c), PKV_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));        \
    } while (0)

pkv_status validate(const pkv_config *cfg, const char **why) {
    *why = "";
    if (!cfg) { *why = "cfg is NULL"; return PKV_ERR_INVALID_ARG; }
    if (cfg->n_layers <= 0 || cfg->n_kv_heads <= 0 || cfg->n_q_heads <= 0 || cfg->max_seqs <= 0 ||
        cfg->max_pages_per_seq <= 0 || cfg->n_dense_slots <= 0 || cfg->n_factor_slots < 0) {
        *why = "counts must be positive"; return PKV_ERR_INVALID_ARG;
    }
    if (cfg->n_q_heads % cfg->n_kv_heads) { *why = "n_q_heads must be a multiple of n_kv_heads"; return PKV_ERR_INVALID_ARG; }
    if (cfg->global_rank <= 0 &&
        (cfg->page_size <= 0 || cfg->rank_k <= 0 || cfg->rank_v <= 0 || cfg->rank_k > cfg->page_size ||
         cfg->rank_v > cfg->page_size || cfg->page_size > cfg->head_dim)) {
        *why = "need 0 < rank <= page_size <= head_dim"; return PKV_ERR_INVALID_ARG;
    }
    if (cfg->sink_tokens < 0 || cfg->recent_tokens < 0 || cfg->sink_tokens % cfg->page_size ||
        cfg->recent_tokens % cfg->page_size) {
        *why = "sink_tokens and recent_tokens must be non-negative multiples of page_size"; return PKV_ERR_INVALID_ARG;
    }
    if (cfg->softmax_scale < 0.f || cfg->jacobi_max_sweeps < 0 || cfg->jacobi_tol < 0.f || cfg->n_ctas < 0 ||
        cfg->decode_variant < 0 || cfg->decode_variant > 3 ||
        cfg->decode_overlap < 0 || cfg->decode_overlap > 2 ||
        (cfg->factor_bits != 0 && cfg->factor_bits != 4 && cfg->factor_bits != 16)) {
        *why = "negative scale / sweep cap / tolerance / n_ctas, or unknown decode_variant / decode_overlap / factor_bits"; return PKV_ERR_INVALID_ARG;
    }
    if (cfg->n_dense_slots > INT32_MAX || cfg->n_factor_slots > INT32_MAX) {
        *why = "slot counts must fit in int32"; return PKV_ERR_INVALID_ARG;
    }
    if (cfg->global_rank < 0) { *why = "global_rank is negative"; return PKV_ERR_INVALID_ARG; }
    if (cfg->global_rank > 0) {
        if (cfg->head_dim != kHeadDim) { *why = "only head_dim = 128 is supported"; return PKV_ERR_UNSUPPORTED; }
        if ((cfg->global_rank != 64 && cfg->global_rank != 80 && cfg->global_rank != 96) ||
            (cfg->page_size != 32 && cfg->page_size != 64) || cfg->factor_bits == 4 || cfg->decode_variant == 1) {
            *why = "the Global SVD form needs global_rank 64, 80 or 96, page_size 32 or 64, bf16 factors, decode_variant 0 or 2";
            return PKV_ERR_UNSUPPORTED;
        }
        if (cfg->n_q_heads / cfg->n_kv_heads > kMaxGroup) { *why = "only n_q_heads/n_kv_heads <= 8 is supported"; return PKV_ERR_UNSUPPORTED; }
        return PKV_OK;
    }
    if (cfg->head_dim != kHeadDim) { *why = "only head_dim = 128 is supported"; return PKV_ERR_UNSUPPORTED; }
    if (cfg->page_size != 16 && cfg->page_size != 32 && cfg->page_size != 64) {
        *why = "only page_size 16, 32 or 64 is supported"; return PKV_ERR_UNSUPPORTED;
    }
    if ((cfg->rank_k + 7) / 8 != (cfg->rank_v + 7) / 8 || cfg->rank_k > 32 || cfg->rank_v > 32) {
        *why = "ranks must be <= 32 and round up to the same multiple of 8 for K and V"; return PKV_ERR_UNSUPPORTED;
    }
    if (cfg->n_q_heads / cfg->n_kv_heads > kMaxGroup) { *why = "only n_q_heads/n_kv_heads <= 8 is supported"; return PKV_ERR_UNSUPPORTED; }
    return PKV_OK;
}

long long align_up(long long x, long long a) { return (x + a - 1) / a * a; }

void derive(const pkv_config &cfg, int n_ctas, Geometry &g, MetaLayout &ml, WorkspaceLayout &wl) {
    const int P = cfg.page_size, d = cfg.head_dim;
    g.n_layers = cfg.n_layers; g.n_kv_heads = cfg.n_kv_heads; g.n_q_heads = cfg.n_q_heads;
    g.group = cfg.n_q_heads / cfg.n_kv_heads;
    g.page = P;
    g.global_rank = cfg.global_rank;
    g.rank_k = cfg.global_rank > 0 ? cfg.global_rank : cfg.rank_k;
    g.rank_v = cfg.global_rank > 0 ? cfg.global_rank : cfg.rank_v;
    g.rank_tiles = (g.rank_k + 7) / 8;
    g.basis_head_bytes = 2 * cfg.global_rank * kRowBytes;
    g.max_seqs = cfg.max_seqs; g.max_pages = cfg.max_pages_per_seq;
    g.n_dense_slots = (int)cfg.n_dense_slots; g.n_factor_slots = (int)cfg.n_factor_slots;
    g.sink_pages = cfg.sink_tokens / P; g.recent_pages = cfg.recent_tokens / P;
    g.ak_off = 0;
    g.bk_off = g.ak_off + P * g.rank_k * 2;
    g.av_off = g.bk_off + (cfg.global_rank > 0 ? 0 : g.rank_k * d * 2);
    g.bv_off = g.av_off + P * g.rank_v * 2;
    g.blob16_bytes = g.bv_off + (cfg.global_rank > 0 ? 0 : g.rank_v * d * 2);
    g.factor_bits = cfg.factor_bits == 4 ? 4 : 16;
    g.cak_off = 0;
    g.cbk_off = g.cak_off + 4 * int4_a_words(P, g.rank_tiles);
    g.cav_off = g.cbk_off + 4 * int4_b_words(d, g.rank_tiles);
    g.cbv_off = g.cav_off + 4 * int4_b_words(P, g.rank_tiles);
    g.codes_bytes = g.cbv_off + 4 * int4_a_words(d, g.rank_tiles);
    g.sak_off = 0;
    g.sbk_off = g.sak_off + 2 * (int)align_up(g.rank_k, 8);
    g.sav_off = g.sbk_off + 2 * d;
    g.sbv_off = g.sav_off + 2 * P;
    const int scales_bytes = g.sbv_off + 2 * d;
    g.blob_bytes = g.factor_bits == 4 ? (int)align_up(g.codes_bytes + scales_bytes, 16) : g.blob16_bytes;
    g.dense_head_bytes = 2 * P * d * 2;
    g.dense_slot_bytes = (long long)cfg.n_kv_heads * g.dense_head_bytes;
    g.factor_slot_bytes = (long long)cfg.n_kv_heads * g.blob_bytes;
    // decode work units: a factor page or a block of rows of a dense page.  A stage must hold either, plus
    // the rows that 8-row tile loads read past the last matrix when rank_v is not a multiple of 8.
    g.block_tokens = (g.factor_bits != 4 && P >= 32 && g.rank_tiles >= 3) ? 32 : 16;
    g.blocks_per_page = P / g.block_tokens;
    const int overread = (8 * g.rank_tiles - g.rank_v) * kRowBytes;
    int factor_stage = g.factor_bits == 4 ? g.blob_bytes : (int)align_up(g.blob16_bytes + overread, 16);
    if (cfg.global_rank > 0) factor_stage = std::max(g.blob16_bytes, cfg.global_rank * kRowBytes);   // a page's rows, or one basis matrix
    g.stage_bytes = (int)align_up(std::max(factor_stage, g.block_tokens * 2 * kRowBytes), 128);
    // two CTAs are resident per SM (consecutive launches overlap, or the grid holds two CTAs per SM),
    // so that one streams while the other is in its prologue or merging
    const int fixed = kConsumerWarps * kPartialFloats * 4 + 1024 + 1024;
    g.n_stages = std::min(16, (kSmemBudget / 2 - fixed) / g.stage_bytes);
    g.n_ctas = n_ctas;
    const float scale = cfg.softmax_scale > 0.f ? cfg.softmax_scale : 1.0f / std::sqrt((float)d);
    g.scale_log2e = scale * 1.4426950408889634f;
    g.jacobi_max_sweeps = cfg.jacobi_max_sweeps > 0 ? cfg.jacobi_max_sweeps : 16;
    g.jacobi_tol = cfg.jacobi_tol > 0.f ? cfg.jacobi_tol : 1e-5f;
    g.jacobi_energy_tol = cfg.jacobi_energy_tol == 0.f ? 1e-4f : cfg.jacobi_energy_tol;

    long long off = 0;
    ml.page_table = off; off = align_up(off + 4LL * cfg.max_seqs * cfg.n_layers * cfg.max_pages_per_seq, 256);
    ml.n_tokens = off;   off = align_up(off + 4LL * cfg.max_seqs * cfg.n_layers, 256);
    long long p = sizeof(PlanHeader);
    ml.plan_cta = p;   p = align_up(p + (long long)sizeof(PlanCta) * (n_ctas + 1), 16);
    ml.plan_entry = p; p = align_up(p + (long long)sizeof(PlanEntry) * cfg.max_seqs, 16);
    ml.plan_cta_entry = p; p = align_up(p + (long long)sizeof(PlanEntry) * (n_ctas + 1), 16);
    ml.plan_seg = p;   p = align_up(p + (long long)sizeof(PlanSeg) * cfg.max_seqs * cfg.n_kv_heads, 256);
    ml.plan_stride = p;
    ml.plans = off;      off = align_up(off + p * cfg.n_layers, 256);
    ml.append_desc = off; off = align_up(off + (long long)sizeof(AppendDesc) * cfg.max_seqs, 256);
    ml.status = off;     off = align_up(off + 4LL * kStatusWords, 256);
    ml.basis = off;      off = align_up(off + (long long)cfg.max_seqs * cfg.n_layers * cfg.n_kv_heads * g.basis_head_bytes, 256);
    ml.total = off;

    wl.n_seg_tickets = (long long)cfg.max_seqs * cfg.n_kv_heads;
    wl.n_flat = (long long)n_ctas + wl.n_seg_tickets;
    wl.n_group = merge_group_slots(wl.n_flat, wl.n_seg_tickets);
    wl.n_partials = wl.n_flat + wl.n_group;
    long long w = 0;
    wl.partials_stride = align_up(wl.n_partials * kPartialFloats * 4, 256);
    wl.tickets_stride = align_up(4LL * (wl.n_seg_tickets + wl.n_group), 256);
    // decode_overlap = 2 rotates over several sets of split-K scratch; the more sets, the rarer the draining launch
    wl.n_sets = 1;
    if (cfg.decode_overlap == 2) {
        // sized for the largest grid pkv_query_sizes() may have assumed (512 CTAs), so that the count does not
        // depend on the grid actually used and the workspace the caller allocated is always large enough
        const long long widest_flat = (long long)std::max(512, n_ctas) + wl.n_seg_tickets;
        const long long widest = align_up((widest_flat + merge_group_slots(widest_flat, wl.n_seg_tickets)) * kPartialFloats * 4, 256);
        const long long fit = kDecodeBufferBudget / (widest + wl.tickets_stride);
        wl.n_sets = (int)std::min<long long>(kMaxDecodeBuffers, std::max<long long>(4, fit));
    }
    wl.partials = w; w += wl.partials_stride * wl.n_sets;
    wl.worklist = w; w = align_up(w + (long long)sizeof(int2) * kCompressChunk, 256);
    wl.tickets = w;  w += wl.tickets_stride * wl.n_sets;
    wl.gram = w;     w = align_up(w + (cfg.global_rank > 0 ? 4LL * cfg.n_kv_heads * 2 * d * d : 0), 256);
    wl.trace = w;    w = align_up(w + 8LL * kTraceSlots * n_ctas, 256);
    wl.rb_partials = w;
    w = align_up(w + (row_block_umma_supported(g) ? 4LL * kRbSplitItems * 128 * kRbStateFloats : 0), 256);
    wl.total = w;
}

int default_ctas(bool dry) {
    if (dry) return 148;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
    return sms;
}

// ---- staging ring -----------------------------------------------------------
pkv_status stager_init(pkv_cache *c) {
    Stager &s = c->stg;
    PKV_CUDA(c, cudaHostAlloc((void **)&s.base, Stager::kChunks * Stager::kChunkBytes, cudaHostAllocDefault));
    for (int i = 0; i < Stager::kChunks; ++i) {
        PKV_CUDA(c, cudaEventCreateWithFlags(&s.ev[i], cudaEventDisableTiming));
        s.pending[i] = false;
    }
    return PKV_OK;
}

// Moves to the next chunk, recording an event for the one just used.
pkv_status stager_flush(pkv_cache *c, cudaStream_t st) {
    Stager &s = c->stg;
    if (!s.dirty) return PKV_OK;
    PKV_CUDA(c, cudaEventRecord(s.ev[s.cur], st));
    s.pending[s.cur] = true;
    s.cur = (s.cur + 1) % Stager::kChunks;
    s.used = 0;
    s.dirty = false;
    if (s.pending[s.cur]) {
        PKV_CUDA(c, cudaEventSynchronize(s.ev[s.cur]));
        s.pending[s.cur] = false;
    }
    return PKV_OK;
}

// Copies `bytes` of host data to device address `dst` through the ring.
pkv_status upload(pkv_cache *c, void *dst, const void *src, size_t bytes, cudaStream_t st) {
    Stager &s = c->stg;
    const unsigned char *p = (const unsigned char *)src;
    unsigned char *d = (unsigned char *)dst;
    while (bytes > 0) {
        if (s.used == Stager::kChunkBytes) {
            pkv_status r = stager_flush(c, st);
            if (r != PKV_OK) return r;
        }
        size_t n = std::min(bytes, Stager::kChunkBytes - s.used);
        unsigned char *h = s.base + (size_t)s.cur * Stager::kChunkBytes + s.used;
        memcpy(h, p, n);
        PKV_CUDA(c, cudaMemcpyAsync(d, h, n, cudaMemcpyHostToDevice, st));
        s.used += align_up((long long)n, 16);
        if (s.used > Stager::kChunkBytes) s.used = Stager::kChunkBytes;
        s.dirty = true;
        p += n; d += n; bytes -= n;
    }
    return PKV_OK;
}

int *dev_page_table_row(pkv_cache *c, int seq, int layer) {
    return (int *)(c->meta + c->ml.page_table) +
           ((size_t)seq * c->cfg.n_layers + layer) * (size_t)c->cfg.max_pages_per_seq;
}

pkv_status check_seq_list(pkv_cache *c, int32_t n_seqs, const int32_t *seq_ids) {
    if (n_seqs <= 0 || n_seqs > c->cfg.max_seqs || !seq_ids)
        return fail(c, PKV_ERR_INVALID_ARG, "n_seqs must be in [1, max_seqs] and seq_ids non-NULL");
    if (++c->stamp_gen == INT32_MAX) { std::fill(c->stamp.begin(), c->stamp.end(), 0); c->stamp_gen = 1; }
    for (int i = 0; i < n_seqs; ++i) {
        int s = seq_ids[i];
        if (s < 0 || s >= c->cfg.max_seqs) return fail(c, PKV_ERR_BAD_SEQ, "sequence id %d out of range", s);
        if (c->stamp[s] == c->stamp_gen) return fail(c, PKV_ERR_BAD_SEQ, "sequence id %d repeated", s);
        c->stamp[s] = c->stamp_gen;
    }
    return PKV_OK;
}

// ---- decode planning ----------------------------------------------------------
struct HeadShape { int d0_units, nf, d1_units, units; long long cost; };

HeadShape head_shape(const Geometry &g, int n_pages, int f_begin, int f_end, long long cf, long long cd) {
    HeadShape h;
    int fb = std::min(f_begin, n_pages), fe = std::min(std::max(f_end, fb), n_pages);
    h.d0_units = fb * g.blocks_per_page;
    h.nf = fe - fb;
    h.d1_units = (n_pages - fe) * g.blocks_per_page;
    h.units = h.d0_units + h.nf + h.d1_units;
    h.cost = (long long)(h.d0_units + h.d1_units) * cd + (long long)h.nf * cf;
    return h;
}

// Smallest unit index u whose start cost (cost of units [0,u)) is >= rem.
int first_unit_at_or_after(const HeadShape &h, long long rem, long long cf, long long cd) {
    if (rem <= 0) return 0;
    long long c0 = (long long)h.d0_units * cd;
    if (rem <= c0) return (int)((rem + cd - 1) / cd);
    rem -= c0;
    long long c1 = (long long)h.nf * cf;
    if (rem <= c1) return h.d0_units + (int)((rem + cf - 1) / cf);
    rem -= c1;
    return h.d0_units + h.nf + (int)std::min<long long>((rem + cd - 1) / cd, h.d1_units);
}

// Query tokens that share one score tile (eight query columns), and plan entries per sequence.
int queries_per_tile(const Geometry &g, int q_len) { return std::max(1, std::min(q_len, kMaxGroup / g.group)); }
int entries_per_seq(const Geometry &g, int q_len) { const int t = queries_per_tile(g, q_len); return (q_len + t - 1) / t; }
// Sibling CTAs per plan range (at most the grid), and plan entries ("passes") per sequence that this leaves.
int sibling_group(const Geometry &g, int q_len) { return std::max(1, std::min(entries_per_seq(g, q_len), g.n_ctas)); }
int passes_per_seq(const Geometry &g, int q_len) { const int s = sibling_group(g, q_len); return (entries_per_seq(g, q_len) + s - 1) / s; }
// Block numbers per sequence, including the empty ones of the last pass: what partial states and tickets are sized by.
int block_slots_per_seq(const Geometry &g, int q_len) { return passes_per_seq(g, q_len) * sibling_group(g, q_len); }

// `n_listed` sequences with q_len queries each.  With entries_per_seq() = b > 1 query blocks per sequence, the
// (sequence, KV head, unit) order is cut into at most n_ctas / s ranges, s = sibling_group(), and the launch's
// CTAs work in groups of s on one range each, one query block per CTA; a sequence appears once in the plan unless
// b exceeds the grid, in which case it appears passes_per_seq() times, each pass for the next s blocks.  The
// partial states and tickets are counted per (sequence, block number, KV head), which is why
// n_listed * block_slots_per_seq() <= max_seqs is required.
// Whether a call with q_len queries for each of n_seqs sequences goes to the row-block kernel (one CTA per 64 query
// rows of a KV head, which walks the whole sequence alone) instead of the pipeline kernel (eight query columns per
// pass over the pages, split over all CTAs).  The row-block kernel needs enough CTAs to fill the GPU; below that the
// pipeline kernel is used if its plan entries fit.
// Token ranges per row block of a tcgen05 row-block launch (documented with pkv_get_row_block_ranges()).
int row_block_ranges(long long n_blocks, int longest_tokens, int page_size, int n_sms) {
    const long long by_fill = std::min<long long>(2LL * n_sms, kRbSplitItems) / n_blocks;
    const long long by_length = (longest_tokens + page_size - 1) / page_size / kRbMinPages;
    const long long ns = std::min<long long>(kRbMaxSplits, std::min(by_fill, by_length));
    return ns >= 2 ? (int)ns : 1;
}

bool uses_row_blocks(const pkv_cache *c, int q_len, int n_seqs) {
    const long long rows = (long long)q_len * c->geo.group;
    if (q_len <= 1 || (c->cfg.decode_variant != 0 && c->cfg.decode_variant != 3) || c->geo.factor_bits == 4 || rows < kRowBlock) return false;
    // (the tcgen05 kernel splits long sequences over several CTAs when the row blocks alone would not fill the GPU)
    if (c->row_maps.valid && c->cfg.decode_variant == 0) return true;
    const long long n_ctas = (long long)n_seqs * c->geo.n_kv_heads * ((rows + kRowBlock - 1) / kRowBlock);
    return n_ctas >= 128 || (long long)n_seqs * block_slots_per_seq(c->geo, q_len) > c->cfg.max_seqs;
}

pkv_status build_plan(pkv_cache *c, int layer, int n_listed, const int32_t *seq_ids, int q_len, cudaStream_t st) {
    const Geometry &g = c->geo;
    PlanCache &pc = c->plans[layer];
    const int H = g.n_kv_heads;
    const long long cf = g.blob_bytes + 2048, cd = (long long)g.block_tokens * 2 * kRowBytes + 2048;
    // (the row-block kernel only reads the entries; the split over CTAs is not used by it)
    const bool blocks = uses_row_blocks(c, q_len, n_listed);
    const int groups = blocks ? 1 : sibling_group(g, q_len), per_seq = blocks ? 1 : passes_per_seq(g, q_len);
    const int N = std::max(1, g.n_ctas / groups), n_seqs = n_listed * per_seq;

    std::vector<PlanEntry> entries(n_seqs);
    std::vector<HeadShape> shapes(n_seqs);
    long long total_cost = 0, total_units = 0;
    for (int i = 0; i < n_seqs; ++i) {
        const int32_t seq = seq_ids[i / per_seq];
        const SeqLayer &s = c->at(seq, layer);
        int n_pages = (s.n_tokens + c->cfg.page_size - 1) / c->cfg.page_size;
        entries[i] = PlanEntry{seq, n_pages, g.sink_pages, s.f_end};
        shapes[i] = head_shape(g, n_pages, g.sink_pages, s.f_end, cf, cd);
        total_cost += shapes[i].cost * H;
        total_units += (long long)shapes[i].units * H;
    }
    // Cut the (entry, head, unit) sequence where the running cost crosses j * total / n_cut.  A CTA's consumer
    // warps take units in turn, so ranges shorter than one unit per warp would not finish sooner and only add
    // partial states to merge: small batches use fewer CTAs.
    const int n_cut = (int)std::max<long long>(1, std::min<long long>(N, total_units / kConsumerWarps));
    std::vector<PlanCta> ctas;
    ctas.reserve(n_cut + 1);
    {
        int i = 0, h = 0;
        long long base = 0;          // cost before (i, h)
        for (int j = 0; j < n_cut; ++j) {
            long long b = (total_cost * j) / n_cut;
            while (i < n_seqs && base + shapes[i].cost <= b) {
                base += shapes[i].cost;
                if (++h == H) { h = 0; ++i; }
            }
            if (i >= n_seqs) break;
            int u = first_unit_at_or_after(shapes[i], b - base, cf, cd);
            PlanCta pos{i, h, u, 0};
            if (u >= shapes[i].units) {          // start of the next (entry, head)
                pos.unit = 0;
                pos.head = h + 1;
                if (pos.head == H) { pos.head = 0; pos.entry = i + 1; }
                if (pos.entry >= n_seqs) break;
            }
            if (!ctas.empty() && ctas.back().entry == pos.entry && ctas.back().head == pos.head &&
                ctas.back().unit == pos.unit)
                continue;                         // empty range: drop it
            ctas.push_back(pos);
        }
    }
    const int n_used = (int)ctas.size();
    ctas.push_back(PlanCta{n_seqs, 0, 0, 0});    // end sentinel
    // Which CTAs hold a partial state of each (entry, head) segment.
    const int n_segs = n_seqs * H;
    std::vector<PlanSeg> segs(n_segs, PlanSeg{0, 0});
    for (int j = 0; j < n_used; ++j) {
        int g0 = ctas[j].entry * H + ctas[j].head;
        int g1 = ctas[j + 1].entry * H + ctas[j + 1].head;     // segment of the first unit NOT in the range
        if (ctas[j + 1].unit == 0) g1 -= 1;                    // range ends exactly at a segment boundary
        for (int s = g0; s <= g1 && s < n_segs; ++s) {
            if (segs[s].n_parts == 0) segs[s].cta_first = j;
            segs[s].n_parts += 1;
        }
    }
    PlanHeader hdr{n_seqs, n_used, n_segs, (int)std::min<long long>(total_units, INT32_MAX)};

    pc.valid = true;
    pc.q_len = q_len;
    pc.seq_ids.assign(seq_ids, seq_ids + n_listed);
    pc.versions.resize(n_listed);
    for (int i = 0; i < n_listed; ++i) pc.versions[i] = c->at(seq_ids[i], layer).version;
    pc.n_segs = n_segs;
    pc.max_parts = 0;
    for (const PlanSeg &sg : segs) pc.max_parts = std::max(pc.max_parts, sg.n_parts);
    pc.units = total_units;
    pc.ctas = ctas;
    pc.segs = segs;

    if (c->dry) return PKV_OK;
    unsigned char *plan = c->meta + c->ml.plans + c->ml.plan_stride * layer;
    pkv_status r;
    if ((r = upload(c, plan, &hdr, sizeof hdr, st)) != PKV_OK) return r;
    if ((r = upload(c, plan + c->ml.plan_cta, ctas.data(), sizeof(PlanCta) * ctas.size(), st)) != PKV_OK) return r;
    {
        std::vector<PlanEntry> first(n_used);
        for (int j = 0; j < n_used; ++j) first[j] = entries[ctas[j].entry];
        if (n_used > 0 && (r = upload(c, plan + c->ml.plan_cta_entry, first.data(), sizeof(PlanEntry) * n_used, st)) != PKV_OK) return r;
    }
    if ((r = upload(c, plan + c->ml.plan_entry, entries.data(), sizeof(PlanEntry) * n_seqs, st)) != PKV_OK) return r;
    if ((r = upload(c, plan + c->ml.plan_seg, segs.data(), sizeof(PlanSeg) * n_segs, st)) != PKV_OK) return r;
    return stager_flush(c, st);
}

bool plan_is_current(pkv_cache *c, int layer, int n_seqs, const int32_t *seq_ids, int q_len) {
    const PlanCache &pc = c->plans[layer];
    if (!pc.valid || (int)pc.seq_ids.size() != n_seqs || pc.q_len != q_len) return false;
    for (int i = 0; i < n_seqs; ++i) {
        if (pc.seq_ids[i] != seq_ids[i]) return false;
        if (pc.versions[i] != c->at(seq_ids[i], layer).version) return false;
    }
    return true;
}

}  // namespace

// =============================================================================
extern "C" {

pkv_status pkv_query_sizes(const pkv_config *cfg, pkv_sizes *out) {
    const char *why;
    pkv_status r = validate(cfg, &why);
    if (r != PKV_OK) return r;
    if (!out) return PKV_ERR_INVALID_ARG;
    Geometry g; MetaLayout ml; WorkspaceLayout wl;
    // meta / workspace sizes depend on the grid size; the default grid never exceeds 512 CTAs
    int n_ctas = cfg->n_ctas > 0 ? cfg->n_ctas : 512;
    derive(*cfg, n_ctas, g, ml, wl);
    out->dense_slot_bytes = g.dense_slot_bytes;
    out->factor_slot_bytes = g.factor_slot_bytes;
    out->dense_pool_bytes = g.dense_slot_bytes * cfg->n_dense_slots;
    out->factor_pool_bytes = g.factor_slot_bytes * cfg->n_factor_slots;
    out->meta_bytes = ml.total;
    out->workspace_bytes = wl.total;
    return PKV_OK;
}

pkv_status pkv_init_cache(const pkv_config *cfg, void *dense_pool, void *factor_pool, void *meta,
                          void *workspace, const int32_t *dense_slot_order,
                          const int32_t *factor_slot_order, pkv_cache **out) {
    const char *why;
    pkv_status r = validate(cfg, &why);
    if (r != PKV_OK) return r;
    if (!out) return PKV_ERR_INVALID_ARG;
    const bool dry = !dense_pool && !factor_pool && !meta && !workspace;
    if (!dry && (!dense_pool || !meta || !workspace || (!factor_pool && cfg->n_factor_slots > 0)))
        return PKV_ERR_INVALID_ARG;
    if (!dry && (((uintptr_t)dense_pool | (uintptr_t)factor_pool | (uintptr_t)meta | (uintptr_t)workspace) & 255))
        return PKV_ERR_INVALID_ARG;
    pkv_cache *c = new (std::nothrow) pkv_cache();
    if (!c) return PKV_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->dry = dry;
    { const char *t = getenv("PKV_DECODE_TRACE"); c->trace = t && t[0] == '1'; }
    { const char *t = getenv("PKV_TEST_WAIT_CLOCKS"); if (t && atoll(t) > 0) c->wait_clocks = atoll(t); }
    { const char *t = getenv("PKV_TEST_DROP_UNIT"); if (t && t[0]) c->drop_unit = atoi(t); }
    // default grid: one CTA per SM when consecutive launches overlap (two launches share each SM),
    // otherwise two CTAs per SM
    c->n_sms = default_ctas(dry);
    int n_ctas = cfg->n_ctas > 0 ? cfg->n_ctas : c->n_sms * (cfg->decode_overlap ? 1 : 2);
    if (cfg->n_ctas == 0 && n_ctas > 512) n_ctas = 512;      // pkv_query_sizes() sized the buffers for <= 512
    derive(*cfg, n_ctas, c->geo, c->ml, c->wl);
    {
        // the caller sized meta and workspace with pkv_query_sizes(): never use more than that
        pkv_sizes promised;
        if (pkv_query_sizes(cfg, &promised) != PKV_OK || c->ml.total > promised.meta_bytes ||
            c->wl.total > promised.workspace_bytes) {
            delete c;
            return PKV_ERR_INVALID_ARG;
        }
    }
    c->dense_pool = (unsigned char *)dense_pool; c->factor_pool = (unsigned char *)factor_pool;
    c->meta = (unsigned char *)meta; c->workspace = (unsigned char *)workspace;
    auto fill = [](FreeList &f, const int32_t *order, int64_t n) -> bool {
        f.order.resize((size_t)n);
        std::vector<char> seen((size_t)n, 0);
        for (int64_t i = 0; i < n; ++i) {
            int32_t s = order ? order[i] : (int32_t)i;
            if (s < 0 || s >= n || seen[s]) return false;
            seen[s] = 1;
            f.order[(size_t)i] = s;
        }
        return true;
    };
    if (!fill(c->dense_free, dense_slot_order, cfg->n_dense_slots) ||
        !fill(c->factor_free, factor_slot_order, cfg->n_factor_slots)) {
        delete c;
        return PKV_ERR_INVALID_ARG;               // slot order is not a permutation
    }
    c->sl.resize((size_t)cfg->max_seqs * cfg->n_layers);
    for (auto &s : c->sl) s.f_end = c->geo.sink_pages;
    c->plans.resize(cfg->n_layers);
    c->pending.resize(cfg->n_layers);
    c->stamp.assign(cfg->max_seqs, 0);
    if (!dry) {
        cudaError_t e = cudaMemset(c->meta, 0, (size_t)c->ml.total);
        if (e == cudaSuccess) e = cudaMemset(c->workspace, 0, (size_t)c->wl.total);
        if (e == cudaSuccess) e = decode_kernel_setup();
        if (e == cudaSuccess) row_block_make_maps(c->geo, c->factor_pool, c->dense_pool, &c->row_maps);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
        if (e != cudaSuccess || stager_init(c) != PKV_OK) { delete c; return PKV_ERR_CUDA; }
    }
    *out = c;
    return PKV_OK;
}

pkv_status pkv_destroy_cache(pkv_cache *c) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (!c->dry && c->stg.base) {
        for (int i = 0; i < Stager::kChunks; ++i) {
            if (c->stg.pending[i]) cudaEventSynchronize(c->stg.ev[i]);
            cudaEventDestroy(c->stg.ev[i]);
        }
        cudaFreeHost(c->stg.base);
    }
    for (PendingCompress &pc : c->pending)
        if (pc.done) { cudaEventSynchronize(pc.done); cudaEventDestroy(pc.done); }
    if (c->order_ev) cudaEventDestroy(c->order_ev);
    if (c->worklist_ev) { cudaEventSynchronize(c->worklist_ev); cudaEventDestroy(c->worklist_ev); }
    delete c;
    return PKV_OK;
}

const char *pkv_last_error(const pkv_cache *c) { return c ? c->err.c_str() : "cache is NULL"; }

// Calls that change host-side state or copy from the staging ring cannot be recorded into a CUDA graph.
static bool is_capturing(cudaStream_t st) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    return cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone;
}

pkv_status pkv_append_kv(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                         const int32_t *n_new, const void *k, const void *v, void *stream) {
    if (!c) return PKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, PKV_ERR_INVALID_ARG, "layer %d out of range", layer);
    pkv_status r = check_seq_list(c, n_seqs, seq_ids);
    if (r != PKV_OK) return r;
    if (!n_new) return fail(c, PKV_ERR_INVALID_ARG, "n_new is NULL");
    long long n_tok = 0, need = 0;
    for (int i = 0; i < n_seqs; ++i) {
        if (n_new[i] < 0) return fail(c, PKV_ERR_INVALID_ARG, "n_new[%d] is negative", i);
        const SeqLayer &s = c->at(seq_ids[i], layer);
        long long after = ((long long)s.n_tokens + n_new[i] + c->cfg.page_size - 1) / c->cfg.page_size;
        if (after > c->cfg.max_pages_per_seq)
            return fail(c, PKV_ERR_POOL_EXHAUSTED, "sequence %d would exceed max_pages_per_seq", seq_ids[i]);
        need += after - (long long)s.slots.size();
        n_tok += n_new[i];
    }
    if (need > c->dense_free.available())
        return fail(c, PKV_ERR_POOL_EXHAUSTED, "dense pool exhausted: need %lld slots, %lld free", need,
                    (long long)c->dense_free.available());
    if (!c->dry && n_tok > 0 && (!k || !v)) return fail(c, PKV_ERR_INVALID_ARG, "k or v is NULL");
    if (((uintptr_t)k | (uintptr_t)v) & 15) return fail(c, PKV_ERR_INVALID_ARG, "k and v must be 16-byte aligned");
    if (n_tok == 0) return PKV_OK;
    if (!c->dry && is_capturing(st))
        return fail(c, PKV_ERR_UNSUPPORTED, "pkv_append_kv cannot be captured into a CUDA graph");

    std::vector<AppendDesc> desc;
    desc.reserve(n_seqs);
    long long tok = 0;
    for (int i = 0; i < n_seqs; ++i) {
        if (n_new[i] == 0) continue;
        SeqLayer &s = c->at(seq_ids[i], layer);
        desc.push_back(AppendDesc{seq_ids[i], s.n_tokens, (int)tok, n_new[i]});
        int before = (int)s.slots.size();
        int after = (s.n_tokens + n_new[i] + c->cfg.page_size - 1) / c->cfg.page_size;
        for (int p = before; p < after; ++p) s.slots.push_back(c->dense_free.alloc());
        s.n_tokens += n_new[i];
        tok += n_new[i];
        if (after > before) {
            s.version++;
            if (!c->dry) {
                r = upload(c, dev_page_table_row(c, seq_ids[i], layer) + before, s.slots.data() + before,
                           sizeof(int32_t) * (after - before), st);
                if (r != PKV_OK) return r;
            }
        }
    }
    if (c->dry) return PKV_OK;
    AppendDesc *ddesc = (AppendDesc *)(c->meta + c->ml.append_desc);
    const bool inl = (int)desc.size() <= kAppendInline;       // small batch: descriptors ride in the kernel parameters
    if (!inl && (r = upload(c, ddesc, desc.data(), sizeof(AppendDesc) * desc.size(), st)) != PKV_OK) return r;
    if ((r = stager_flush(c, st)) != PKV_OK) return r;
    c->cache_written = true;
    PKV_CUDA(c, launch_append(c->geo, c->dense_pool, (const int *)(c->meta + c->ml.page_table),
                              (int *)(c->meta + c->ml.n_tokens), ddesc, inl ? desc.data() : nullptr, (int)desc.size(),
                              n_tok, layer, k, v, (int *)(c->meta + c->ml.status), st));
    return PKV_OK;
}

// Uploads a work list of (dense slot, factor slot) pairs and launches the compression kernel on it.  The device
// work list is one buffer: an upload first waits for the last kernel that read it, whatever stream that ran on.
static pkv_status run_worklist(pkv_cache *c, const std::vector<int2> &work, cudaStream_t st) {
    int2 *dwl = (int2 *)(c->workspace + c->wl.worklist);
    if (c->worklist_busy) PKV_CUDA(c, cudaStreamWaitEvent(st, c->worklist_ev, 0));
    pkv_status rr = upload(c, dwl, work.data(), sizeof(int2) * work.size(), st);
    if (rr != PKV_OK) return rr;
    if ((rr = stager_flush(c, st)) != PKV_OK) return rr;
    c->cache_written = true;
    PKV_CUDA(c, launch_compress(c->geo, c->dense_pool, c->factor_pool, dwl, (int)work.size(),
                                (int *)(c->meta + c->ml.status), st));
    if (!c->worklist_ev) PKV_CUDA(c, cudaEventCreateWithFlags(&c->worklist_ev, cudaEventDisableTiming));
    PKV_CUDA(c, cudaEventRecord(c->worklist_ev, st));
    c->worklist_busy = true;
    return PKV_OK;
}

// Global SVD form (Section 4.2): per (sequence, layer) the eligible pages are converted together.  The first
// conversion fixes the bases of the sequence's KV heads from exactly those pages (region Gram matrix, Jacobi
// eigen-solve, leading eigenvectors); then, and at every later conversion, each page stores A = X_page B^T.  Same
// page order, slot allocation and page-table updates as the page-wise path.
static pkv_status compress_global(pkv_cache *c, int l0, int l1, int64_t *n_pages_compressed, cudaStream_t st) {
    const Geometry &g = c->geo;
    int64_t done = 0;
    bool exhausted = false;
    for (int seq = 0; seq < c->cfg.max_seqs && !exhausted; ++seq) {
        for (int ly = l0; ly < l1 && !exhausted; ++ly) {
            SeqLayer &s = c->at(seq, ly);
            const int hi = std::max(g.sink_pages, s.n_tokens / c->cfg.page_size - g.recent_pages);
            if (s.f_end >= hi) continue;
            const int first = s.f_end;
            std::vector<int2> work;
            for (int p = s.f_end; p < hi && (int)work.size() < kCompressChunk; ++p) {
                if (c->factor_free.available() == 0) { exhausted = true; break; }
                const int32_t fs = c->factor_free.alloc(), ds = s.slots[p];
                work.push_back(make_int2(ds, fs));
                s.slots[p] = fs;
                c->dense_free.release(ds);
                s.f_end = p + 1;
                ++done;
            }
            if (work.empty()) continue;
            s.version++;
            if (c->dry) { s.has_basis = true; continue; }
            int2 *dwl = (int2 *)(c->workspace + c->wl.worklist);
            if (c->worklist_busy) PKV_CUDA(c, cudaStreamWaitEvent(st, c->worklist_ev, 0));
            pkv_status r = upload(c, dwl, work.data(), sizeof(int2) * work.size(), st);
            if (r != PKV_OK) return r;
            if ((r = stager_flush(c, st)) != PKV_OK) return r;
            c->cache_written = true;
            unsigned char *basis = c->meta + c->ml.basis +
                                   ((long long)seq * c->cfg.n_layers + ly) * g.n_kv_heads * g.basis_head_bytes;
            int *status = (int *)(c->meta + c->ml.status);
            if (!s.has_basis) {
                PKV_CUDA(c, launch_region_basis(g, c->dense_pool, dwl, (int)work.size(), (float *)(c->workspace + c->wl.gram),
                                                basis, status, st));
                s.has_basis = true;
            }
            PKV_CUDA(c, launch_project_pages(g, c->dense_pool, c->factor_pool, dwl, (int)work.size(), basis, status, st));
            if (!c->worklist_ev) PKV_CUDA(c, cudaEventCreateWithFlags(&c->worklist_ev, cudaEventDisableTiming));
            PKV_CUDA(c, cudaEventRecord(c->worklist_ev, st));
            c->worklist_busy = true;
            // the page-table rows of the converted pages, behind the kernels that read their dense slots
            if ((r = upload(c, dev_page_table_row(c, seq, ly) + first, s.slots.data() + first,
                            sizeof(int32_t) * (s.f_end - first), st)) != PKV_OK) return r;
            if ((r = stager_flush(c, st)) != PKV_OK) return r;
        }
    }
    c->pages_compressed += done;
    if (n_pages_compressed) *n_pages_compressed = done;
    if (exhausted) return fail(c, PKV_ERR_POOL_EXHAUSTED, "factor pool exhausted after %lld pages", (long long)done);
    return PKV_OK;
}

pkv_status pkv_compress_eligible_pages(pkv_cache *c, int32_t layer, int64_t *n_pages_compressed,
                                       void *stream) {
    if (!c) return PKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (n_pages_compressed) *n_pages_compressed = 0;
    if (layer < -1 || layer >= c->cfg.n_layers) return fail(c, PKV_ERR_INVALID_ARG, "layer %d out of range", layer);
    if (!c->dry && is_capturing(st))
        return fail(c, PKV_ERR_UNSUPPORTED, "pkv_compress_eligible_pages cannot be captured into a CUDA graph");
    if (layer < 0 ? c->n_pending > 0 : c->pending[layer].active)
        return fail(c, PKV_ERR_UNSUPPORTED, "a compression begun with pkv_compress_begin is not committed yet");
    const Geometry &g = c->geo;
    const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? c->cfg.n_layers : layer + 1;
    if (g.global_rank > 0) return compress_global(c, l0, l1, n_pages_compressed, st);
    std::vector<int2> work;
    int64_t done = 0;
    bool exhausted = false;
    pkv_status r;
    auto flush_work = [&]() -> pkv_status {
        if (work.empty() || c->dry) { work.clear(); return PKV_OK; }
        pkv_status rr = run_worklist(c, work, st);
        work.clear();
        return rr;
    };
    // Page-table uploads of converted pages are queued behind the kernel that reads the dense slots.
    struct Flip { int seq, layer, first, last; };
    std::vector<Flip> flips;
    auto flush_flips = [&]() -> pkv_status {
        for (const Flip &f : flips) {
            if (c->dry) break;
            const SeqLayer &s = c->at(f.seq, f.layer);
            pkv_status rr = upload(c, dev_page_table_row(c, f.seq, f.layer) + f.first, s.slots.data() + f.first,
                                   sizeof(int32_t) * (f.last - f.first), st);
            if (rr != PKV_OK) return rr;
        }
        flips.clear();
        return stager_flush(c, st);
    };
    for (int seq = 0; seq < c->cfg.max_seqs && !exhausted; ++seq) {
        for (int ly = l0; ly < l1 && !exhausted; ++ly) {
            SeqLayer &s = c->at(seq, ly);
            const int n_c = s.n_tokens / c->cfg.page_size;
            const int hi = std::max(g.sink_pages, n_c - g.recent_pages);   // eligible: sink_pages <= p < hi
            if (s.f_end >= hi) continue;
            const int first = s.f_end;
            for (int p = s.f_end; p < hi; ++p) {
                if (c->factor_free.available() == 0) { exhausted = true; break; }
                int32_t fs = c->factor_free.alloc();
                int32_t ds = s.slots[p];
                work.push_back(make_int2(ds, fs));
                s.slots[p] = fs;
                c->dense_free.release(ds);
                s.f_end = p + 1;
                ++done;
                if ((int)work.size() == kCompressChunk) {
                    flips.push_back(Flip{seq, ly, first, s.f_end});
                    if ((r = flush_work()) != PKV_OK) return r;
                    if ((r = flush_flips()) != PKV_OK) return r;
                }
            }
            if (s.f_end > first) {
                s.version++;
                flips.push_back(Flip{seq, ly, first, s.f_end});
            }
        }
    }
    if ((r = flush_work()) != PKV_OK) return r;
    if ((r = flush_flips()) != PKV_OK) return r;
    c->pages_compressed += done;
    if (n_pages_compressed) *n_pages_compressed = done;
    if (exhausted) return fail(c, PKV_ERR_POOL_EXHAUSTED, "factor pool exhausted after %lld pages", (long long)done);
    return PKV_OK;
}

pkv_status pkv_compress_begin(pkv_cache *c, int32_t layer, void *main_stream, void *side_stream,
                              int64_t *n_pages_begun) {
    if (!c) return PKV_ERR_INVALID_ARG;
    cudaStream_t ms = (cudaStream_t)main_stream, ss = (cudaStream_t)side_stream;
    if (n_pages_begun) *n_pages_begun = 0;
    if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, PKV_ERR_INVALID_ARG, "layer %d out of range", layer);
    PendingCompress &pd = c->pending[layer];
    if (c->geo.global_rank > 0) return fail(c, PKV_ERR_UNSUPPORTED, "pkv_compress_begin is not available in the Global SVD form");
    if (pd.active) return fail(c, PKV_ERR_UNSUPPORTED, "layer %d already has an uncommitted compression", layer);
    if (!c->dry && (is_capturing(ms) || is_capturing(ss)))
        return fail(c, PKV_ERR_UNSUPPORTED, "pkv_compress_begin cannot be captured into a CUDA graph");
    const Geometry &g = c->geo;
    pd.pages.clear();
    bool exhausted = false;
    for (int seq = 0; seq < c->cfg.max_seqs && !exhausted; ++seq) {
        const SeqLayer &s = c->at(seq, layer);
        const int hi = std::max(g.sink_pages, s.n_tokens / c->cfg.page_size - g.recent_pages);
        for (int p = s.f_end; p < hi; ++p) {
            if (c->factor_free.available() == 0) { exhausted = true; break; }
            pd.pages.push_back(PendingPage{seq, p, s.slots[p], c->factor_free.alloc()});
        }
    }
    if (n_pages_begun) *n_pages_begun = (int64_t)pd.pages.size();
    if (!pd.pages.empty()) {
        pd.active = true;
        c->n_pending++;
        if (!c->dry) {
            // the pages were written by work enqueued on the main stream: the side stream starts behind it
            if (!c->order_ev) PKV_CUDA(c, cudaEventCreateWithFlags(&c->order_ev, cudaEventDisableTiming));
            if (!pd.done) PKV_CUDA(c, cudaEventCreateWithFlags(&pd.done, cudaEventDisableTiming));
            PKV_CUDA(c, cudaEventRecord(c->order_ev, ms));
            PKV_CUDA(c, cudaStreamWaitEvent(ss, c->order_ev, 0));
            std::vector<int2> work;
            pkv_status r;
            for (size_t i = 0; i < pd.pages.size(); ++i) {
                work.push_back(make_int2(pd.pages[i].dense_slot, pd.pages[i].factor_slot));
                if ((int)work.size() == kCompressChunk || i + 1 == pd.pages.size()) {
                    const bool written = c->cache_written;       // nothing a decode launch reads changes before the commit
                    r = run_worklist(c, work, ss);
                    c->cache_written = written;
                    if (r != PKV_OK) return r;
                    work.clear();
                }
            }
            PKV_CUDA(c, cudaEventRecord(pd.done, ss));
        }
    }
    if (exhausted)
        return fail(c, PKV_ERR_POOL_EXHAUSTED, "factor pool exhausted after %lld pages", (long long)pd.pages.size());
    return PKV_OK;
}

pkv_status pkv_compress_commit(pkv_cache *c, int32_t layer, void *main_stream, int64_t *n_pages_compressed) {
    if (!c) return PKV_ERR_INVALID_ARG;
    cudaStream_t ms = (cudaStream_t)main_stream;
    if (n_pages_compressed) *n_pages_compressed = 0;
    if (layer < -1 || layer >= c->cfg.n_layers) return fail(c, PKV_ERR_INVALID_ARG, "layer %d out of range", layer);
    if (!c->dry && is_capturing(ms))
        return fail(c, PKV_ERR_UNSUPPORTED, "pkv_compress_commit cannot be captured into a CUDA graph");
    const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? c->cfg.n_layers : layer + 1;
    int64_t done = 0;
    for (int ly = l0; ly < l1; ++ly) {
        PendingCompress &pd = c->pending[ly];
        if (!pd.active) continue;
        if (!c->dry) PKV_CUDA(c, cudaStreamWaitEvent(ms, pd.done, 0));
        // the same state changes, in the same order, as pkv_compress_eligible_pages makes page by page
        for (size_t i = 0; i < pd.pages.size();) {
            const int seq = pd.pages[i].seq;
            SeqLayer &s = c->at(seq, ly);
            const int first = pd.pages[i].page;
            for (; i < pd.pages.size() && pd.pages[i].seq == seq; ++i) {
                const PendingPage &pp = pd.pages[i];
                s.slots[pp.page] = pp.factor_slot;
                c->dense_free.release(pp.dense_slot);
                s.f_end = pp.page + 1;
                ++done;
            }
            s.version++;
            if (!c->dry) {
                pkv_status r = upload(c, dev_page_table_row(c, seq, ly) + first, s.slots.data() + first,
                                      sizeof(int32_t) * (s.f_end - first), ms);
                if (r != PKV_OK) return r;
            }
        }
        pd.pages.clear();
        pd.active = false;
        c->n_pending--;
        c->cache_written = true;
    }
    if (!c->dry) { pkv_status r = stager_flush(c, ms); if (r != PKV_OK) return r; }
    c->pages_compressed += done;
    if (n_pages_compressed) *n_pages_compressed = done;
    return PKV_OK;
}

static pkv_status decode_impl(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids, int32_t q_len,
                              const void *q, void *out, float *out_f32, float *state, void *stream,
                              bool static_scratch = false);

pkv_status pkv_decode_attention(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                const void *q, void *out, float *out_f32, void *stream) {
    return decode_impl(c, layer, n_seqs, seq_ids, 1, q, out, out_f32, nullptr, stream);
}

pkv_status pkv_decode_attention_multi(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                      int32_t q_len, const void *q, void *out, float *out_f32, void *stream) {
    return decode_impl(c, layer, n_seqs, seq_ids, q_len, q, out, out_f32, nullptr, stream);
}

// Same validation, plan and accounting as pkv_decode_attention(); only the split-K scratch differs.
pkv_status pkv_decode_attention_static_scratch(pkv_cache *c, int32_t layer, int32_t n_seqs,
                                               const int32_t *seq_ids, const void *q, void *out, float *out_f32,
                                               void *stream) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (c->dry) return fail(c, PKV_ERR_INVALID_ARG, "no device buffers in dry-run mode");
    if (!out) return fail(c, PKV_ERR_INVALID_ARG, "q or out is NULL");
    return decode_impl(c, layer, n_seqs, seq_ids, 1, q, out, out_f32, nullptr, stream, true);
}

pkv_status pkv_decode_attention_partial(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                        const void *q, float *state, void *stream) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (c->cfg.decode_variant == 1)
        return fail(c, PKV_ERR_UNSUPPORTED, "pkv_decode_attention_partial needs the tensor-core kernel (decode_variant 0)");
    if (!c->dry && !state) return fail(c, PKV_ERR_INVALID_ARG, "state is NULL");
    return decode_impl(c, layer, n_seqs, seq_ids, 1, q, nullptr, nullptr, state, stream);
}

pkv_status pkv_merge_attention_states(const float *states, int32_t n_shards, int64_t n_rows, void *out, float *out_f32,
                                      void *stream) {
    if (!states || n_shards < 1 || n_rows < 0 || (!out && !out_f32)) return PKV_ERR_INVALID_ARG;
    if (((uintptr_t)states & 7) || ((uintptr_t)out & 7) || ((uintptr_t)out_f32 & 15)) return PKV_ERR_INVALID_ARG;
    return launch_merge_states(states, n_shards, n_rows, out, out_f32, (cudaStream_t)stream) == cudaSuccess
               ? PKV_OK : PKV_ERR_CUDA;
}

// Alignment the kernels rely on: q rows are read as 32-bit words, out is written 8 bytes at a time, out_f32 16,
// state rows (d + 2 floats) 8.
static bool misaligned(const void *p, uintptr_t a) { return p && ((uintptr_t)p & (a - 1)) != 0; }

static pkv_status decode_impl(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids, int32_t q_len,
                              const void *q, void *out, float *out_f32, float *state, void *stream,
                              bool static_scratch) {
    if (!c) return PKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, PKV_ERR_INVALID_ARG, "layer %d out of range", layer);
    pkv_status r = check_seq_list(c, n_seqs, seq_ids);
    if (r != PKV_OK) return r;
    for (int i = 0; i < n_seqs; ++i)
        if (c->at(seq_ids[i], layer).n_tokens == 0)
            return fail(c, PKV_ERR_INVALID_ARG, "sequence %d has no tokens in layer %d", seq_ids[i], layer);
    if (q_len < 1 || q_len > 32767) return fail(c, PKV_ERR_INVALID_ARG, "q_len %d out of range", q_len);
    if (q_len > 1) {
        if (c->geo.global_rank > 0)
            return fail(c, PKV_ERR_UNSUPPORTED, "several queries per sequence are not available in the Global SVD form");
        if (c->cfg.decode_variant == 1)
            return fail(c, PKV_ERR_UNSUPPORTED, "several queries per sequence need the tensor-core kernels (decode_variant 0)");
        if (!uses_row_blocks(c, q_len, n_seqs) && (long long)n_seqs * block_slots_per_seq(c->geo, q_len) > c->cfg.max_seqs)
            return fail(c, PKV_ERR_INVALID_ARG, "%d sequences x %d query blocks exceed max_seqs = %d", n_seqs,
                        block_slots_per_seq(c->geo, q_len), c->cfg.max_seqs);
        for (int i = 0; i < n_seqs; ++i) {
            const SeqLayer &s = c->at(seq_ids[i], layer);
            // every query must see every factor page whole (and at least its own position)
            const int first_visible = s.n_tokens - q_len + 1;
            if (first_visible < 1 || (s.f_end > c->geo.sink_pages && s.f_end * c->cfg.page_size > first_visible))
                return fail(c, PKV_ERR_INVALID_ARG, "sequence %d: the %d newest positions reach into compressed pages "
                            "or past the start (%d tokens, factor pages end at token %d)", seq_ids[i], q_len, s.n_tokens,
                            s.f_end > c->geo.sink_pages ? s.f_end * c->cfg.page_size : 0);
        }
    }
    if (!c->dry && (!q || (!out && !state))) return fail(c, PKV_ERR_INVALID_ARG, "q or out is NULL");
    if (misaligned(q, 4) || misaligned(out, 8) || misaligned(out_f32, 16) || misaligned(state, 8))
        return fail(c, PKV_ERR_INVALID_ARG, "misaligned pointer: q needs 4-byte, out 8-byte, out_f32 16-byte, state 8-byte alignment");
    if (!plan_is_current(c, layer, n_seqs, seq_ids, q_len)) {
        // the plan is uploaded through the staging ring: a copy recorded into a graph would replay stale bytes
        if (!c->dry && is_capturing(st))
            return fail(c, PKV_ERR_UNSUPPORTED, "the decode plan of layer %d must be rebuilt: call pkv_decode_attention "
                        "once outside the stream capture for this layer and batch first", layer);
        if ((r = build_plan(c, layer, n_seqs, seq_ids, q_len, st)) != PKV_OK) return r;
    }
    const PlanCache &pc = c->plans[layer];
    int64_t bytes = 2LL * n_seqs * q_len * c->cfg.n_q_heads * kRowBytes;  // q and out
    for (int i = 0; i < n_seqs; ++i) {
        const SeqLayer &s = c->at(seq_ids[i], layer);
        const int n_pages = (int)s.slots.size();
        const int nf = std::min(s.f_end, n_pages) - std::min(c->geo.sink_pages, n_pages);
        const bool last_dense = !(n_pages - 1 >= c->geo.sink_pages && n_pages - 1 < s.f_end);
        int64_t rows = (int64_t)(n_pages - nf) * c->cfg.page_size;
        if (last_dense) rows -= (int64_t)n_pages * c->cfg.page_size - s.n_tokens;  // unfilled rows of the last page are not read
        bytes += (int64_t)c->geo.n_kv_heads * ((int64_t)nf * c->geo.blob_bytes + rows * 2 * kRowBytes);
        if (nf > 0) bytes += (int64_t)c->geo.n_kv_heads * c->geo.basis_head_bytes;     // Global SVD form: the shared bases, once
    }
    c->last_decode_bytes = bytes;
    c->last_decode_units = pc.units;
    if (c->dry) return PKV_OK;
    DecodeArgs a;
    a.geo = c->geo;
    a.dense_pool = c->dense_pool; a.factor_pool = c->factor_pool;
    a.page_table = (const int *)(c->meta + c->ml.page_table);
    a.n_tokens = (const int *)(c->meta + c->ml.n_tokens);
    a.basis = c->meta + c->ml.basis;
    a.plan = c->meta + c->ml.plans + c->ml.plan_stride * layer;
    a.plan_cta = c->ml.plan_cta; a.plan_entry = c->ml.plan_entry; a.plan_seg = c->ml.plan_seg;
    a.plan_cta_entry = c->ml.plan_cta_entry;
    a.q = q; a.out = out; a.out_f32 = out_f32;
    a.state = state;
    a.wait_clocks = c->wait_clocks;
    a.drop_unit = c->drop_unit;
    c->drop_unit = -1;                                    // (one launch only)
    if (c->tickets_dirty && !is_capturing(st)) {
        // an earlier launch gave up on a wait and may have left merge tickets drawn: start from zero again
        PKV_CUDA(c, cudaMemsetAsync(c->workspace + c->wl.tickets, 0, (size_t)(c->wl.tickets_stride * c->wl.n_sets), st));
        c->tickets_dirty = false;
    }
    a.q_len = q_len;
    a.q_tpt = queries_per_tile(c->geo, q_len);
    a.q_group = sibling_group(c->geo, q_len);
    a.q_nblk = block_slots_per_seq(c->geo, q_len);
    a.q_cols = a.q_tpt * c->geo.group;
    // decode_overlap = 2: launches never wait for one another, so launches in flight must not share split-K
    // scratch.  The scratch rotates over wl.n_sets sets and every (n_sets-1)-th launch is a plain
    // one (no programmatic serialization: it starts after all earlier work on the stream has finished), so
    // between two users of a set the stream has always drained once.
    int buf = 0;
    // whatever the overlap mode, a decode that follows this library's own append / compression kernels is
    // launched the ordinary way, after everything before it on the stream has finished
    a.plain_launch = c->cache_written ? 1 : 0;
    c->cache_written = false;
    if (uses_row_blocks(c, q_len, n_seqs)) {
        // one ordinary launch (starts after everything before it on the stream); no split-K scratch involved
        a.partials = nullptr; a.tickets = nullptr; a.gpartials = nullptr; a.gtickets = nullptr;
        a.status = (int *)(c->meta + c->ml.status);
        a.layer = layer;
        a.variant = c->cfg.decode_variant == 3 ? 3 : 0; a.overlap = 0; a.plain_launch = 1; a.trace = nullptr;
        c->cache_written = false;
        // tcgen05 kernel: with fewer row blocks than half the CTAs the GPU holds, each block's sequence is cut into
        // ranges of at least kRbMinPages pages, one CTA each
        a.rb_splits = 1;
        a.rb_partials = (float *)(c->workspace + c->wl.rb_partials);
        if (a.variant == 0 && c->row_maps.valid) {
            const long long n_blocks = (long long)n_seqs * c->geo.n_kv_heads * (((long long)q_len * c->geo.group + 127) / 128);
            int longest = 0;
            for (int i = 0; i < n_seqs; ++i) longest = std::max(longest, c->at(seq_ids[i], layer).n_tokens);
            a.rb_splits = row_block_ranges(n_blocks, longest, c->cfg.page_size, c->n_sms);
        }
        PKV_CUDA(c, launch_decode_blocks(a, n_seqs, c->row_maps, st));
        return PKV_OK;
    }
    if (static_scratch) {
        // partial states and tickets live in the library's own array (set by the launcher); the memset that clears
        // the tickets already orders the launch behind all earlier work on the stream
        a.partials = nullptr; a.tickets = nullptr; a.gpartials = nullptr; a.gtickets = nullptr;
        a.plain_launch = 0;
        a.status = (int *)(c->meta + c->ml.status);
        a.layer = layer;
        a.variant = c->cfg.decode_variant;
        a.overlap = c->cfg.decode_overlap;
        a.trace = nullptr;
        const char *why = "";
        cudaError_t e = launch_decode_static_scratch(a, pc.n_segs, st, &why);
        if (e == cudaErrorInvalidValue && why[0])
            return fail(c, PKV_ERR_INVALID_ARG, "pkv_decode_attention_static_scratch: %s", why);
        if (e != cudaSuccess)
            return fail(c, PKV_ERR_CUDA, "pkv_decode_attention_static_scratch: %s: %s", why, cudaGetErrorString(e));
        return PKV_OK;
    }
    if (c->cfg.decode_overlap == 2 && c->cfg.decode_variant != 1) {
        // Recorded into a CUDA graph, a launch keeps the set chosen here in every replay.  That is sound inside a
        // graph (same rotation, same draining launches) and between graph launches (each starts after the previous
        // one has finished); a launch outside a graph could however meet a set that a graph's last launches still
        // use, so once this cache has been captured its launches outside a graph are ordinary ones.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        PKV_CUDA(c, cudaStreamIsCapturing(st, &cap));
        if (cap != cudaStreamCaptureStatusNone) c->captured_mode2 = true;
        else if (c->captured_mode2) a.plain_launch = 1;
        buf = (int)(c->decode_seq % c->wl.n_sets);
        if ((c->decode_seq % (c->wl.n_sets - 1)) == 0) a.plain_launch = 1;
        c->decode_seq++;
    }
    a.partials = (float *)(c->workspace + c->wl.partials + c->wl.partials_stride * buf);
    a.tickets = (int *)(c->workspace + c->wl.tickets + c->wl.tickets_stride * buf);
    a.gpartials = a.partials + c->wl.n_flat * kPartialFloats;
    a.gtickets = a.tickets + c->wl.n_seg_tickets;
    a.status = (int *)(c->meta + c->ml.status);
    a.layer = layer;
    a.variant = c->cfg.decode_variant;
    a.overlap = c->cfg.decode_overlap;
    a.trace = c->trace ? (long long *)(c->workspace + c->wl.trace) : nullptr;
    PKV_CUDA(c, launch_decode(a, pc.n_segs, st));
    return PKV_OK;
}

pkv_status pkv_decode_attention_host(pkv_cache *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                     const void *q_host, void *out_host, void *q_stage, void *out_stage,
                                     void *stream) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (c->dry) return pkv_decode_attention(c, layer, n_seqs, seq_ids, nullptr, nullptr, nullptr, stream);
    if (!q_host || !out_host || !q_stage || !out_stage || n_seqs <= 0)
        return fail(c, PKV_ERR_INVALID_ARG, "host or staging buffer is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bytes = (size_t)n_seqs * c->cfg.n_q_heads * kRowBytes;
    // Pinned, device-mapped host buffers: the kernel reads q and writes out across the bus itself, so no
    // copy operation sits between consecutive launches (they keep overlapping).  The bytes still cross
    // the bus inside this call.  Anything else goes through the staging buffers.
    auto mapped = [](const void *p) -> void * {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
    };
    void *q_dev = mapped(q_host), *out_dev = mapped(out_host);
    if (q_dev && out_dev) return pkv_decode_attention(c, layer, n_seqs, seq_ids, q_dev, out_dev, nullptr, stream);
    PKV_CUDA(c, cudaMemcpyAsync(q_stage, q_host, bytes, cudaMemcpyHostToDevice, st));
    pkv_status r = pkv_decode_attention(c, layer, n_seqs, seq_ids, q_stage, out_stage, nullptr, stream);
    if (r != PKV_OK) return r;
    PKV_CUDA(c, cudaMemcpyAsync(out_host, out_stage, bytes, cudaMemcpyDeviceToHost, st));
    return PKV_OK;
}

pkv_status pkv_get_page_table(const pkv_cache *c, int32_t seq, int32_t layer, int32_t *kinds,
                              int32_t *slots, int32_t *n_pages, int32_t *n_tokens) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (seq < 0 || seq >= c->cfg.max_seqs) return PKV_ERR_BAD_SEQ;
    if (layer < 0 || layer >= c->cfg.n_layers) return PKV_ERR_INVALID_ARG;
    const SeqLayer &s = c->at(seq, layer);
    for (size_t p = 0; p < s.slots.size(); ++p) {
        if (kinds) kinds[p] = ((int)p >= c->geo.sink_pages && (int)p < s.f_end) ? PKV_KIND_FACTOR : PKV_KIND_DENSE;
        if (slots) slots[p] = s.slots[p];
    }
    if (n_pages) *n_pages = (int32_t)s.slots.size();
    if (n_tokens) *n_tokens = s.n_tokens;
    return PKV_OK;
}

pkv_status pkv_get_decode_plan(const pkv_cache *c, int32_t layer, int32_t *n_used_ctas, int32_t *cta_starts,
                               int32_t *n_segs, int32_t *seg_parts) {
    if (!c || layer < 0 || layer >= c->cfg.n_layers) return PKV_ERR_INVALID_ARG;
    const PlanCache &pc = c->plans[layer];
    if (!pc.valid) return PKV_ERR_INVALID_ARG;
    if (n_used_ctas) *n_used_ctas = (int32_t)pc.ctas.size() - 1;
    if (n_segs) *n_segs = pc.n_segs;
    if (cta_starts)
        for (size_t j = 0; j < pc.ctas.size(); ++j) {
            cta_starts[3 * j] = pc.ctas[j].entry; cta_starts[3 * j + 1] = pc.ctas[j].head; cta_starts[3 * j + 2] = pc.ctas[j].unit;
        }
    if (seg_parts)
        for (int s = 0; s < pc.n_segs; ++s) { seg_parts[2 * s] = pc.segs[s].cta_first; seg_parts[2 * s + 1] = pc.segs[s].n_parts; }
    return PKV_OK;
}

pkv_status pkv_get_decode_trace(pkv_cache *c, int64_t *out, int32_t n_ctas, void *stream) {
    if (!c || !out || c->dry || n_ctas <= 0 || n_ctas > c->geo.n_ctas) return PKV_ERR_INVALID_ARG;
    if (!c->trace) return fail(c, PKV_ERR_INVALID_ARG, "tracing is off: set PKV_DECODE_TRACE=1 before pkv_init_cache");
    PKV_CUDA(c, cudaStreamSynchronize((cudaStream_t)stream));
    PKV_CUDA(c, cudaMemcpy(out, c->workspace + c->wl.trace, 8 * (size_t)kTraceSlots * n_ctas, cudaMemcpyDeviceToHost));
    return PKV_OK;
}

pkv_status pkv_get_stats(pkv_cache *c, pkv_stats *out, void *stream) {
    if (!c || !out) return PKV_ERR_INVALID_ARG;
    memset(out, 0, sizeof *out);
    out->dense_slots_in_use = c->dense_free.in_use();
    out->factor_slots_in_use = c->factor_free.in_use();
    out->pages_compressed = c->pages_compressed;
    out->last_decode_bytes = c->last_decode_bytes;
    out->last_decode_units = c->last_decode_units;
    if (!c->dry) {
        int32_t st[kStatusWords];
        PKV_CUDA(c, cudaStreamSynchronize((cudaStream_t)stream));
        PKV_CUDA(c, cudaMemcpy(st, c->meta + c->ml.status, sizeof st, cudaMemcpyDeviceToHost));
        out->device_timeouts = st[0];
        if (st[0] != c->timeouts_seen) { c->timeouts_seen = st[0]; c->tickets_dirty = true; }
        out->page_svds_not_converged = st[1];
        out->bad_slot_indices = st[2];
        uint64_t wide[2];
        memcpy(wide, st + 4, sizeof wide);
        out->jacobi_rounds = (int64_t)wide[0];
        out->page_svds = (int64_t)wide[1];
    }
    return PKV_OK;
}

pkv_status pkv_free_seq(pkv_cache *c, int32_t seq) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (seq < 0 || seq >= c->cfg.max_seqs) return fail(c, PKV_ERR_BAD_SEQ, "sequence id %d out of range", seq);
    for (int ly = 0; ly < c->cfg.n_layers && c->n_pending > 0; ++ly)
        for (const PendingPage &pp : c->pending[ly].pages)
            if (pp.seq == seq)
                return fail(c, PKV_ERR_UNSUPPORTED, "sequence %d has pages in an uncommitted compression (layer %d)", seq, ly);
    for (int ly = 0; ly < c->cfg.n_layers; ++ly) {
        SeqLayer &s = c->at(seq, ly);
        for (size_t p = 0; p < s.slots.size(); ++p) {
            if ((int)p >= c->geo.sink_pages && (int)p < s.f_end) c->factor_free.release(s.slots[p]);
            else c->dense_free.release(s.slots[p]);
        }
        s.slots.clear();
        s.n_tokens = 0;
        s.f_end = c->geo.sink_pages;
        s.has_basis = false;
        s.version++;
    }
    return PKV_OK;
}

static pkv_status slot_args(pkv_cache *c, int64_t slot, int64_t n_slots, int32_t head) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (c->dry) return fail(c, PKV_ERR_INVALID_ARG, "no device buffers in dry-run mode");
    if (slot < 0 || slot >= n_slots || head < 0 || head >= c->cfg.n_kv_heads)
        return fail(c, PKV_ERR_INVALID_ARG, "slot or head out of range");
    return PKV_OK;
}

pkv_status pkv_read_factors(pkv_cache *c, int64_t slot, int32_t head, void *A_k, void *B_k, void *A_v,
                            void *B_v, void *stream) {
    pkv_status r = slot_args(c, slot, c ? c->cfg.n_factor_slots : 0, head);
    if (r != PKV_OK) return r;
    if (!A_k || !A_v || (c->geo.global_rank == 0 && (!B_k || !B_v))) return fail(c, PKV_ERR_INVALID_ARG, "output pointer is NULL");
    const unsigned char *blob = c->factor_pool + slot * c->geo.factor_slot_bytes + (int64_t)head * c->geo.blob_bytes;
    PKV_CUDA(c, launch_read_factors(c->geo, blob, A_k, B_k, A_v, B_v, (cudaStream_t)stream));
    return PKV_OK;
}

pkv_status pkv_write_factors(pkv_cache *c, int64_t slot, int32_t head, const void *A_k, const void *B_k,
                             const void *A_v, const void *B_v, void *stream) {
    pkv_status r = slot_args(c, slot, c ? c->cfg.n_factor_slots : 0, head);
    if (r != PKV_OK) return r;
    if (!A_k || !B_k || !A_v || !B_v) return fail(c, PKV_ERR_INVALID_ARG, "input pointer is NULL");
    if (c->geo.factor_bits == 4) return fail(c, PKV_ERR_UNSUPPORTED, "pkv_write_factors is not available with INT4 factors");
    if (c->geo.global_rank > 0) return fail(c, PKV_ERR_UNSUPPORTED, "pkv_write_factors is not available in the Global SVD form");
    unsigned char *blob = c->factor_pool + slot * c->geo.factor_slot_bytes + (int64_t)head * c->geo.blob_bytes;
    c->cache_written = true;                     // the next decode launch must not start ahead of this kernel
    PKV_CUDA(c, launch_write_factors(c->geo, blob, A_k, B_k, A_v, B_v, (cudaStream_t)stream));
    return PKV_OK;
}

pkv_status pkv_get_row_block_ranges(int64_t n_row_blocks, int32_t longest_tokens, int32_t page_size, int32_t n_sms,
                                    int32_t *n_ranges) {
    if (!n_ranges || n_row_blocks < 1 || longest_tokens < 1 || page_size < 1 || n_sms < 1) return PKV_ERR_INVALID_ARG;
    *n_ranges = row_block_ranges(n_row_blocks, longest_tokens, page_size, n_sms);
    return PKV_OK;
}

pkv_status pkv_get_rotation_schedule(int32_t page_size, uint8_t *members, int64_t capacity, int32_t *n_rounds,
                                     int32_t *groups_per_round, int32_t *group_size) {
    int nr = 0, ng = 0, gs = 0;
    if (!pkv::rotation_schedule(page_size, members, capacity, &nr, &ng, &gs)) return PKV_ERR_INVALID_ARG;
    *n_rounds = nr; *groups_per_round = ng; *group_size = gs;
    return PKV_OK;
}

pkv_status pkv_read_basis(pkv_cache *c, int32_t seq, int32_t layer, int32_t head, void *B_k, void *B_v, void *stream) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (c->dry) return fail(c, PKV_ERR_INVALID_ARG, "no device buffers in dry-run mode");
    if (c->geo.global_rank == 0) return fail(c, PKV_ERR_INVALID_ARG, "the cache does not use the Global SVD form");
    if (seq < 0 || seq >= c->cfg.max_seqs) return fail(c, PKV_ERR_BAD_SEQ, "sequence id %d out of range", seq);
    if (layer < 0 || layer >= c->cfg.n_layers || head < 0 || head >= c->cfg.n_kv_heads || !B_k || !B_v)
        return fail(c, PKV_ERR_INVALID_ARG, "layer or head out of range, or an output pointer is NULL");
    if (!c->at(seq, layer).has_basis) return fail(c, PKV_ERR_INVALID_ARG, "sequence %d has no basis in layer %d yet", seq, layer);
    const unsigned char *b = c->meta + c->ml.basis +
                             (((long long)seq * c->cfg.n_layers + layer) * c->geo.n_kv_heads + head) * c->geo.basis_head_bytes;
    PKV_CUDA(c, launch_read_basis(c->geo, b, B_k, B_v, (cudaStream_t)stream));
    return PKV_OK;
}

pkv_status pkv_read_dense(pkv_cache *c, int64_t slot, int32_t head, void *K, void *V, void *stream) {
    pkv_status r = slot_args(c, slot, c ? c->cfg.n_dense_slots : 0, head);
    if (r != PKV_OK) return r;
    if (!K || !V) return fail(c, PKV_ERR_INVALID_ARG, "output pointer is NULL");
    const unsigned char *base = c->dense_pool + slot * c->geo.dense_slot_bytes + (int64_t)head * c->geo.dense_head_bytes;
    PKV_CUDA(c, launch_read_dense(c->geo, base, K, V, (cudaStream_t)stream));
    return PKV_OK;
}

}  // extern "C"
