// C ABI of the library: configuration checks, workspace plan, stage sequencing.
// Every numeric step runs in the kernels launched from here.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/liec.h"
#include "kernels.h"
#include "plan.h"
#include "topk_common.cuh"

using namespace liec;

namespace {

thread_local char g_no_ctx_error[256] = "";

struct Region {
    size_t off = 0, bytes = 0;
};

struct Plan {
    int32_t N = 0, T = 0, TT = 0, KTT = 0;
    int64_t d = 0, W = 0, K = 0, CAP = 0, cap_max = 0, down_CAP = 0;
    std::vector<int64_t> seg_off, word_off, k_off, cap_off, down_cap_off, topk_k;
    std::vector<int32_t> tile_prefix, tile_seg, small_seg, large_seg, ktile_prefix, ktile_seg;
    Region r_seg_off, r_word_off, r_k_off, r_cap_off, r_down_cap_off, r_tile_prefix, r_tile_seg, r_small_seg, r_large_seg, r_status;
    Region r_tel_partials, r_tel_e, r_tel_v, r_tel_g, r_tel_kept, r_ktile_prefix, r_ktile_seg;
    Region r_up_words, r_up_scales, r_up_partials, r_down_words, r_down_scales, r_down_partials, r_vbuf;
    Region r_up_idx, r_up_val, r_down_idx, r_down_val;
    Region r_up_hist, r_down_hist, r_up_hist2, r_down_hist2, r_up_sel, r_down_sel;
    Region r_up_cand_idx, r_up_cand_val, r_down_cand_idx, r_down_cand_val;
    Region r_up_tile_meta, r_down_tile_meta, r_up_outbase, r_down_outbase, r_up_scan_parts, r_down_scan_parts, r_gen_scan_parts;
    Region r_gen_sets, r_gen_val, r_gen_hist, r_gen_hist2, r_gen_sel, r_gen_cand_idx, r_gen_cand_val, r_gen_meta, r_gen_outbase;
    size_t total = 0;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carver {
    size_t cursor = 0;
    Region take(size_t bytes, size_t align = 256) {
        Region r;
        cursor = align_up(cursor, align);
        r.off = cursor;
        r.bytes = bytes;
        cursor += bytes;
        return r;
    }
};

liec_status fail(std::string *msg, liec_status st, const char *text) {
    if (msg) *msg = text;
    return st;
}

liec_status make_plan(const liec_config *cfg, Plan &pl, std::string *msg) {
    if (!cfg) return fail(msg, LIEC_ERR_INVALID_ARG, "config is NULL");
    if (cfg->num_workers < 1) return fail(msg, LIEC_ERR_INVALID_ARG, "num_workers must be >= 1");
    if (cfg->num_workers > 65535) return fail(msg, LIEC_ERR_UNSUPPORTED, "num_workers above 65535 (grid y limit)");
    if (cfg->dim < 1) return fail(msg, LIEC_ERR_INVALID_ARG, "dim must be >= 1");
    if (cfg->dim >= (int64_t(1) << 32)) return fail(msg, LIEC_ERR_UNSUPPORTED, "dim must be below 2^32 (32-bit indices)");
    if (cfg->num_segments < 1) return fail(msg, LIEC_ERR_INVALID_ARG, "num_segments must be >= 1");
    if (cfg->num_segments > 65535) return fail(msg, LIEC_ERR_UNSUPPORTED, "num_segments above 65535 (grid limit)");
    if (!cfg->seg_offsets) return fail(msg, LIEC_ERR_INVALID_ARG, "seg_offsets is NULL");
    auto comp_ok = [](int32_t c) { return c == LIEC_COMP_IDENTITY || c == LIEC_COMP_SCALED_SIGN || c == LIEC_COMP_TOPK || c == LIEC_COMP_RANDK; };
    if (!comp_ok(cfg->uplink) || !comp_ok(cfg->downlink)) return fail(msg, LIEC_ERR_INVALID_ARG, "unknown compressor");
    if (cfg->grad_dtype != LIEC_F32 && cfg->grad_dtype != LIEC_BF16) return fail(msg, LIEC_ERR_INVALID_ARG, "unknown grad_dtype");
    const int T = cfg->num_segments;
    if (cfg->seg_offsets[0] != 0 || cfg->seg_offsets[T] != cfg->dim)
        return fail(msg, LIEC_ERR_INVALID_ARG, "seg_offsets must start at 0 and end at dim");
    for (int t = 0; t < T; ++t)
        if (cfg->seg_offsets[t + 1] <= cfg->seg_offsets[t])
            return fail(msg, LIEC_ERR_INVALID_ARG, "seg_offsets must be strictly increasing");
    const bool any_topk = comp_is_sparse(cfg->uplink) || comp_is_sparse(cfg->downlink);  // sides with k entries per segment
    if (any_topk) {
        if (!cfg->topk_k) return fail(msg, LIEC_ERR_INVALID_ARG, "topk_k is NULL but a side uses top-k or random-k");
        for (int t = 0; t < T; ++t) {
            int64_t n = cfg->seg_offsets[t + 1] - cfg->seg_offsets[t];
            if (cfg->topk_k[t] < 1 || cfg->topk_k[t] > n)
                return fail(msg, LIEC_ERR_INVALID_ARG, "topk_k[t] must satisfy 1 <= k_t <= n_t");
        }
    }

    pl.N = cfg->num_workers;
    pl.T = T;
    pl.d = cfg->dim;
    pl.seg_off.assign(cfg->seg_offsets, cfg->seg_offsets + T + 1);
    pl.word_off.assign(T + 1, 0);
    pl.k_off.assign(T + 1, 0);
    pl.cap_off.assign(T + 1, 0);
    pl.down_cap_off.assign(T + 1, 0);
    pl.tile_prefix.assign(T + 1, 0);
    pl.topk_k.assign(T, 0);
    int64_t tiles = 0;
    for (int t = 0; t < T; ++t) {
        int64_t n = pl.seg_off[t + 1] - pl.seg_off[t];
        pl.word_off[t + 1] = pl.word_off[t] + (n + 31) / 32;
        tiles += (n + TILE - 1) / TILE;
        if (tiles > 0x7fffffff) return fail(msg, LIEC_ERR_UNSUPPORTED, "too many tiles");
        pl.tile_prefix[t + 1] = (int32_t)tiles;
        if (any_topk) {
            int64_t k = cfg->topk_k[t];
            pl.topk_k[t] = k;
            pl.k_off[t + 1] = pl.k_off[t] + k;
            int64_t cap = 2 * k + 2048;  // room for the entries sharing the threshold's first digit
            if (cap > n) cap = n;
            pl.cap_off[t + 1] = pl.cap_off[t] + cap;
            if (cap > pl.cap_max) pl.cap_max = cap;
            // The downlink has one row, and in a long segment (a flat vector, an embedding matrix) the
            // entries of v at or above the start of the threshold's first-digit bin run to several times k
            // (error feedback piles v up under the threshold): room for 8 k of them costs little there and
            // saves the dense second-digit pass over the segment in most iterations.
            int64_t down_cap = cap;
            if ((n + TILE - 1) / TILE >= LONG_SEG_TILES) down_cap = std::min<int64_t>(n, 8 * k + 2048);
            pl.down_cap_off[t + 1] = pl.down_cap_off[t] + down_cap;
        }
    }
    // a sparse message's values, tiled like the model (for their squared norms): segment t owns k_t entries
    pl.ktile_prefix.assign(T + 1, 0);
    if (any_topk) {
        int64_t ktiles = 0;
        for (int t = 0; t < T; ++t) {
            ktiles += (pl.topk_k[t] + TILE - 1) / TILE;
            pl.ktile_prefix[t + 1] = (int32_t)ktiles;   // (at most the model's own tile count)
        }
        pl.KTT = (int32_t)ktiles;
        pl.ktile_seg.resize(pl.KTT);
        for (int t = 0; t < T; ++t)
            for (int q = pl.ktile_prefix[t]; q < pl.ktile_prefix[t + 1]; ++q) pl.ktile_seg[q] = t;
    }
    pl.W = pl.word_off[T];
    pl.K = pl.k_off[T];
    pl.CAP = pl.cap_off[T];
    pl.down_CAP = pl.down_cap_off[T];
    pl.TT = (int32_t)tiles;
    pl.tile_seg.resize(pl.TT);
    for (int t = 0; t < T; ++t) {
        for (int q = pl.tile_prefix[t]; q < pl.tile_prefix[t + 1]; ++q) pl.tile_seg[q] = t;
        (pl.tile_prefix[t + 1] - pl.tile_prefix[t] == 1 ? pl.small_seg : pl.large_seg).push_back(t);
    }
    // the per-problem kernels take the largest segments first (their CTAs run longest)
    std::stable_sort(pl.large_seg.begin(), pl.large_seg.end(), [&](int32_t a, int32_t b) {
        return pl.seg_off[a + 1] - pl.seg_off[a] > pl.seg_off[b + 1] - pl.seg_off[b];
    });

    Carver c;
    pl.r_seg_off = c.take(sizeof(int64_t) * (T + 1));
    pl.r_word_off = c.take(sizeof(int64_t) * (T + 1));
    pl.r_k_off = c.take(sizeof(int64_t) * (T + 1));
    pl.r_cap_off = c.take(sizeof(int64_t) * (T + 1));
    pl.r_down_cap_off = c.take(sizeof(int64_t) * (T + 1));
    pl.r_tile_prefix = c.take(sizeof(int32_t) * (T + 1));
    pl.r_tile_seg = c.take(sizeof(int32_t) * pl.TT);
    pl.r_small_seg = c.take(sizeof(int32_t) * pl.small_seg.size());
    pl.r_large_seg = c.take(sizeof(int32_t) * pl.large_seg.size());
    pl.r_status = c.take(256);
    pl.r_tel_partials = c.take(sizeof(double) * (size_t)pl.N * pl.TT);
    pl.r_tel_e = c.take(sizeof(double) * (size_t)pl.TT);
    pl.r_tel_v = c.take(sizeof(double) * (size_t)pl.TT);
    pl.r_tel_g = c.take(sizeof(double) * (size_t)pl.N * pl.TT);
    pl.r_ktile_prefix = c.take(sizeof(int32_t) * (T + 1));
    pl.r_ktile_seg = c.take(sizeof(int32_t) * pl.KTT);
    pl.r_tel_kept = c.take(sizeof(double) * (size_t)pl.N * pl.KTT);
    const size_t N = pl.N;
    if (cfg->uplink == LIEC_COMP_SCALED_SIGN) {
        pl.r_up_words = c.take(sizeof(uint32_t) * N * pl.W);
        pl.r_up_scales = c.take(sizeof(float) * N * T);
        pl.r_up_partials = c.take(sizeof(double) * N * pl.TT);
    }
    if (cfg->downlink == LIEC_COMP_SCALED_SIGN) {
        // words and scales are adjacent: together they are the downlink message
        pl.r_down_words = c.take(sizeof(uint32_t) * pl.W + sizeof(float) * T);
        pl.r_down_words.bytes = sizeof(uint32_t) * pl.W;
        pl.r_down_scales.off = pl.r_down_words.off + pl.r_down_words.bytes;
        pl.r_down_scales.bytes = sizeof(float) * T;
        pl.r_down_partials = c.take(sizeof(double) * pl.TT);
    }
    if (cfg->downlink == LIEC_COMP_IDENTITY) pl.r_vbuf = c.take(sizeof(float) * pl.d);
    int max_seg_tiles = 0;
    for (int t = 0; t < T; ++t) max_seg_tiles = std::max(max_seg_tiles, pl.tile_prefix[t + 1] - pl.tile_prefix[t]);
    const size_t scan_parts = (size_t)(max_seg_tiles + SCAN_PART - 1) / SCAN_PART;
    auto topk_regions = [&](size_t rows, int64_t cap_total, Region &idx, Region &val, Region &hist, Region &hist2, Region &sel,
                            Region &cidx, Region &cval, Region &meta, Region &outbase, Region &parts) {
        parts = c.take(sizeof(uint32_t) * rows * T * scan_parts * 2);
        idx = c.take(sizeof(uint32_t) * rows * pl.K * 2);  // idx then val, adjacent
        idx.bytes = sizeof(uint32_t) * rows * pl.K;
        val.off = idx.off + idx.bytes;
        val.bytes = sizeof(float) * rows * pl.K;
        hist = c.take(sizeof(uint32_t) * rows * T * DIGIT1_BINS);
        hist2 = c.take(sizeof(uint32_t) * rows * T * DIGIT1_BINS);
        sel = c.take(sizeof(uint32_t) * rows * T * SEL_WORDS);
        cidx = c.take(sizeof(uint32_t) * rows * cap_total);
        cval = c.take(sizeof(float) * rows * cap_total);
        meta = c.take(sizeof(uint32_t) * rows * pl.TT * 4);
        outbase = c.take(sizeof(uint32_t) * rows * (pl.TT + 1));
    };
    // random-k needs the message and the per-tile offsets only
    auto randk_regions = [&](size_t rows, Region &idx, Region &val, Region &outbase) {
        idx = c.take(sizeof(uint32_t) * rows * pl.K * 2);
        idx.bytes = sizeof(uint32_t) * rows * pl.K;
        val.off = idx.off + idx.bytes;
        val.bytes = sizeof(float) * rows * pl.K;
        outbase = c.take(sizeof(uint32_t) * rows * (pl.TT + 1));
    };
    if (cfg->uplink == LIEC_COMP_RANDK) randk_regions(N, pl.r_up_idx, pl.r_up_val, pl.r_up_outbase);
    if (cfg->downlink == LIEC_COMP_RANDK) randk_regions(1, pl.r_down_idx, pl.r_down_val, pl.r_down_outbase);
    if (cfg->uplink == LIEC_COMP_RANDK || cfg->downlink == LIEC_COMP_RANDK)   // scratch of the seeded draw (liec_draw_subsets)
        topk_regions(N + 1, pl.CAP, pl.r_gen_sets, pl.r_gen_val, pl.r_gen_hist, pl.r_gen_hist2, pl.r_gen_sel, pl.r_gen_cand_idx,
                     pl.r_gen_cand_val, pl.r_gen_meta, pl.r_gen_outbase, pl.r_gen_scan_parts);
    if (cfg->uplink == LIEC_COMP_TOPK)
        topk_regions(N, pl.CAP, pl.r_up_idx, pl.r_up_val, pl.r_up_hist, pl.r_up_hist2, pl.r_up_sel, pl.r_up_cand_idx,
                     pl.r_up_cand_val, pl.r_up_tile_meta, pl.r_up_outbase, pl.r_up_scan_parts);
    if (cfg->downlink == LIEC_COMP_TOPK)
        topk_regions(1, pl.down_CAP, pl.r_down_idx, pl.r_down_val, pl.r_down_hist, pl.r_down_hist2, pl.r_down_sel,
                     pl.r_down_cand_idx, pl.r_down_cand_val, pl.r_down_tile_meta, pl.r_down_outbase, pl.r_down_scan_parts);
    pl.total = align_up(c.cursor, 256);
    return LIEC_OK;
}

}  // namespace

struct liec_ctx {
    Plan plan;
    Params p;
    liec_config cfg;
    char *ws = nullptr;
    int stage = 0;  // 0 idle, 1 after uplink, 2 after aggregate, 3 after downlink
    int64_t launches = 0;
    bool telemetry_valid = false;  // an iteration has completed with the telemetry switched on
    std::string err;
    // top-k: the single-tile segments are selected on a stream of the context's own, forked from
    // and joined to the caller's stream by events, so that they overlap the dense passes
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaEvent_t ev_tail_fork = nullptr, ev_tail_join = nullptr;   // the tail launch of the big problems
};

namespace {

template <typename Tp>
Tp *at(liec_ctx *c, const Region &r) {
    return r.bytes ? reinterpret_cast<Tp *>(c->ws + r.off) : nullptr;
}

liec_status cuda_fail(liec_ctx *c, cudaError_t e, const char *what) {
    c->err = std::string(what) + ": " + cudaGetErrorString(e);
    return LIEC_ERR_CUDA;
}

#define LIEC_LAUNCH(ctx, call)                                        \
    do {                                                              \
        cudaError_t e__ = (call);                                     \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call);    \
        ++(ctx)->launches;                                            \
    } while (0)

#define LIEC_CALL(ctx, call)                                          \
    do {                                                              \
        cudaError_t e__ = (call);                                     \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call);    \
    } while (0)

bool aligned16(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

void release_side(liec_ctx *c) {
    for (cudaEvent_t ev : {c->ev_fork, c->ev_join, c->ev_tail_fork, c->ev_tail_join})
        if (ev) cudaEventDestroy(ev);
    if (c->side) cudaStreamDestroy(c->side);
    c->ev_fork = c->ev_join = c->ev_tail_fork = c->ev_tail_join = nullptr;
    c->side = nullptr;
    c->p.tail_stream = c->p.tail_fork = c->p.tail_join = nullptr;
}

// Top-k side: the single-tile segments on the context's own stream (between a fork after what `s`
// holds so far and a join that the caller issues with join_side), the rest on `s`.
liec_status fork_small_segments(liec_ctx *c, bool uplink, cudaStream_t s) {
    if (!c->side || c->p.n_small == 0) return LIEC_OK;
    LIEC_CALL(c, cudaEventRecord(c->ev_fork, s));
    LIEC_CALL(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
    LIEC_CALL(c, launch_topk_small_segments(c->p, uplink, c->side, &c->launches));
    LIEC_CALL(c, cudaEventRecord(c->ev_join, c->side));
    return LIEC_OK;
}

liec_status join_side(liec_ctx *c, cudaStream_t s) {
    if (!c->side || c->p.n_small == 0) return LIEC_OK;
    LIEC_CALL(c, cudaStreamWaitEvent(s, c->ev_join, 0));
    return LIEC_OK;
}

}  // namespace

extern "C" {

size_t liec_workspace_bytes(const liec_config *cfg) {
    Plan pl;
    if (make_plan(cfg, pl, nullptr) != LIEC_OK) return 0;
    return pl.total;
}

static liec_status wire_bytes(const liec_config *cfg, bool shared_seed, int64_t *uplink_bytes, int64_t *downlink_bytes,
                              int64_t *full_precision_bytes) {
    Plan pl;
    std::string msg;
    liec_status st = make_plan(cfg, pl, &msg);
    if (st != LIEC_OK) {
        snprintf(g_no_ctx_error, sizeof(g_no_ctx_error), "%s", msg.c_str());
        return st;
    }
    auto message = [&](int32_t comp) -> int64_t {
        if (comp == LIEC_COMP_SCALED_SIGN) return 4 * (pl.W + (int64_t)pl.T);  // packed signs + one scale per segment
        if (comp == LIEC_COMP_RANDK && shared_seed) return 4 * pl.K;             // values only: the receiver redraws the subset
        if (comp_is_sparse(comp)) return 8 * pl.K;                               // (index, value) pairs
        return 4 * pl.d;                                                          // identity: the dense vector
    };
    if (uplink_bytes) *uplink_bytes = message(cfg->uplink);
    if (downlink_bytes) *downlink_bytes = message(cfg->downlink);
    if (full_precision_bytes) *full_precision_bytes = 4 * pl.d;
    return LIEC_OK;
}

liec_status liec_wire_bytes(const liec_config *cfg, int64_t *uplink_bytes, int64_t *downlink_bytes,
                            int64_t *full_precision_bytes) {
    return wire_bytes(cfg, false, uplink_bytes, downlink_bytes, full_precision_bytes);
}

liec_status liec_wire_bytes_seeded(const liec_config *cfg, int64_t *uplink_bytes, int64_t *downlink_bytes,
                                   int64_t *full_precision_bytes) {
    return wire_bytes(cfg, true, uplink_bytes, downlink_bytes, full_precision_bytes);
}

size_t liec_down_message_bytes(const liec_config *cfg) {
    Plan pl;
    if (make_plan(cfg, pl, nullptr) != LIEC_OK) return 0;
    if (cfg->downlink == LIEC_COMP_SCALED_SIGN) return sizeof(uint32_t) * pl.W + sizeof(float) * pl.T;
    if (comp_is_sparse(cfg->downlink)) return (sizeof(uint32_t) + sizeof(float)) * pl.K;
    return 0;
}

liec_status liec_init(const liec_config *cfg, float *params, float *error, void *workspace,
                      size_t workspace_bytes, liec_ctx **out) {
    std::string msg;
    auto bail = [&](liec_status st, const char *text) {
        snprintf(g_no_ctx_error, sizeof(g_no_ctx_error), "%s", text);
        return st;
    };
    if (!out) return bail(LIEC_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    liec_ctx *c = new (std::nothrow) liec_ctx();
    if (!c) return bail(LIEC_ERR_INVALID_ARG, "out of host memory");
    liec_status st = make_plan(cfg, c->plan, &msg);
    if (st != LIEC_OK) { delete c; return bail(st, msg.c_str()); }
    if (!params || !error || !workspace) { delete c; return bail(LIEC_ERR_INVALID_ARG, "params, error and workspace must be non-NULL"); }
    if (!aligned16(params) || !aligned16(error)) { delete c; return bail(LIEC_ERR_INVALID_ARG, "params and error must be 16-byte aligned"); }
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) { delete c; return bail(LIEC_ERR_INVALID_ARG, "workspace must be 256-byte aligned"); }
    if (workspace_bytes < c->plan.total) { delete c; return bail(LIEC_ERR_WORKSPACE, "workspace smaller than liec_workspace_bytes()"); }

    const Plan &pl = c->plan;
    c->cfg = *cfg;
    c->cfg.seg_offsets = nullptr;
    c->cfg.topk_k = nullptr;
    c->ws = static_cast<char *>(workspace);
    Params &p = c->p;
    memset(&p, 0, sizeof(p));
    p.N = pl.N; p.T = pl.T; p.TT = pl.TT; p.d = pl.d; p.W = pl.W; p.K = pl.K; p.CAP = pl.CAP; p.cap_max = pl.cap_max;
    p.up = cfg->uplink; p.down = cfg->downlink; p.gdt = cfg->grad_dtype;
    p.copy_wait_limit = COPY_WAIT_LIMIT_DEFAULT;
    p.copy_expect_extra = 0u;
    p.seg_off = at<int64_t>(c, pl.r_seg_off);
    p.word_off = at<int64_t>(c, pl.r_word_off);
    p.k_off = at<int64_t>(c, pl.r_k_off);
    p.cap_off = at<int64_t>(c, pl.r_cap_off);
    p.down_cap_off = at<int64_t>(c, pl.r_down_cap_off);
    p.down_CAP = pl.down_CAP;
    p.tile_prefix = at<int32_t>(c, pl.r_tile_prefix);
    p.tile_seg = at<int32_t>(c, pl.r_tile_seg);
    p.small_seg = at<int32_t>(c, pl.r_small_seg);
    p.large_seg = at<int32_t>(c, pl.r_large_seg);
    p.n_small = (int32_t)pl.small_seg.size();
    p.n_large = (int32_t)pl.large_seg.size();
    // the leading (largest) multi-tile segments whose candidate buffers are big: their tails get a launch of their own
    p.n_big = 0;
    p.cap_rest_max = 0;
    if (pl.K > 0) {
        auto cap_of = [&](int q) { return pl.cap_off[pl.large_seg[q] + 1] - pl.cap_off[pl.large_seg[q]]; };
        while (p.n_big < p.n_large && cap_of(p.n_big) >= TAIL_BIG_CAP) ++p.n_big;
        for (int q = p.n_big; q < p.n_large; ++q) p.cap_rest_max = std::max<int64_t>(p.cap_rest_max, cap_of(q));
    }
    p.n_long = 0;
    p.cap_long_max = 0;
    p.down_cap_long_max = 0;
    if (pl.K > 0) {
        auto tiles_of = [&](int q) { return pl.tile_prefix[pl.large_seg[q] + 1] - pl.tile_prefix[pl.large_seg[q]]; };
        while (p.n_long < p.n_large && tiles_of(p.n_long) >= LONG_SEG_TILES) {
            p.cap_long_max = std::max<int64_t>(p.cap_long_max, pl.cap_off[pl.large_seg[p.n_long] + 1] - pl.cap_off[pl.large_seg[p.n_long]]);
            p.down_cap_long_max = std::max<int64_t>(p.down_cap_long_max, pl.down_cap_off[pl.large_seg[p.n_long] + 1] - pl.down_cap_off[pl.large_seg[p.n_long]]);
            ++p.n_long;
        }
    }
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms = 0;
        p.num_sms = sms;
    }
    p.max_seg_tiles = 0;
    for (int t = 0; t < pl.T; ++t) p.max_seg_tiles = std::max(p.max_seg_tiles, pl.tile_prefix[t + 1] - pl.tile_prefix[t]);
    p.scan_parts = (p.max_seg_tiles + SCAN_PART - 1) / SCAN_PART;
    p.status = at<int32_t>(c, pl.r_status);
    p.X = params;
    p.e = error;
    p.up_words = at<uint32_t>(c, pl.r_up_words);
    p.up_scales = at<float>(c, pl.r_up_scales);
    p.up_partials = at<double>(c, pl.r_up_partials);
    p.down_words = at<uint32_t>(c, pl.r_down_words);
    p.down_scales = at<float>(c, pl.r_down_scales);
    p.down_partials = at<double>(c, pl.r_down_partials);
    p.vbuf = at<float>(c, pl.r_vbuf);
    p.tel_partials = at<double>(c, pl.r_tel_partials);
    p.telemetry = 0;
    p.tel_e = at<double>(c, pl.r_tel_e);
    p.tel_v = at<double>(c, pl.r_tel_v);
    p.tel_g = at<double>(c, pl.r_tel_g);
    p.tel_kept = at<double>(c, pl.r_tel_kept);
    p.KTT = pl.KTT;
    p.ktile_prefix = at<int32_t>(c, pl.r_ktile_prefix);
    p.ktile_seg = at<int32_t>(c, pl.r_ktile_seg);
    p.up_idx = at<uint32_t>(c, pl.r_up_idx);       p.up_val = at<float>(c, pl.r_up_val);
    p.down_idx = at<uint32_t>(c, pl.r_down_idx);   p.down_val = at<float>(c, pl.r_down_val);
    p.up_hist = at<uint32_t>(c, pl.r_up_hist);     p.down_hist = at<uint32_t>(c, pl.r_down_hist);
    p.up_hist2 = at<uint32_t>(c, pl.r_up_hist2);   p.down_hist2 = at<uint32_t>(c, pl.r_down_hist2);
    p.up_sel = at<uint32_t>(c, pl.r_up_sel);       p.down_sel = at<uint32_t>(c, pl.r_down_sel);
    p.up_cand_idx = at<uint32_t>(c, pl.r_up_cand_idx);   p.down_cand_idx = at<uint32_t>(c, pl.r_down_cand_idx);
    p.up_cand_val = at<float>(c, pl.r_up_cand_val);      p.down_cand_val = at<float>(c, pl.r_down_cand_val);
    p.up_tile_meta = at<uint32_t>(c, pl.r_up_tile_meta); p.down_tile_meta = at<uint32_t>(c, pl.r_down_tile_meta);
    p.up_outbase = at<uint32_t>(c, pl.r_up_outbase);     p.down_outbase = at<uint32_t>(c, pl.r_down_outbase);
    p.gen_sets = at<uint32_t>(c, pl.r_gen_sets);         p.gen_val = at<float>(c, pl.r_gen_val);
    p.gen_hist = at<uint32_t>(c, pl.r_gen_hist);         p.gen_hist2 = at<uint32_t>(c, pl.r_gen_hist2);
    p.gen_sel = at<uint32_t>(c, pl.r_gen_sel);           p.gen_meta = at<uint32_t>(c, pl.r_gen_meta);
    p.gen_cand_idx = at<uint32_t>(c, pl.r_gen_cand_idx); p.gen_cand_val = at<float>(c, pl.r_gen_cand_val);
    p.gen_outbase = at<uint32_t>(c, pl.r_gen_outbase);
    p.up_scan_parts = at<uint32_t>(c, pl.r_up_scan_parts); p.down_scan_parts = at<uint32_t>(c, pl.r_down_scan_parts);
    p.gen_scan_parts = at<uint32_t>(c, pl.r_gen_scan_parts);

    struct Up { const Region *r; const void *src; };
    const Up ups[] = {
        {&pl.r_seg_off, pl.seg_off.data()}, {&pl.r_word_off, pl.word_off.data()}, {&pl.r_k_off, pl.k_off.data()},
        {&pl.r_cap_off, pl.cap_off.data()}, {&pl.r_down_cap_off, pl.down_cap_off.data()}, {&pl.r_tile_prefix, pl.tile_prefix.data()},
        {&pl.r_tile_seg, pl.tile_seg.data()}, {&pl.r_small_seg, pl.small_seg.data()}, {&pl.r_large_seg, pl.large_seg.data()},
        {&pl.r_ktile_prefix, pl.ktile_prefix.data()}, {&pl.r_ktile_seg, pl.ktile_seg.data()},
    };
    for (const Up &u : ups) {
        if (!u.r->bytes) continue;
        cudaError_t e = cudaMemcpy(c->ws + u.r->off, u.src, u.r->bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            snprintf(g_no_ctx_error, sizeof(g_no_ctx_error), "cudaMemcpy of tables failed: %s", cudaGetErrorString(e));
            delete c;
            return LIEC_ERR_CUDA;
        }
    }
    // status word and every selection scratch region start at zero
    auto zero = [&](const Region &r) { return r.bytes ? cudaMemset(c->ws + r.off, 0, r.bytes) : cudaSuccess; };
    const Region *zs[] = {&pl.r_status, &pl.r_up_hist, &pl.r_down_hist, &pl.r_up_hist2, &pl.r_down_hist2,
                          &pl.r_up_sel, &pl.r_down_sel, &pl.r_up_tile_meta, &pl.r_down_tile_meta,
                          &pl.r_up_outbase, &pl.r_down_outbase,
                          &pl.r_gen_hist, &pl.r_gen_hist2, &pl.r_gen_sel, &pl.r_gen_meta, &pl.r_gen_outbase};
    for (const Region *r : zs) {
        cudaError_t e = zero(*r);
        if (e != cudaSuccess) {
            snprintf(g_no_ctx_error, sizeof(g_no_ctx_error), "cudaMemset of scratch failed: %s", cudaGetErrorString(e));
            delete c;
            return LIEC_ERR_CUDA;
        }
    }
    cudaError_t e = configure_topk_kernels();
    if (e == cudaSuccess) e = configure_average_kernels();
    if (e == cudaSuccess && ((c->plan.K > 0 && (!c->plan.small_seg.empty() || p.n_big > 0)) || p.down == COMP_SIGN)) {
        int prio_low = 0, prio_high = 0;   // the helper stream carries the longest-running CTAs of a stage: they go first
        e = cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&c->side, cudaStreamNonBlocking, prio_high);
        for (cudaEvent_t *ev : {&c->ev_fork, &c->ev_join, &c->ev_tail_fork, &c->ev_tail_join})
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
        if (e != cudaSuccess) release_side(c);
        else { p.tail_stream = c->side; p.tail_fork = c->ev_tail_fork; p.tail_join = c->ev_tail_join; }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        snprintf(g_no_ctx_error, sizeof(g_no_ctx_error), "kernel configuration / synchronize failed: %s", cudaGetErrorString(e));
        delete c;
        return LIEC_ERR_CUDA;
    }
    *out = c;
    return LIEC_OK;
}

static liec_status check_stage(liec_ctx *c, int want, const char *name) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    if (c->stage != want) {
        c->err = std::string(name) + " called out of order (stages: uplink, aggregate, downlink, update)";
        return LIEC_ERR_STATE;
    }
    return LIEC_OK;
}

liec_status liec_uplink_compress(liec_ctx *c, const void *grads, void *stream) {
    liec_status st = check_stage(c, 0, "liec_uplink_compress");
    if (st != LIEC_OK) return st;
    if (!grads || !aligned16(grads)) { c->err = "grads must be non-NULL and 16-byte aligned"; return LIEC_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    c->p.G = grads;
    if (c->p.up == COMP_SIGN) {
        LIEC_LAUNCH(c, launch_sign_uplink(c->p, s));
        LIEC_LAUNCH(c, launch_scale_finalize(c->p, true, s));
    } else if (c->p.up == COMP_TOPK) {
        if ((st = fork_small_segments(c, true, s)) != LIEC_OK) return st;
        LIEC_CALL(c, launch_topk_hist1(c->p, true, s, &c->launches));
        LIEC_CALL(c, launch_topk_select(c->p, true, s, &c->launches));
        if ((st = join_side(c, s)) != LIEC_OK) return st;
    } else if (c->p.up == COMP_RANDK) {
        if (!c->p.up_sets) { c->err = "random-k uplink: no subsets given (liec_set_subsets)"; return LIEC_ERR_STATE; }
        LIEC_CALL(c, launch_randk_compress(c->p, true, s, &c->launches));
    }
    c->stage = 1;
    return LIEC_OK;
}

liec_status liec_server_aggregate(liec_ctx *c, void *stream) {
    liec_status st = check_stage(c, 1, "liec_server_aggregate");
    if (st != LIEC_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (comp_is_sparse(c->p.up)) {
        LIEC_CALL(c, launch_server_topk(c->p, s, &c->launches));
    } else {
        LIEC_LAUNCH(c, launch_server_dense(c->p, s));
    }
    c->stage = 2;
    return LIEC_OK;
}

liec_status liec_downlink_compress(liec_ctx *c, void *stream) {
    liec_status st = check_stage(c, 2, "liec_downlink_compress");
    if (st != LIEC_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c->p.down == COMP_SIGN) {
        LIEC_LAUNCH(c, launch_scale_finalize(c->p, false, s));
        LIEC_LAUNCH(c, launch_sign_error(c->p, s));
    } else if (c->p.down == COMP_IDENTITY) {
        LIEC_LAUNCH(c, launch_identity_downlink(c->p, s));
    } else if (c->p.down == COMP_RANDK) {
        if (!c->p.down_set) { c->err = "random-k downlink: no subset given (liec_set_subsets)"; return LIEC_ERR_STATE; }
        LIEC_CALL(c, launch_randk_compress(c->p, false, s, &c->launches));
    } else {
        // the first-digit histogram of v is fused into the server pass after a sparse uplink
        if ((st = fork_small_segments(c, false, s)) != LIEC_OK) return st;
        if (!comp_is_sparse(c->p.up)) LIEC_CALL(c, launch_topk_hist1(c->p, false, s, &c->launches));
        LIEC_CALL(c, launch_topk_select(c->p, false, s, &c->launches));
        if ((st = join_side(c, s)) != LIEC_OK) return st;
    }
    c->stage = 3;
    return LIEC_OK;
}

liec_status liec_worker_update(liec_ctx *c, const void *grads, float lr, void *stream) {
    liec_status st = check_stage(c, 3, "liec_worker_update");
    if (st != LIEC_OK) return st;
    if (grads != c->p.G) { c->err = "liec_worker_update needs the gradient pointer given to liec_uplink_compress"; return LIEC_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    LIEC_LAUNCH(c, launch_worker_update(c->p, lr, s));
    c->stage = 0;
    c->telemetry_valid = c->p.telemetry != 0;
    return LIEC_OK;
}

liec_status liec_set_subsets(liec_ctx *c, const uint32_t *up_sets, const uint32_t *down_set) {
    liec_status st = check_stage(c, 0, "liec_set_subsets");
    if (st != LIEC_OK) return st;
    if ((reinterpret_cast<uintptr_t>(up_sets) | reinterpret_cast<uintptr_t>(down_set)) & 3u) {
        c->err = "subsets must be 4-byte aligned";
        return LIEC_ERR_INVALID_ARG;
    }
    c->p.up_sets = up_sets;
    c->p.down_set = down_set;
    return LIEC_OK;
}

liec_status liec_draw_subsets(liec_ctx *c, uint64_t seed, uint32_t epoch, void *stream) {
    liec_status st = check_stage(c, 0, "liec_draw_subsets");
    if (st != LIEC_OK) return st;
    if (c->p.up != COMP_RANDK && c->p.down != COMP_RANDK) {
        c->err = "liec_draw_subsets: no side uses random-k";
        return LIEC_ERR_INVALID_ARG;
    }
    const Params &p = c->p;
    TopkSide s;
    s.src = nullptr; s.row_stride = 0; s.R = p.N + 1;
    s.gen = ScoreStream{(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), epoch};
    s.idx = p.gen_sets; s.val = p.gen_val; s.hist = p.gen_hist; s.hist2 = p.gen_hist2; s.sel = p.gen_sel;
    s.cand_idx = p.gen_cand_idx; s.cand_val = p.gen_cand_val; s.meta = p.gen_meta; s.outbase = p.gen_outbase; s.scan_parts = p.gen_scan_parts;
    s.cap_off = p.cap_off; s.CAP = p.CAP; s.cap_long_max = p.cap_long_max;
    s.zero_out = nullptr;
    s.spec = 1;
    cudaStream_t main_stream = static_cast<cudaStream_t>(stream);
    const bool forked = c->side && p.n_small > 0;   // single-tile segments beside the dense pass, as in the top-k stages
    if (forked) {
        LIEC_CALL(c, cudaEventRecord(c->ev_fork, main_stream));
        LIEC_CALL(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        LIEC_CALL(c, launch_randk_draw_small(p, s, c->side, &c->launches));
        LIEC_CALL(c, cudaEventRecord(c->ev_join, c->side));
    } else {
        LIEC_CALL(c, launch_randk_draw_small(p, s, main_stream, &c->launches));
    }
    LIEC_CALL(c, launch_randk_draw(p, s, main_stream, &c->launches));
    if (forked) LIEC_CALL(c, cudaStreamWaitEvent(main_stream, c->ev_join, 0));
    c->p.up_sets = p.up == COMP_RANDK ? p.gen_sets : nullptr;
    c->p.down_set = p.down == COMP_RANDK ? p.gen_sets + (int64_t)p.N * p.K : nullptr;
    return LIEC_OK;
}

// Scaled-sign downlink inside liec_step: the message is complete once the scales are final; the
// error update e <- v -/+ s (which only the next iteration reads) and the worker update (which
// reads the message, not e) do not depend on one another, so the first runs on the helper stream
// beside the second.  Same kernels, same bytes as the two stage calls in sequence.
static liec_status sign_downlink_beside_update(liec_ctx *c, const void *grads, float lr, cudaStream_t s) {
    liec_status st = check_stage(c, 2, "liec_step");
    if (st != LIEC_OK) return st;
    LIEC_LAUNCH(c, launch_scale_finalize(c->p, false, s));
    LIEC_CALL(c, cudaEventRecord(c->ev_fork, s));
    LIEC_CALL(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
    LIEC_LAUNCH(c, launch_sign_error(c->p, c->side));
    LIEC_CALL(c, cudaEventRecord(c->ev_join, c->side));
    c->stage = 3;
    st = liec_worker_update(c, grads, lr, s);
    LIEC_CALL(c, cudaStreamWaitEvent(s, c->ev_join, 0));   // (also after a refused update: nothing stays forked)
    return st;
}

liec_status liec_step(liec_ctx *c, const void *grads, float lr, void *stream) {
    liec_status st = liec_uplink_compress(c, grads, stream);
    if (st != LIEC_OK) return st;  // nothing was enqueued: the context is where it was
    if ((st = liec_server_aggregate(c, stream)) == LIEC_OK) {
        if (c->p.down == COMP_SIGN && c->side) {
            st = sign_downlink_beside_update(c, grads, lr, static_cast<cudaStream_t>(stream));
        } else if ((st = liec_downlink_compress(c, stream)) == LIEC_OK) {
            st = liec_worker_update(c, grads, lr, stream);
        }
    }
    if (st != LIEC_OK) c->stage = 0;  // a half-done iteration: back to idle, state unspecified (see liec_abort_step)
    return st;
}

liec_status liec_abort_step(liec_ctx *c) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    c->stage = 0;
    return LIEC_OK;
}

liec_status liec_set_copy_wait(liec_ctx *c, uint32_t poll_limit, uint32_t expect_extra_bytes) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    if (expect_extra_bytes & 15u) { c->err = "expect_extra_bytes must be a multiple of 16"; return LIEC_ERR_INVALID_ARG; }
    if (expect_extra_bytes > 1024u) { c->err = "expect_extra_bytes must be at most 1024"; return LIEC_ERR_INVALID_ARG; }
    c->p.copy_wait_limit = poll_limit ? poll_limit : COPY_WAIT_LIMIT_DEFAULT;
    c->p.copy_expect_extra = expect_extra_bytes;
    return LIEC_OK;
}

liec_status liec_average_step(liec_ctx *c, const void *grads, float lr, void *stream) {
    liec_status st = check_stage(c, 0, "liec_average_step");
    if (st != LIEC_OK) return st;
    if (!grads || !aligned16(grads)) { c->err = "grads must be non-NULL and 16-byte aligned"; return LIEC_ERR_INVALID_ARG; }
    c->p.G = grads;
    LIEC_LAUNCH(c, launch_average_step(c->p, lr, static_cast<cudaStream_t>(stream)));
    return LIEC_OK;
}

liec_status liec_mean_params(liec_ctx *c, float *out, void *stream) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    if (!out) { c->err = "out must be non-NULL"; return LIEC_ERR_INVALID_ARG; }
    LIEC_LAUNCH(c, launch_mean_params(c->p, out, static_cast<cudaStream_t>(stream)));
    return LIEC_OK;
}

liec_status liec_sumsq(liec_ctx *c, int32_t which, const void *grads, double *out, void *stream) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    if (!out) { c->err = "out must be non-NULL"; return LIEC_ERR_INVALID_ARG; }
    if (which < 0 || which > 2) { c->err = "which must be LIEC_SUMSQ_ERROR, _GRADS or _PARAMS"; return LIEC_ERR_INVALID_ARG; }
    if (which == 1 && (!grads || !aligned16(grads))) { c->err = "grads must be non-NULL and 16-byte aligned"; return LIEC_ERR_INVALID_ARG; }
    const void *src = which == 0 ? (const void *)c->p.e : which == 1 ? grads : (const void *)c->p.X;
    const int rows = which == 0 ? 1 : c->p.N;
    const bool bf16 = which == 1 && c->p.gdt == DT_BF16;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    LIEC_LAUNCH(c, launch_sumsq(c->p, src, which == 0 ? 0 : c->p.d, rows, bf16, s));
    LIEC_LAUNCH(c, launch_sum_finalize(c->p, c->p.tel_partials, rows, out, s));
    return LIEC_OK;
}

liec_status liec_set_telemetry(liec_ctx *c, int32_t on) {
    liec_status st = check_stage(c, 0, "liec_set_telemetry");
    if (st != LIEC_OK) return st;
    c->p.telemetry = on ? 1 : 0;
    c->telemetry_valid = false;
    return LIEC_OK;
}

liec_status liec_get_telemetry(liec_ctx *c, double *e_sumsq, double *v_sumsq, double *g_sumsq,
                               double *up_kept_sumsq, double *down_kept_sumsq, void *stream) {
    liec_status st = check_stage(c, 0, "liec_get_telemetry");
    if (st != LIEC_OK) return st;
    if (!c->telemetry_valid) {
        c->err = "liec_get_telemetry: no iteration has run since liec_set_telemetry switched the telemetry on";
        return LIEC_ERR_STATE;
    }
    if ((up_kept_sumsq && !comp_is_sparse(c->p.up)) || (down_kept_sumsq && !comp_is_sparse(c->p.down))) {
        c->err = "liec_get_telemetry: kept-value norms exist only for a top-k or random-k side";
        return LIEC_ERR_INVALID_ARG;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const Params &p = c->p;
    if (e_sumsq) LIEC_LAUNCH(c, launch_sum_finalize(p, p.tel_e, 1, e_sumsq, s));
    if (v_sumsq) LIEC_LAUNCH(c, launch_sum_finalize(p, p.tel_v, 1, v_sumsq, s));
    if (g_sumsq) LIEC_LAUNCH(c, launch_sum_finalize(p, p.tel_g, p.N, g_sumsq, s));
    if (up_kept_sumsq || down_kept_sumsq) {
        // the message values laid out like a model of K entries with segments of k_t: the same two
        // kernels as liec_sumsq, driven by the tables of that layout
        Params pk = p;
        pk.seg_off = p.k_off;
        pk.tile_prefix = p.ktile_prefix;
        pk.tile_seg = p.ktile_seg;
        pk.TT = p.KTT;
        pk.tel_partials = p.tel_kept;
        if (up_kept_sumsq) {
            LIEC_LAUNCH(c, launch_sumsq(pk, p.up_val, p.K, p.N, false, s));
            LIEC_LAUNCH(c, launch_sum_finalize(pk, pk.tel_partials, p.N, up_kept_sumsq, s));
        }
        if (down_kept_sumsq) {
            LIEC_LAUNCH(c, launch_sumsq(pk, p.down_val, 0, 1, false, s));
            LIEC_LAUNCH(c, launch_sum_finalize(pk, pk.tel_partials, 1, down_kept_sumsq, s));
        }
    }
    return LIEC_OK;
}

liec_status liec_step_host(liec_ctx *c, const void *grads_host, void *grads_dev, float lr, void *down_msg_host,
                           void *stream) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    if (!grads_host || !grads_dev) { c->err = "grads_host and grads_dev must be non-NULL"; return LIEC_ERR_INVALID_ARG; }
    // before anything is enqueued: a copy into grads_dev in the middle of an iteration would overwrite
    // the gradients that the pending worker update still has to read
    liec_status st0 = check_stage(c, 0, "liec_step_host");
    if (st0 != LIEC_OK) return st0;
    if (!aligned16(grads_dev)) { c->err = "grads_dev must be 16-byte aligned"; return LIEC_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esz = c->p.gdt == DT_BF16 ? 2 : 4;
    const size_t row_bytes = esz * (size_t)c->p.d;
    for (int i = 0; i < c->p.N; ++i) {
        cudaError_t e = cudaMemcpyAsync(static_cast<char *>(grads_dev) + i * row_bytes,
                                        static_cast<const char *>(grads_host) + i * row_bytes, row_bytes,
                                        cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(grads)");
    }
    liec_status st = liec_step(c, grads_dev, lr, stream);
    if (st != LIEC_OK) return st;
    if (down_msg_host) {
        const void *src = nullptr;
        size_t bytes = 0;
        if (c->p.down == COMP_SIGN) { src = c->p.down_words; bytes = sizeof(uint32_t) * c->p.W + sizeof(float) * c->p.T; }
        else if (comp_is_sparse(c->p.down)) { src = c->p.down_idx; bytes = 2 * sizeof(uint32_t) * c->p.K; }
        if (bytes) {
            cudaError_t e = cudaMemcpyAsync(down_msg_host, src, bytes, cudaMemcpyDeviceToHost, s);
            if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(down message)");
        }
    }
    return LIEC_OK;
}

liec_status liec_get_messages(const liec_ctx *c, liec_messages *out) {
    if (!c || !out) return LIEC_ERR_INVALID_ARG;
    out->up_words = c->p.up_words;
    out->up_scales = c->p.up_scales;
    out->up_idx = c->p.up_idx;
    out->up_val = c->p.up_val;
    out->down_words = c->p.down_words;
    out->down_scales = c->p.down_scales;
    out->down_idx = c->p.down_idx;
    out->down_val = c->p.down_val;
    out->v = c->p.e;
    out->num_words = c->p.W;
    out->num_topk = c->p.K;
    return LIEC_OK;
}

liec_status liec_device_status(liec_ctx *c, void *stream, int32_t *out) {
    if (!c || !out) return LIEC_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(out, c->p.status, sizeof(int32_t), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(status)");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamSynchronize");
    if (*out != 0) { c->err = "a kernel recorded a failed internal check"; return LIEC_ERR_DEVICE_CHECK; }
    return LIEC_OK;
}

liec_status liec_topk_route_counts(liec_ctx *c, void *stream, int32_t uplink, int64_t *out, uint8_t *per_problem) {
    if (!c || !out) return LIEC_ERR_INVALID_ARG;
    const uint32_t *sel = uplink ? c->p.up_sel : c->p.down_sel;
    const int64_t problems = (int64_t)(uplink ? c->p.N : 1) * c->p.T;
    out[0] = out[1] = out[2] = out[3] = out[4] = 0;
    if (!sel) { c->err = "this side does not use top-k"; return LIEC_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<uint32_t> host((size_t)problems * SEL_WORDS);
    cudaError_t e = cudaMemcpyAsync(host.data(), sel, host.size() * sizeof(uint32_t), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(selection state)");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamSynchronize");
    out[0] = problems;
    for (int64_t q = 0; q < problems; ++q) {
        const uint32_t *w = host.data() + q * SEL_WORDS;
        const uint32_t route = w[SEL_ROUTE];
        out[1] += (route & ROUTE_SINGLE) != 0; out[2] += (route & ROUTE_REFINED) != 0;
        out[3] += (route & ROUTE_SLOW) != 0;   out[4] += (route & ROUTE_DIRECT) != 0;
        if (per_problem) per_problem[q] = (uint8_t)route;
    }
    return LIEC_OK;
}

liec_status liec_clear_status(liec_ctx *c, void *stream) {
    if (!c) return LIEC_ERR_INVALID_ARG;
    cudaError_t e = cudaMemsetAsync(c->p.status, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemsetAsync(status)");
    return LIEC_OK;
}

int64_t liec_launch_count(const liec_ctx *c) { return c ? c->launches : 0; }

const char *liec_last_error(const liec_ctx *c) { return c ? c->err.c_str() : g_no_ctx_error; }

void liec_destroy(liec_ctx *c) {
    if (!c) return;
    release_side(c);
    delete c;
}

}  // extern "C"
