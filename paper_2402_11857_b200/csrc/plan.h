// Host-side plan (workspace layout, tile tables) and the parameter block handed to kernels.
//
// Work decomposition: every segment t is cut into tiles of TILE consecutive elements
// counted from the segment's own start, so that a tile is always an aligned subtree of
// the segment's balanced summation tree and owns whole 32-bit sign words.
#pragma once
#include <cstddef>
#include <cstdint>

namespace liec {

constexpr int TILE = 8192;             // elements per tile
constexpr int TILE_WORDS = TILE / 32;  // sign words per tile
constexpr int THREADS = 256;           // threads per CTA in the tile kernels (8 warps x 1024 elements)

constexpr int COMP_IDENTITY = 0, COMP_SIGN = 1, COMP_TOPK = 2, COMP_RANDK = 3;
// top-k and random-k share the (index, value) message layout and everything that consumes it
constexpr bool comp_is_sparse(int c) { return c == COMP_TOPK || c == COMP_RANDK; }
constexpr int DT_F32 = 0, DT_BF16 = 1;

// top-k selection constants
constexpr int DIGIT1_BITS = 12;                 // first radix digit: key bits 30..19
constexpr int DIGIT1_BINS = 1 << DIGIT1_BITS;
constexpr int DIGIT1_SHIFT = 31 - DIGIT1_BITS;  // 19

struct Params {
    int32_t N, T, TT;      // workers, segments, tiles per row
    int64_t d, W, K;       // dimension, words per row, top-k entries per row
    int32_t up, down, gdt;

    // tables (device, in the workspace)
    const int64_t *seg_off;      // [T+1]
    const int64_t *word_off;     // [T+1]
    const int64_t *k_off;        // [T+1] (top-k only)
    const int64_t *cap_off;      // [T+1] candidate capacity prefix (top-k only)
    const int64_t *down_cap_off; // [T+1] the same for the downlink (its long segments get more room: see make_plan)
    const int32_t *tile_prefix;  // [T+1] tiles before segment t
    const int32_t *tile_seg;     // [TT] segment of every tile
    const int32_t *small_seg;    // [n_small] segments of one tile (top-k: selected directly by one CTA)
    const int32_t *large_seg;    // [n_large] segments of several tiles
    int32_t n_small, n_large;
    int32_t n_big;               // leading entries of large_seg whose candidate capacity is TAIL_BIG_CAP or more
    int64_t cap_rest_max;        // largest candidate capacity among the other entries of large_seg
    int32_t n_long;              // leading entries of large_seg with LONG_SEG_TILES tiles or more
    int64_t cap_long_max;        // largest candidate capacity among them
    int64_t down_CAP, down_cap_long_max;   // the downlink's total and largest long-segment capacity
    // host side only: the context's helper stream and the events that fork / join the tail launch of
    // the big problems (cudaStream_t / cudaEvent_t; NULL = everything on the caller's stream)
    void *tail_stream, *tail_fork, *tail_join;
    int32_t num_sms;             // SMs of the device the context was created on
    int32_t max_seg_tiles;       // tiles of the longest segment

    // state
    float *X;         // [N][d]
    float *e;         // [d]
    const void *G;    // [N][d] current gradients

    // sign messages
    uint32_t *up_words;    // [N][W]
    float *up_scales;      // [N][T]
    double *up_partials;   // [N][TT]
    uint32_t *down_words;  // [W]
    float *down_scales;    // [T]
    double *down_partials; // [TT]
    double *tel_partials;  // [N][TT] squared norms on demand (liec_sumsq)

    // telemetry fused into the iteration's own passes (switched by liec_set_telemetry): per-tile
    // binary64 partial sums of squares, written by the kernels that hold the values anyway
    int32_t telemetry;     // 0 = off: the kernels without any of it
    double *tel_e;         // [TT]    ||e_t||^2, the error as the server pass reads it
    double *tel_v;         // [TT]    ||v_t||^2, as the server pass writes it
    double *tel_g;         // [N][TT] ||g^i_t||^2, from the worker update
    // the values of a sparse message are tiled like the model: segment t owns k_t entries
    int32_t KTT;                  // tiles of one row of a sparse message
    const int32_t *ktile_prefix;  // [T+1]
    const int32_t *ktile_seg;     // [KTT]
    double *tel_kept;             // [N][KTT] scratch for the squared norms of message values

    // top-k messages and scratch (row count R = N for uplink, 1 for downlink)
    const uint32_t *up_sets, *down_set;  // random-k: the caller's subsets [N][K] / [K]
    uint32_t *up_idx;  float *up_val;    // [N][K]
    uint32_t *down_idx; float *down_val; // [K]
    uint32_t *up_hist, *down_hist;       // [R][T][DIGIT1_BINS]
    uint32_t *up_hist2, *down_hist2;     // [R][T][DIGIT1_BINS] second / third digit
    uint32_t *up_sel, *down_sel;         // [R][T][SEL_WORDS] per-problem selection state
    uint32_t *up_cand_idx, *down_cand_idx;   // [R][CAP] candidate entries
    float *up_cand_val, *down_cand_val;      // [R][CAP]
    uint32_t *up_tile_meta, *down_tile_meta; // [R][TT][4] pos, cnt, n_greater, n_ties
    uint32_t *up_outbase, *down_outbase;     // [R][TT+1] first output slot of each tile
    uint32_t *up_scan_parts, *down_scan_parts, *gen_scan_parts;   // [R][T][scan_parts][2]: sums of a segment's per-tile counts over runs of SCAN_PART tiles (wide form)
    int32_t scan_parts;                      // runs of SCAN_PART tiles in the longest segment
    int64_t CAP;                              // candidate capacity per row
    int64_t cap_max;                          // largest candidate capacity of one segment

    // seeded random-k draw (rows 0..N-1: the workers' subsets, row N: the server's): the subset lists
    // it produces and the scratch of the selection that produces them
    uint32_t *gen_sets;                       // [N+1][K]
    float *gen_val;                           // [N+1][K] scores of the kept elements (scratch)
    uint32_t *gen_hist, *gen_hist2, *gen_sel; // [N+1][T][...]
    uint32_t *gen_cand_idx; float *gen_cand_val;  // [N+1][CAP]
    uint32_t *gen_meta, *gen_outbase;         // [N+1][TT][4], [N+1][TT+1]

    float *vbuf;      // [d] identity downlink copy of v
    int32_t *status;  // device status word

    // bounded waits on bulk copies into shared memory: polls before a copy is declared lost, and
    // bytes added to what its barrier is told to expect (0 in operation; a diagnostic setting
    // makes the barrier never complete although the copy lands, which exercises the timeout path)
    uint32_t copy_wait_limit, copy_expect_extra;
};
constexpr uint32_t COPY_WAIT_LIMIT_DEFAULT = 1u << 20;
constexpr int SCAN_PART = THREADS * 16;   // tiles whose output offsets one CTA of the wide form's scan computes
constexpr int LONG_SEG_TILES = 1024;   // from here on a segment's candidate passes walk its candidate region as a whole, not tile block by tile block

// per-problem selection state words
constexpr int SEL_WORDS = 20;
constexpr int SEL_PREFIX = 0;     // key prefix fixed so far (aligned to its bit position)
constexpr int SEL_REMAIN = 1;     // rank still to find inside the prefix bin (1-based)
constexpr int SEL_CAND_COUNT = 2; // atomic cursor: candidates appended so far
constexpr int SEL_THRESH = 3;     // final threshold key T
constexpr int SEL_TIES = 4;       // number of entries equal to T to accept, lowest index first
constexpr int SEL_CUT = 5;        // flat index of the last accepted tie
constexpr int SEL_FLAGS = 6;      // bit0: slow path (one CTA, dense passes); bit1: refined (24-bit prefix found by a dense second-digit pass)
                                  // (segments of a single tile never enter this machinery: one CTA selects them directly)
constexpr int SEL_NCAND = 7;      // exact number of candidates (entries at or above the prefix)
constexpr int SEL_ABOVE = 8;      // entries whose first digit is strictly above the threshold's
constexpr int SEL_LO1 = 9;        // lowest / highest non-empty bin of the first-digit histogram (so that the
constexpr int SEL_HI1 = 10;       // pick reads and clears only that range); reset to ~0 / 0 after use
constexpr int SEL_LO2 = 11;       // same for the second-digit histogram
constexpr int SEL_HI2 = 12;
constexpr int SEL_GUESS = 13;      // uplink: lower bound (31-bit key) tried first in the next step; 0 = none
constexpr int SEL_MODE = 14;       // uplink, this step: 1 = candidates collected with the guess, 0 = regular two-pass path
constexpr int SEL_ROUTE = 16;      // how the last iteration's selection was done (ROUTE_* bits; diagnostics)
constexpr int SEL_MARGIN = 17;     // uplink: first-digit bins between the next guess and the threshold's bin (0 = not yet chosen)
constexpr int ROUTE_SINGLE = 1, ROUTE_REFINED = 2, ROUTE_SLOW = 4, ROUTE_DIRECT = 8;
constexpr int SEL_SPEC_FAIL = 15;  // uplink, this step: the guess let too many candidates through (written by the
                                   // filter, read only by later kernels, which then send the problem down the regular path)

// words of the status block (int32 each)
constexpr int STATUS_WORD = 0;        // failed internal checks
constexpr unsigned STATUS_BAD_SUBSET = 16;   // bit of the status word: a random-k subset entry outside its segment or out of order
constexpr unsigned STATUS_COPY_TIMEOUT = 8;  // bit of the status word: a TMA bulk copy did not land within the wait limit
constexpr int STATUS_ANY_REGULAR = 12; // uplink: some problem takes the regular two-pass path this step
constexpr int STATUS_ANY_REFINE = 8;  // +0 uplink, +1 downlink: some problem needs the dense second-digit pass
constexpr int STATUS_ANY_DENSE = 16;  // +0 uplink, +1 downlink: some problem has no candidates and is finished in the dense source (wide form)

}  // namespace liec
