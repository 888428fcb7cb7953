/*
 * CPU oracle for one compressed iteration of LIEC-SGD (Algorithm 1, the branch
 * taken when (t+1) mod floor(1/delta) != 0).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * step computes.  Tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it; the product library never does, and the two share no code,
 * headers, tables or helpers.
 *
 * What is computed (per iteration, N workers, d parameters, T contiguous
 * segments with offsets off[0..T], n_t = off[t+1]-off[t]):
 *
 *   uplink   p^i = C(g^i)                      Algorithm 1, worker compress step
 *   server   v   = e + (1/N) sum_i p^i         Algorithm 1, server compensate step
 *   downlink p   = C(v)                        Algorithm 1, server compress step
 *   error    e'  = v - p                       Algorithm 1, global error update
 *   update   x^i = x^i - eta (p - p^i + g^i)   Algorithm 1, local model update
 *
 * with C one of
 *   scaled sign, per segment:  C(x)_j = (||x_t||_1 / n_t) sign(x_j)   Def. 4 / Def. 5
 *   top-k, per segment:        keep the k_t entries of largest |x_j|   Def. 2
 *   random-k, per segment:     keep the entries of a given k_t-subset  Def. 3
 *   identity:                  C(x) = x
 *
 * Readings fixed where the paper is silent (every one is arithmetic that the
 * CUDA library has to reproduce, so they are spelled out):
 *   - All state arithmetic is IEEE binary32, round to nearest even, one rounding
 *     per written operation, no fused multiply-add (build with -ffp-contract=off).
 *   - sign(x) is binary: negative iff x < 0; +0, -0 decode to +scale.
 *   - ||x_t||_1 is summed in binary64 over a balanced binary tree: leaves are
 *     |x_j| widened to double for j < n_t and +0 up to the next power of two L;
 *     node(lo,len) = node(lo,len/2) + node(lo+len/2,len/2).  The scale is that
 *     sum divided by (double)n_t, then rounded once to binary32.
 *   - top-k compares magnitudes through the binary32 bit pattern with the sign
 *     bit cleared; among equal magnitudes the lower index wins, so the selected
 *     set is unique.  The message lists (index, value) ascending by index.
 *   - random-k: the k_t-subset of every segment (one per worker for the uplink, one for the
 *     downlink) is an input of the iteration, listed as flat indices ascending inside the
 *     segment (Def. 3 wants it uniform over the k_t-subsets).  The message has the top-k layout.
 *     liec_oracle_draw_subsets below is the seeded draw of such subsets: every element gets a
 *     pseudo-random score from a counter-based generator and the k_t highest scores of a segment
 *     are its subset (equal scores: lower index first).
 *   - The server sums messages in worker order in binary32 starting from +0,
 *     divides by (float)N, then adds e.
 *   - The update is evaluated left to right as printed: ((p - p^i) + g), times
 *     eta, subtracted from x.
 *   - Sign message layout: segment t owns ceil(n_t/32) 32-bit words; bit b of
 *     word w is set iff element off[t]+32w+b is negative; padding bits are 0.
 *
 * The model-averaging iteration of Algorithm 1 (taken when (t+1) mod floor(1/delta) == 0; the
 * experiments use a fixed period of 32 or 100) is liec_oracle_average_step below: gradients and
 * models travel uncompressed, p = v, the global error becomes 0 and every worker restarts from the
 * averaged model.
 *
 * Parity pins (tests/test_oracle_*.py): hand-worked iterations, exact rational
 * means, brute-force bit packing and sorting, the contraction identities of
 * Def. 1, p + e' = v, Lemma 3, identity compressor with N=1 reducing to SGD.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_IDENTITY = 0, ORACLE_SIGN = 1, ORACLE_TOPK = 2, ORACLE_RANDK = 3 };

static uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }

/* bf16 -> binary32 is exact: the 16 stored bits are the top half of the word. */
void liec_oracle_widen_bf16(const uint16_t *in, float *out, int64_t n)
{
    for (int64_t j = 0; j < n; ++j) {
        uint32_t u = (uint32_t)in[j] << 16;
        memcpy(&out[j], &u, 4);
    }
}

/* ---- scaled sign (Def. 4, Def. 5) ------------------------------------------------- */

static double tree_node(const float *x, int64_t n, int64_t lo, int64_t len)
{
    if (len == 1) {
        if (lo >= n) return 0.0;
        float a = x[lo];
        if (a < 0.0f) a = -a;
        if (a == 0.0f) a = 0.0f;        /* |-0| = +0 */
        return (double)a;
    }
    double left = tree_node(x, n, lo, len / 2);
    double right = tree_node(x, n, lo + len / 2, len / 2);
    return left + right;
}

/* ||x||_1 over the balanced tree described in the header. */
double liec_oracle_tree_abs_sum(const float *x, int64_t n)
{
    int64_t L = 1;
    while (L < n) L *= 2;
    return tree_node(x, n, 0, L);
}

/* ||x||_1 / n as a binary32 number (Def. 4). */
float liec_oracle_scale(const float *x, int64_t n)
{
    double S = liec_oracle_tree_abs_sum(x, n);
    double mean = S / (double)n;
    return (float)mean;
}

/* ---- telemetry: squared norms ------------------------------------------------------- */

static double tree_sq_node(const float *x, int64_t n, int64_t lo, int64_t len)
{
    if (len == 1) {
        if (lo >= n) return 0.0;
        double a = (double)x[lo];
        return a * a;                  /* exact: 24-bit significands */
    }
    double left = tree_sq_node(x, n, lo, len / 2);
    double right = tree_sq_node(x, n, lo + len / 2, len / 2);
    return left + right;
}

/* ||x||_2^2 in binary64 over the same balanced tree as the L1 norm.  With it the quantities the
 * paper reports follow: the error norm ||e_t|| (its figure of error norms) and the measured
 * contraction delta = 1 - ||x - C(x)||^2 / ||x||^2 of Def. 1 (its table of measured delta). */
double liec_oracle_tree_sumsq(const float *x, int64_t n)
{
    int64_t L = 1;
    while (L < n) L *= 2;
    return tree_sq_node(x, n, 0, L);
}

static int64_t words_of(int64_t n) { return (n + 31) / 32; }

/* Segment-wise scaled sign of x[0..off[T]).  words: sum_t ceil(n_t/32) entries,
 * scales: T entries, dec: dense decoded C(x) (may be NULL). */
void liec_oracle_sign(const float *x, int32_t T, const int64_t *off,
                      uint32_t *words, float *scales, float *dec)
{
    int64_t woff = 0;
    for (int32_t t = 0; t < T; ++t) {
        const float *xs = x + off[t];
        int64_t n = off[t + 1] - off[t];
        float s = liec_oracle_scale(xs, n);
        scales[t] = s;
        for (int64_t w = 0; w < words_of(n); ++w) words[woff + w] = 0u;
        for (int64_t j = 0; j < n; ++j) {
            int neg = xs[j] < 0.0f;
            if (neg) words[woff + j / 32] |= (uint32_t)1 << (j % 32);
            if (dec) dec[off[t] + j] = neg ? -s : s;
        }
        woff += words_of(n);
    }
}

/* ---- top-k (Def. 2) ---------------------------------------------------------------- */

typedef struct { uint32_t key; uint32_t pos; } keypos;

static int by_magnitude_then_index(const void *a, const void *b)
{
    const keypos *p = (const keypos *)a, *q = (const keypos *)b;
    if (p->key != q->key) return p->key > q->key ? -1 : 1;   /* larger |x| first */
    if (p->pos != q->pos) return p->pos < q->pos ? -1 : 1;   /* lower index first */
    return 0;
}

/* Segment-wise top-k_t of x.  idx/val: sum_t k_t entries, flat indices ascending
 * inside each segment; dec: dense decoded C(x) (may be NULL).  Returns 0, or -1
 * when memory runs out. */
int liec_oracle_topk(const float *x, int32_t T, const int64_t *off, const int64_t *k,
                     uint32_t *idx, float *val, float *dec)
{
    int64_t koff = 0;
    for (int32_t t = 0; t < T; ++t) {
        const float *xs = x + off[t];
        int64_t n = off[t + 1] - off[t];
        keypos *order = (keypos *)malloc((size_t)n * sizeof(keypos));
        unsigned char *chosen = (unsigned char *)calloc((size_t)n, 1);
        if (!order || !chosen) { free(order); free(chosen); return -1; }
        for (int64_t j = 0; j < n; ++j) {
            order[j].key = f32_bits(xs[j]) & 0x7fffffffu;
            order[j].pos = (uint32_t)j;
        }
        qsort(order, (size_t)n, sizeof(keypos), by_magnitude_then_index);
        for (int64_t r = 0; r < k[t]; ++r) chosen[order[r].pos] = 1;
        int64_t out = koff;
        for (int64_t j = 0; j < n; ++j) {
            if (chosen[j]) {
                idx[out] = (uint32_t)(off[t] + j);
                val[out] = xs[j];
                ++out;
            }
            if (dec) dec[off[t] + j] = chosen[j] ? xs[j] : 0.0f;
        }
        koff += k[t];
        free(order);
        free(chosen);
    }
    return 0;
}

/* Segment-wise random-k (Def. 3) with the subset given: set lists, segment after segment, the
 * k_t flat indices kept in segment t, ascending.  idx/val/dec as for top-k.  Returns 0, or -3
 * when the set leaves its segment or is not strictly ascending. */
int liec_oracle_randk(const float *x, int32_t T, const int64_t *off, const int64_t *k,
                      const uint32_t *set, uint32_t *idx, float *val, float *dec)
{
    int64_t q = 0;
    for (int32_t t = 0; t < T; ++t) {
        if (dec) for (int64_t j = off[t]; j < off[t + 1]; ++j) dec[j] = 0.0f;
        for (int64_t r = 0; r < k[t]; ++r, ++q) {
            int64_t j = (int64_t)set[q];
            if (j < off[t] || j >= off[t + 1]) return -3;
            if (r > 0 && set[q - 1] >= set[q]) return -3;
            idx[q] = set[q];
            val[q] = x[j];
            if (dec) dec[j] = x[j];
        }
    }
    return 0;
}

/* ---- one iteration ----------------------------------------------------------------- */

static int compress(int32_t kind, const float *x, int64_t d, int32_t T, const int64_t *off,
                    const int64_t *k, const uint32_t *set, uint32_t *words, float *scales,
                    uint32_t *idx, float *val, float *dec)
{
    if (kind == ORACLE_SIGN) { liec_oracle_sign(x, T, off, words, scales, dec); return 0; }
    if (kind == ORACLE_TOPK) return liec_oracle_topk(x, T, off, k, idx, val, dec);
    if (kind == ORACLE_RANDK) return set ? liec_oracle_randk(x, T, off, k, set, idx, val, dec) : -3;
    if (kind == ORACLE_IDENTITY) { memcpy(dec, x, (size_t)d * sizeof(float)); return 0; }
    return -2;
}

/*
 * One compressed LIEC-SGD iteration.
 *   G [N][d] gradients already widened to binary32;  X [N][d] local models and
 *   e [d] global error are updated in place.
 * Optional outputs (NULL to skip): the uplink messages of every worker
 * (up_words [N][W], up_scales [N][T], up_idx/up_val [N][K]), the downlink message
 * (down_words [W], down_scales [T], down_idx/down_val [K]) and v [d].
 * W = sum_t ceil(n_t/32), K = sum_t k_t.
 * Random-k sides take their subsets from up_sets [N][K] and down_set [K] (NULL otherwise).
 * Returns 0 on success, -1 out of memory, -2 unknown compressor, -3 bad or missing subset.
 */
int liec_oracle_step_sets(int32_t N, int64_t d, int32_t T, const int64_t *off,
                     int32_t up, int32_t down, const int64_t *k,
                     const uint32_t *up_sets, const uint32_t *down_set,
                     const float *G, float lr, float *X, float *e,
                     uint32_t *up_words, float *up_scales, uint32_t *up_idx, float *up_val,
                     uint32_t *down_words, float *down_scales, uint32_t *down_idx, float *down_val,
                     float *v_out)
{
    int64_t W = 0, K = 0;
    for (int32_t t = 0; t < T; ++t) {
        W += words_of(off[t + 1] - off[t]);
        if (k) K += k[t];
    }
    float *P = (float *)malloc((size_t)N * (size_t)d * sizeof(float));   /* decoded p^i */
    float *v = (float *)malloc((size_t)d * sizeof(float));
    float *p = (float *)malloc((size_t)d * sizeof(float));               /* decoded p */
    uint32_t *tw = (uint32_t *)malloc((size_t)(W ? W : 1) * sizeof(uint32_t));
    float *ts = (float *)malloc((size_t)T * sizeof(float));
    uint32_t *ti = (uint32_t *)malloc((size_t)(K ? K : 1) * sizeof(uint32_t));
    float *tv = (float *)malloc((size_t)(K ? K : 1) * sizeof(float));
    int rc = 0;
    if (!P || !v || !p || !tw || !ts || !ti || !tv) { rc = -1; goto done; }

    /* Uplink: every worker compresses its own gradient. */
    for (int32_t i = 0; i < N && rc == 0; ++i) {
        rc = compress(up, G + (size_t)i * d, d, T, off, k,
                      up_sets ? up_sets + (size_t)i * K : NULL,
                      up_words ? up_words + (size_t)i * W : tw,
                      up_scales ? up_scales + (size_t)i * T : ts,
                      up_idx ? up_idx + (size_t)i * K : ti,
                      up_val ? up_val + (size_t)i * K : tv,
                      P + (size_t)i * d);
    }
    if (rc) goto done;

    /* Server: average in worker order, add the global error. */
    for (int64_t j = 0; j < d; ++j) {
        float acc = 0.0f;
        for (int32_t i = 0; i < N; ++i) acc = acc + P[(size_t)i * d + j];
        float mean = acc / (float)N;
        v[j] = e[j] + mean;
    }
    if (v_out) memcpy(v_out, v, (size_t)d * sizeof(float));

    /* Downlink: the same operator applied to v. */
    rc = compress(down, v, d, T, off, k, down_set,
                  down_words ? down_words : tw, down_scales ? down_scales : ts,
                  down_idx ? down_idx : ti, down_val ? down_val : tv, p);
    if (rc) goto done;

    /* Global error. */
    for (int64_t j = 0; j < d; ++j) e[j] = v[j] - p[j];

    /* Local immediate error compensation and model update. */
    for (int32_t i = 0; i < N; ++i) {
        const float *g = G + (size_t)i * d;
        const float *pi = P + (size_t)i * d;
        float *x = X + (size_t)i * d;
        for (int64_t j = 0; j < d; ++j) {
            float diff = p[j] - pi[j];
            float u = diff + g[j];
            float step = lr * u;
            x[j] = x[j] - step;
        }
    }

done:
    free(P); free(v); free(p); free(tw); free(ts); free(ti); free(tv);
    return rc;
}

/* The same iteration for the compressors that need no subset. */
int liec_oracle_step(int32_t N, int64_t d, int32_t T, const int64_t *off,
                     int32_t up, int32_t down, const int64_t *k,
                     const float *G, float lr, float *X, float *e,
                     uint32_t *up_words, float *up_scales, uint32_t *up_idx, float *up_val,
                     uint32_t *down_words, float *down_scales, uint32_t *down_idx, float *down_val,
                     float *v_out)
{
    return liec_oracle_step_sets(N, d, T, off, up, down, k, NULL, NULL, G, lr, X, e,
                                 up_words, up_scales, up_idx, up_val,
                                 down_words, down_scales, down_idx, down_val, v_out);
}

/*
 * Model-averaging iteration of Algorithm 1 (the branch with (t+1) mod period == 0):
 *   p^i = g^i,   v = e + (1/N) sum_i g^i,   p = v,   e' = v - p = 0,
 *   xbar = (1/N) sum_i x^i,   x^i <- xbar - eta (p - p^i + g^i).
 * Same arithmetic readings as the compressed iteration: sums over workers run in worker order
 * in binary32 from +0 and are divided by (float)N; the update is ((p - p^i) + g), times eta,
 * subtracted from xbar.  Optional outputs v_out [d] and xbar_out [d].
 * Also used for the algorithm's final output, xbar_T = mean_i x_T^i (liec_oracle_mean_params).
 */
void liec_oracle_mean_params(int32_t N, int64_t d, const float *X, float *xbar)
{
    for (int64_t j = 0; j < d; ++j) {
        float acc = 0.0f;
        for (int32_t i = 0; i < N; ++i) acc = acc + X[(size_t)i * d + j];
        xbar[j] = acc / (float)N;
    }
}

int liec_oracle_average_step(int32_t N, int64_t d, const float *G, float lr, float *X, float *e,
                             float *v_out, float *xbar_out)
{
    float *v = (float *)malloc((size_t)d * sizeof(float));
    float *xbar = (float *)malloc((size_t)d * sizeof(float));
    if (!v || !xbar) { free(v); free(xbar); return -1; }
    for (int64_t j = 0; j < d; ++j) {
        float acc = 0.0f;
        for (int32_t i = 0; i < N; ++i) acc = acc + G[(size_t)i * d + j];
        float gmean = acc / (float)N;
        v[j] = e[j] + gmean;
    }
    liec_oracle_mean_params(N, d, X, xbar);
    for (int32_t i = 0; i < N; ++i) {
        const float *g = G + (size_t)i * d;
        float *x = X + (size_t)i * d;
        for (int64_t j = 0; j < d; ++j) {
            float delta = v[j] - g[j];    /* p - p^i with p = v, p^i = g^i */
            float upd = delta + g[j];
            float scaled = lr * upd;
            x[j] = xbar[j] - scaled;
        }
    }
    for (int64_t j = 0; j < d; ++j) e[j] = v[j] - v[j];   /* e' = v - p, p = v */
    if (v_out) memcpy(v_out, v, (size_t)d * sizeof(float));
    if (xbar_out) memcpy(xbar_out, xbar, (size_t)d * sizeof(float));
    free(v); free(xbar);
    return 0;
}

/* ---- seeded draw of the random-k subsets (Def. 3) ----------------------------------------
 *
 * Def. 3 asks for S uniform over the k-element subsets of a segment.  Ranking the elements by
 * independent, identically distributed scores and keeping the k highest gives exactly that (the
 * ranking is a uniformly random permutation), up to equal scores, which go to the lower index.
 * The scores come from the counter-based generator Philox4x32-10 (Salmon, Moraes, Dror, Shaw:
 * "Parallel random numbers: as easy as 1, 2, 3", SC 2011), so that a sender and a receiver who
 * share (seed, epoch) compute the same subsets without exchanging indices:
 *
 *   key     = (seed mod 2^32, seed div 2^32)
 *   counter = (q, t, row, epoch)   q = block of four consecutive elements of segment t,
 *                                  row = worker index for an uplink subset, N for the server's
 *   the four output words go to elements 4q, 4q+1, 4q+2, 4q+3 of the segment (in that order)
 *   score   = word >> 2            (30 bits)
 */

static void philox_round(uint32_t c[4], const uint32_t k[2])
{
    const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c[1] ^ k[0];
    const uint32_t n2 = hi0 ^ c[3] ^ k[1];
    c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

/* Philox4x32 with 10 rounds: out = the block for this counter and key. */
void liec_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c[4] = { ctr[0], ctr[1], ctr[2], ctr[3] };
    uint32_t k[2] = { key[0], key[1] };
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }   /* key schedule: Weyl sequence */
        philox_round(c, k);
    }
    out[0] = c[0]; out[1] = c[1]; out[2] = c[2]; out[3] = c[3];
}

/* Scores of the n elements of segment t for the subset of `row` in draw `epoch`. */
void liec_oracle_subset_scores(uint64_t seed, uint32_t epoch, uint32_t row, uint32_t t,
                               int64_t n, uint32_t *scores)
{
    const uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    for (int64_t j = 0; j < n; ++j) {
        const uint32_t ctr[4] = { (uint32_t)(j / 4), t, row, epoch };
        uint32_t out[4];
        liec_oracle_philox4x32_10(ctr, key, out);
        scores[j] = out[j % 4] >> 2;
    }
}

typedef struct { uint32_t score; uint32_t pos; } scorepos;

static int by_score_then_index(const void *a, const void *b)
{
    const scorepos *p = (const scorepos *)a, *q = (const scorepos *)b;
    if (p->score != q->score) return p->score > q->score ? -1 : 1;   /* higher score first */
    if (p->pos != q->pos) return p->pos > q->pos ? 1 : -1;           /* lower index first */
    return 0;
}

static int by_value(const void *a, const void *b)
{
    const uint32_t x = *(const uint32_t *)a, y = *(const uint32_t *)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

/* The k positions (0-based inside the segment) with the highest scores, ascending.  Returns 0,
 * or -1 when memory runs out. */
int liec_oracle_subset_from_scores(const uint32_t *scores, int64_t n, int64_t k, uint32_t *subset)
{
    scorepos *order = (scorepos *)malloc((size_t)n * sizeof(scorepos));
    if (!order) return -1;
    for (int64_t j = 0; j < n; ++j) { order[j].score = scores[j]; order[j].pos = (uint32_t)j; }
    qsort(order, (size_t)n, sizeof(scorepos), by_score_then_index);
    for (int64_t r = 0; r < k; ++r) subset[r] = order[r].pos;
    qsort(subset, (size_t)k, sizeof(uint32_t), by_value);
    free(order);
    return 0;
}

/* The subsets of `rows` rows (workers 0..N-1, then the server as row N when rows = N+1) for
 * every segment: sets [rows][K] flat indices, segment after segment, ascending inside a
 * segment; the layout liec_oracle_step_sets takes.  Returns 0, or -1 when memory runs out. */
int liec_oracle_draw_subsets(uint64_t seed, uint32_t epoch, int32_t rows, int32_t T,
                             const int64_t *off, const int64_t *k, uint32_t *sets)
{
    int64_t K = 0, nmax = 0;
    for (int32_t t = 0; t < T; ++t) {
        K += k[t];
        if (off[t + 1] - off[t] > nmax) nmax = off[t + 1] - off[t];
    }
    uint32_t *scores = (uint32_t *)malloc((size_t)nmax * sizeof(uint32_t));
    if (!scores) return -1;
    int rc = 0;
    for (int32_t row = 0; row < rows && rc == 0; ++row) {
        int64_t koff = 0;
        for (int32_t t = 0; t < T && rc == 0; ++t) {
            const int64_t n = off[t + 1] - off[t];
            uint32_t *dst = sets + (size_t)row * K + koff;
            liec_oracle_subset_scores(seed, epoch, (uint32_t)row, (uint32_t)t, n, scores);
            rc = liec_oracle_subset_from_scores(scores, n, k[t], dst);
            for (int64_t r = 0; r < k[t]; ++r) dst[r] += (uint32_t)off[t];   /* flat index */
            koff += k[t];
        }
    }
    free(scores);
    return rc;
}
