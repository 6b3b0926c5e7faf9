/*
 * CPU oracle for the SirLLM retention pass.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what the retention pass computes,
 * written from the paper (Yao, Li, Zhao: "SirLLM: Streaming Infinite Retentive LLM",
 * Sections 3.1-3.3 and Algorithm 1).  It exists so that the CUDA library can be
 * checked against something that is obviously right; it is never part of the
 * product path, shares no code with it and is only called by the tests, the smoke
 * check and the benchmark's CPU-baseline leg.
 *
 * Arithmetic is double precision wherever arithmetic occurs, except where the
 * method itself fixes the precision: the entropy cache E is stored as fp32 and the
 * decay is one fp32 multiply per round (so that repeated decay is reproducible
 * bit for bit).  Build with -ffp-contract=off and without any fast-math option.
 *
 * Every function is pinned by tests/test_oracle_*.py against closed forms, the
 * paper's printed cache example, brute force on tiny caches, a long-double
 * recomputation and invariants.  The end-to-end composition (oracle_step) has no
 * number in the paper to be pinned to; it is pinned by seven rounds of Algorithm 1
 * worked by hand on a four-token cache (tests/golden/algorithm1_hand_trace.txt) and
 * by the invariants of the multi-round tests.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1

/* ---- reading one logit exactly ------------------------------------------------- */

static double logit_at(const void *row, int dtype, int64_t v)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)row)[v];
    /* bfloat16: the upper half of an IEEE binary32 */
    uint32_t bits = (uint32_t)((const uint16_t *)row)[v] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/*
 * Token Entropy of one token (Section 3.2, the display equation defining e_i):
 *     e = -log P(x | context),   P = softmax(z)[x]
 * with the natural logarithm.  Written as (m - z[x]) + log(sum_v exp(z[v] - m)),
 * m = max_v z[v]; both addends are >= 0.  A token id of -1 means that no
 * prediction exists for the position (the first token of a stream) and gives 0.
 * An id outside [0, V) other than -1 also gives 0 and raises *bad_id.
 */
double oracle_token_entropy(const void *row, int dtype, int64_t V, int32_t id, int *bad_id)
{
    if (id == -1)
        return 0.0;
    if (id < 0 || (int64_t)id >= V) {
        if (bad_id)
            *bad_id = 1;
        return 0.0;
    }
    double m = -INFINITY;
    for (int64_t v = 0; v < V; ++v) {
        double z = logit_at(row, dtype, v);
        if (z > m)
            m = z;
    }
    double s = 0.0;
    for (int64_t v = 0; v < V; ++v)
        s += exp(logit_at(row, dtype, v) - m);
    return (m - logit_at(row, dtype, id)) + log(s);
}

/* Scores of the T tokens of one round (Algorithm 1: E_t = Entropy([I_t, R_t])).
 * Row t of `logits` (row_stride elements apart) is the distribution token ids[t]
 * was drawn from.  Returns the number of out-of-range ids. */
int oracle_score(const void *logits, int dtype, int64_t T, int64_t V, int64_t row_stride,
                 const int32_t *ids, float *out_e)
{
    int n_bad = 0;
    size_t esz = dtype == ORACLE_F32 ? 4 : 2;
    for (int64_t t = 0; t < T; ++t) {
        int bad = 0;
        const char *row = (const char *)logits + (size_t)t * (size_t)row_stride * esz;
        out_e[t] = (float)oracle_token_entropy(row, dtype, V, ids[t], &bad);
        n_bad += bad;
    }
    return n_bad;
}

/*
 * Token Entropy from split-vocabulary partial results (same definition, Section 3.2): when a
 * logits row is cut into tiles and tile i is summarised by m_i = max of its logits and
 * s_i = sum over the tile of exp(z - m_i), then sum_v exp(z_v) = sum_i s_i exp(m_i) and
 *     e = log(sum_i s_i exp(m_i)) - z[x].
 * pairs = (m_0, s_0, m_1, s_1, ...) in fp32 as a producer would emit them; a tile with
 * s_i = 0 (fully masked) contributes nothing.  id rules as in oracle_token_entropy.
 */
double oracle_entropy_from_pairs(const float *pairs, int64_t n_tiles, float target_logit, int32_t id,
                                 int64_t V, int *bad_id)
{
    if (id == -1)
        return 0.0;
    if (id < 0 || (int64_t)id >= V) {
        if (bad_id)
            *bad_id = 1;
        return 0.0;
    }
    double M = -INFINITY;
    for (int64_t i = 0; i < n_tiles; ++i)
        if (pairs[2 * i + 1] > 0.0f && (double)pairs[2 * i] > M)
            M = (double)pairs[2 * i];
    double S = 0.0;
    for (int64_t i = 0; i < n_tiles; ++i)
        if (pairs[2 * i + 1] > 0.0f)
            S += (double)pairs[2 * i + 1] * exp((double)pairs[2 * i] - M);
    return (M - (double)target_logit) + log(S);
}

int oracle_score_pairs(const float *pairs, int64_t T, int64_t n_tiles, int64_t pair_row_stride,
                       const float *target_logit, const int32_t *ids, int64_t V, float *out_e)
{
    int n_bad = 0;
    for (int64_t t = 0; t < T; ++t) {
        int bad = 0;
        out_e[t] = (float)oracle_entropy_from_pairs(pairs + 2 * t * pair_row_stride, n_tiles,
                                                    target_logit[t], ids[t], V, &bad);
        n_bad += bad;
    }
    return n_bad;
}

/*
 * One rank's share of a logits row under a vocabulary-parallel LM head (Section 3.2, the sum in
 * the softmax split over column ranges): for the columns [v0, v1) of the row,
 *     m = max of the logits,   s = sum exp(z - m)   (m = 0, s = 0 for an empty or fully masked
 * range), both in double and rounded once to fp32; and the target logit z[id] if v0 <= id < v1,
 * else 0.  The pairs of all ranges of a row feed oracle_entropy_from_pairs.
 */
void oracle_range_pair(const void *row, int dtype, int64_t v0, int64_t v1, int32_t id, float *pair,
                       float *target)
{
    double m = -INFINITY;
    for (int64_t v = v0; v < v1; ++v) {
        double z = logit_at(row, dtype, v);
        if (z > m)
            m = z;
    }
    double s = 0.0;
    if (m > -INFINITY)
        for (int64_t v = v0; v < v1; ++v)
            s += exp(logit_at(row, dtype, v) - m);
    pair[0] = s > 0.0 ? (float)m : 0.0f;
    pair[1] = (float)s;
    *target = (id >= 0 && (int64_t)id >= v0 && (int64_t)id < v1) ? (float)logit_at(row, dtype, id) : 0.0f;
}

/* Memory decay (Section 3.3, E = E x eta_decay; Algorithm 1 applies it once per
 * round, after the round's scores were appended): one fp32 multiply per entry. */
void oracle_decay(float *E, int64_t l, float eta)
{
    for (int64_t i = 0; i < l; ++i) {
        volatile float p = E[i] * eta; /* volatile: keep the product a rounded fp32 */
        E[i] = p;
    }
}

/* Total order on fp32 bit patterns used to rank scores: larger key = larger score.
 * Negative values have all bits flipped, non-negative ones the sign bit set. */
uint32_t oracle_order_key(float x)
{
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

typedef struct {
    uint32_t key;
    int32_t slot;
} ranked_t;

static int by_score_desc_then_slot_asc(const void *pa, const void *pb)
{
    const ranked_t *a = pa, *b = pb;
    if (a->key != b->key)
        return a->key > b->key ? -1 : 1;
    return (a->slot > b->slot) - (a->slot < b->slot);
}

static int by_int_asc(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/*
 * Which slots stay (Sections 3.1 and 3.3; Algorithm 1, the branch taken when the
 * cache holds more than L tokens).  E[0..l) are the (already decayed) scores.
 *   l <= threshold : nothing is evicted, keep = 0..l-1.
 *   otherwise      : keep = sinks [0, n_sink)  U  the k = budget - n_sink - n_recent
 *                    best-scored slots of the middle [n_sink, l - n_recent)
 *                    U  recent [l - n_recent, l), listed in ascending slot order.
 * Ranking in the middle: higher score first, equal scores -> the lower slot first.
 * Returns the number of kept slots, or -1 on inconsistent parameters.
 */
int32_t oracle_select(const float *E, int32_t l, int32_t n_sink, int32_t n_recent, int32_t budget,
                      int32_t threshold, int32_t *keep)
{
    if (l < 0 || n_sink < 0 || n_recent < 0 || budget < n_sink + n_recent || threshold < budget)
        return -1;
    if (l <= threshold) {
        for (int32_t i = 0; i < l; ++i)
            keep[i] = i;
        return l;
    }
    int32_t lo = n_sink, hi = l - n_recent, k = budget - n_sink - n_recent;
    int32_t n_mid = hi - lo;
    ranked_t *mid = malloc(sizeof(ranked_t) * (size_t)(n_mid > 0 ? n_mid : 1));
    for (int32_t i = lo; i < hi; ++i) {
        mid[i - lo].key = oracle_order_key(E[i]);
        mid[i - lo].slot = i;
    }
    qsort(mid, (size_t)n_mid, sizeof(ranked_t), by_score_desc_then_slot_asc);
    int32_t n = 0;
    for (int32_t i = 0; i < lo; ++i)
        keep[n++] = i;
    for (int32_t r = 0; r < k; ++r)
        keep[n++] = mid[r].slot;
    for (int32_t i = hi; i < l; ++i)
        keep[n++] = i;
    free(mid);
    qsort(keep, (size_t)n, sizeof(int32_t), by_int_asc);
    return n;
}

/* X[Id] of Section 3.1: out[j] = in[keep[j]] for rows of row_bytes bytes, into a
 * separate output array. */
void oracle_gather_rows(const void *src, void *dst, int64_t row_bytes, const int32_t *keep,
                        int32_t n_keep)
{
    for (int32_t j = 0; j < n_keep; ++j)
        memcpy((char *)dst + (size_t)j * (size_t)row_bytes,
               (const char *)src + (size_t)keep[j] * (size_t)row_bytes, (size_t)row_bytes);
}

/*
 * One round of one stream, Algorithm 1 rotated so that the eviction of turn t+1
 * happens at the end of turn t (the caches the model sees are the same):
 *   append the round's T scores to E (and serial numbers to `serial`), l += T;
 *   decay all l scores once; if l > threshold select and compact E, serial and
 *   every K/V plane; return the new live length.
 * new_e          [T]  scores of the round's tokens (already computed)
 * E, serial      [capacity] per-slot score and token serial number, updated in place
 * k, v           [n_planes, capacity, row_bytes] caches whose slots [l, l+T) already
 *                hold the round's new rows; compacted in place through a scratch copy
 * keep           [max(threshold, .)] out: the kept slots (identity when nothing is evicted)
 * Returns the new live length, or -1 if l + T > capacity (nothing is changed).
 */
int32_t oracle_step(const float *new_e, int32_t T, float *E, int64_t *serial, int64_t *next_serial,
                    int32_t l, float eta, int32_t capacity, int32_t n_sink, int32_t n_recent,
                    int32_t budget, int32_t threshold, void *k, void *v, int64_t n_planes,
                    int64_t row_bytes, int32_t *keep)
{
    if (l + T > capacity)
        return -1;
    for (int32_t t = 0; t < T; ++t) {
        E[l + t] = new_e[t];
        if (serial)
            serial[l + t] = (*next_serial)++;
    }
    l += T;
    oracle_decay(E, l, eta);
    int32_t n_keep = oracle_select(E, l, n_sink, n_recent, budget, threshold, keep);
    if (n_keep < 0 || l <= threshold)
        return n_keep;

    float *E2 = malloc(sizeof(float) * (size_t)n_keep);
    for (int32_t j = 0; j < n_keep; ++j)
        E2[j] = E[keep[j]];
    memcpy(E, E2, sizeof(float) * (size_t)n_keep);
    free(E2);
    if (serial) {
        int64_t *s2 = malloc(sizeof(int64_t) * (size_t)n_keep);
        for (int32_t j = 0; j < n_keep; ++j)
            s2[j] = serial[keep[j]];
        memcpy(serial, s2, sizeof(int64_t) * (size_t)n_keep);
        free(s2);
    }
    size_t kept_bytes = (size_t)n_keep * (size_t)row_bytes;
    char *tmp = malloc(kept_bytes ? kept_bytes : 1);
    void *caches[2] = {k, v};
    for (int c = 0; c < 2; ++c) {
        if (!caches[c])
            continue;
        for (int64_t p = 0; p < n_planes; ++p) {
            char *plane = (char *)caches[c] + (size_t)p * (size_t)capacity * (size_t)row_bytes;
            oracle_gather_rows(plane, tmp, row_bytes, keep, n_keep);
            memcpy(plane, tmp, kept_bytes);
        }
    }
    free(tmp);
    return n_keep;
}

/* ---- the paper's comparison policies (Section 4.1.1) as keep-list generators ---------
 * They feed the same K/V gather as the entropy selection.  All use the trigger of
 * Algorithm 1 (nothing is evicted while l <= threshold) and list the kept slots ascending. */

/* StreamLLM (Sections 3.1, 4.1.1): the sink tokens and the most recent tokens only,
 * budget slots in all. */
int32_t oracle_keep_stream(int32_t l, int32_t n_sink, int32_t budget, int32_t threshold, int32_t *keep)
{
    if (l <= threshold) {
        for (int32_t i = 0; i < l; ++i)
            keep[i] = i;
        return l;
    }
    int32_t n = 0;
    for (int32_t i = 0; i < n_sink; ++i)
        keep[n++] = i;
    for (int32_t i = l - (budget - n_sink); i < l; ++i)
        keep[n++] = i;
    return n;
}

/* IntervalLLM (Section 4.1.1): the sink tokens, then one historical token every `interval`
 * slots, interval = floor(history length / cache size), until the cache is full.  The
 * configured recent window (0 in the paper's rows) is kept as in the entropy policy. */
int32_t oracle_keep_interval(int32_t l, int32_t n_sink, int32_t n_recent, int32_t budget,
                             int32_t threshold, int32_t *keep)
{
    if (l <= threshold) {
        for (int32_t i = 0; i < l; ++i)
            keep[i] = i;
        return l;
    }
    int32_t interval = l / budget;
    int32_t k = budget - n_sink - n_recent, n = 0;
    for (int32_t i = 0; i < n_sink; ++i)
        keep[n++] = i;
    for (int32_t i = n_sink, taken = 0; i < l - n_recent && taken < k; i += interval, ++taken)
        keep[n++] = i;
    for (int32_t i = l - n_recent; i < l; ++i)
        keep[n++] = i;
    return n;
}

/* Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, "Parallel random
 * numbers: as easy as 1, 2, 3", SC'11): ten rounds of two 32x32->64 multiplies. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0, c1 = n1, c2 = n2, c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0, out[1] = c1, out[2] = c2, out[3] = c3;
}

/* RandomLLM (Section 4.1.1): the sink tokens and a uniformly random choice of k historical
 * tokens.  Slot i of the middle draws the 24-bit number
 *     u_i = philox(counter = (i, round, stream, 0), key = seed)[0] >> 8
 * and the k largest stay (equal draws: the lower slot), which is a uniform k-subset. */
int32_t oracle_keep_random(int32_t l, int32_t n_sink, int32_t n_recent, int32_t budget,
                           int32_t threshold, uint64_t seed, int32_t stream, int32_t round,
                           int32_t *keep)
{
    if (l <= threshold) {
        for (int32_t i = 0; i < l; ++i)
            keep[i] = i;
        return l;
    }
    int32_t lo = n_sink, hi = l - n_recent, k = budget - n_sink - n_recent, n_mid = hi - lo;
    ranked_t *mid = malloc(sizeof(ranked_t) * (size_t)(n_mid > 0 ? n_mid : 1));
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int32_t i = lo; i < hi; ++i) {
        uint32_t ctr[4] = {(uint32_t)i, (uint32_t)round, (uint32_t)stream, 0u}, out[4];
        oracle_philox4x32_10(ctr, key, out);
        mid[i - lo].key = out[0] >> 8;
        mid[i - lo].slot = i;
    }
    qsort(mid, (size_t)n_mid, sizeof(ranked_t), by_score_desc_then_slot_asc);
    int32_t n = 0;
    for (int32_t i = 0; i < lo; ++i)
        keep[n++] = i;
    for (int32_t r = 0; r < k; ++r)
        keep[n++] = mid[r].slot;
    for (int32_t i = hi; i < l; ++i)
        keep[n++] = i;
    free(mid);
    qsort(keep, (size_t)n, sizeof(int32_t), by_int_asc);
    return n;
}

/* ---- re-indexing of positions for caches that hold keys AFTER rotary embedding ----------
 * Section 3.3 (the paragraph on positions): a token's position is its place inside the cache,
 * not in the text; after an eviction the kept tokens take positions 0..n-1 in slot order.  A
 * model that stores keys already rotated for the position they were written at therefore has
 * to turn the key that moved from slot keep[j] to slot j by the angle of (j - keep[j])
 * positions.  Rotary embedding (Su et al., RoFormer): pair i of a row, i < d/2, is the complex
 * number x + iy turned by the angle  position * theta_i,  theta_i = base^(-2i/d);
 * layout 0 pairs (row[i], row[i + d/2]), layout 1 pairs (row[2i], row[2i+1]). */
#define ORACLE_ROPE_HALF 0
#define ORACLE_ROPE_INTERLEAVED 1

void oracle_rope_rotate_f64(double *row, int32_t d, int32_t delta, double base, int layout)
{
    int32_t hp = d / 2;
    for (int32_t i = 0; i < hp; ++i) {
        double theta = pow(base, -2.0 * (double)i / (double)d);
        double ang = (double)delta * theta, c = cos(ang), s = sin(ang);
        double *px = layout == ORACLE_ROPE_HALF ? &row[i] : &row[2 * i];
        double *py = layout == ORACLE_ROPE_HALF ? &row[i + hp] : &row[2 * i + 1];
        double x = *px, y = *py;
        *px = x * c - y * s;
        *py = x * s + y * c;
    }
}

/* Round a double to the nearest value with `p` significant bits and minimum exponent
 * `emin` (ties to even; needs the default rounding mode), i.e. to bf16 (p = 8, emin = -126)
 * or fp16 (p = 11, emin = -14) without passing through fp32. */
static double round_to_format(double v, int p, int emin)
{
    if (v == 0.0 || isnan(v) || isinf(v))
        return v;
    int e;
    double m = frexp(v, &e); /* v = m * 2^e, 0.5 <= |m| < 1: the leading bit has weight 2^(e-1) */
    int keep = p;
    if (e - 1 < emin)
        keep = p - (emin - (e - 1)); /* subnormal: fewer bits */
    if (keep <= 0)
        return ldexp(nearbyint(ldexp(v, -(emin - p + 1))), emin - p + 1);
    return ldexp(nearbyint(ldexp(m, keep)), e - keep);
}

static double from_bits16(uint16_t h, int dtype_is_bf16)
{
    if (dtype_is_bf16) {
        uint32_t b = (uint32_t)h << 16;
        float f;
        memcpy(&f, &b, sizeof f);
        return (double)f;
    }
    int sign = h >> 15, ex = (h >> 10) & 31, fr = h & 1023;
    double v = ex == 0 ? ldexp((double)fr, -24) : ex == 31 ? (fr ? NAN : INFINITY)
                                                            : ldexp((double)(fr | 1024), ex - 25);
    return sign ? -v : v;
}

static uint16_t to_bits16(double v, int dtype_is_bf16)
{
    double r = dtype_is_bf16 ? round_to_format(v, 8, -126) : round_to_format(v, 11, -14);
    if (dtype_is_bf16) {
        float f = (float)r; /* exact: r has 8 significant bits */
        if (isinf(f) && !isinf(v))
            f = copysignf(INFINITY, f);
        uint32_t b;
        memcpy(&b, &f, sizeof b);
        return (uint16_t)(b >> 16);
    }
    uint16_t sign = signbit(r) ? 0x8000u : 0;
    double a = fabs(r);
    if (isnan(a))
        return sign | 0x7E00u;
    if (a >= 65520.0)
        return sign | 0x7C00u;
    if (a == 0.0)
        return sign;
    int e;
    double m = frexp(a, &e); /* a = m 2^e */
    if (e - 1 < -14)
        return sign | (uint16_t)ldexp(a, 24); /* subnormal: a / 2^-24, an integer < 1024 */
    return sign | (uint16_t)(((e - 1 + 15) << 10) | ((int)ldexp(m, 11) & 1023));
}

double oracle_round16(double v, int dtype_is_bf16)
{
    return from_bits16(to_bits16(v, dtype_is_bf16), dtype_is_bf16);
}

/* Re-rotate the live rows of one K plane in place: row j by (j - keep[j]) positions, computed
 * in double and rounded once to the storage type.  plane: [slots][d] 16-bit elements. */
void oracle_rerotate_plane(void *plane, int dtype_is_bf16, int32_t d, const int32_t *keep,
                           int32_t n_keep, double base, int layout)
{
    double *row = malloc(sizeof(double) * (size_t)d);
    for (int32_t j = 0; j < n_keep; ++j) {
        int32_t delta = j - keep[j];
        if (delta == 0)
            continue;
        uint16_t *h = (uint16_t *)plane + (size_t)j * (size_t)d;
        for (int32_t c = 0; c < d; ++c)
            row[c] = from_bits16(h[c], dtype_is_bf16);
        oracle_rope_rotate_f64(row, d, delta, base, layout);
        for (int32_t c = 0; c < d; ++c)
            h[c] = to_bits16(row[c], dtype_is_bf16);
    }
    free(row);
}
