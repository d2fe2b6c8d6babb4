/*
 * CPU oracle for the composed-prefill hot path.  TEST INFRASTRUCTURE ONLY:
 * it is what the CUDA library is checked against and what the bench times as
 * its CPU baseline; no product code path may call it.
 *
 * Plain definitions in fp64, one token / one row at a time, no tiling, no
 * online softmax, no page skipping.  It shares no code with the CUDA library.
 *
 *   oracle_placement      - "placement before preparation" (Sec. 5.3): the request's
 *                           final KV slots are fixed first; storage blocks of B
 *                           tokens, ceil(n/B) per unit, not adjacent (Sec. 5.1).
 *   oracle_rope_rotate    - rotary embedding of one head vector by an angle index
 *                           delta (Sec. 2.2: queries and keys are rotated, values
 *                           are not; a cached key is brought to its new offset).
 *   oracle_assemble       - "preparing cache hits" + "completing prefill" (Sec. 5.3):
 *                           cached rows placed at request positions with keys
 *                           rotated to the new positions; recomputed rows private
 *                           to the request override cached ones.
 *   oracle_e4m3_*         - the 8-bit storage form of cached units (1-4-3 float, bias 7, no
 *                           infinities, maximum 448): decode, and encode with round-to-nearest-
 *                           even and saturation.  The paper stores conventional 16-bit K/V
 *                           (Sec. 8); the 8-bit tier is this build's extension and these two
 *                           functions are its definition.
 *   oracle_f64_to_bf16_rne - one round-to-nearest-even of a double to bf16 (how an expanded
 *                           8-bit row is defined: the exact product code x scale, rounded once).
 *   oracle_attention_rows - the extend pass restricted to the recompute rows
 *                           (Sec. 5.3, Sec. 6.1 "Implementation"): causal softmax
 *                           attention of a query at position p over keys 0..p.
 *   oracle_attention_rows_qf64 - the same with the queries given as doubles (decoded 8-bit
 *                           queries of this build's 8-bit-key attention).
 *   oracle_assemble_ex(.., fresh_k_raw) - fresh keys handed over before rotation (Sec. 6.1: the
 *                           forward path captures pre-RoPE keys): the request sees them rotated
 *                           for their positions.
 *
 * Pins (tests/test_oracle_pins.py): composition and relative-position identities,
 * one-hot closed form, a library rotary routine (also for the fresh_k_raw branch), a 2-D
 * rotation matrix, the paper's worked position example, brute-force attention (bf16 and
 * fp64 queries), library causal attention, uniform-softmax closed form, per-token placement
 * loop and hand-worked slot numbers (tests/golden/placement_slots.txt), the retained form
 * R(-(p0 + i)) with one worked number, the library's e4m3 and bf16 conversions, exact
 * rational arithmetic for the single rounding of code x scale.  No function is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* -------------------------------------------------------------------------
 * 8-bit floating point "e4m3": sign, 4 exponent bits (bias 7), 3 mantissa bits.
 * Exponent field 0 holds subnormals m * 2^-9; field 15 with mantissa 7 is NaN,
 * every other pattern is finite (largest 1.75 * 2^8 = 448).  No infinities.
 * ------------------------------------------------------------------------- */
double oracle_e4m3_to_double(uint8_t b)
{
    int sign = b >> 7, e = (b >> 3) & 15, m = b & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* Nearest representable value, ties to the even mantissa; magnitudes beyond 448 (and
 * infinities) saturate to +-448; NaN stays NaN.  The input is a float: the decision
 * is taken on that float exactly (every float is a dyadic rational, so the comparison
 * with the two neighbouring codes is exact in double arithmetic). */
uint8_t oracle_f32_to_e4m3(float f)
{
    uint8_t sign;
    double a, lo_v, hi_v;
    int lo, hi;
    if (isnan(f)) return 0x7f;
    sign = signbit(f) ? 0x80 : 0x00;
    a = fabs((double)f);
    if (a >= 448.0) return sign | 0x7e;
    /* codes 0x00..0x7e are increasing in value: bisect for the last code <= a */
    lo = 0; hi = 0x7e;
    while (hi - lo > 1) {
        int mid = (lo + hi) / 2;
        if (oracle_e4m3_to_double((uint8_t)mid) <= a) lo = mid; else hi = mid;
    }
    lo_v = oracle_e4m3_to_double((uint8_t)lo);
    hi_v = oracle_e4m3_to_double((uint8_t)hi);
    if (a - lo_v < hi_v - a) return sign | (uint8_t)lo;
    if (a - lo_v > hi_v - a) return sign | (uint8_t)hi;
    return sign | (uint8_t)((lo & 1) ? hi : lo);      /* tie: even mantissa */
}

void oracle_e4m3_decode(const uint8_t *in, double *out, long n)
{
    for (long i = 0; i < n; ++i) out[i] = oracle_e4m3_to_double(in[i]);
}

void oracle_e4m3_encode(const float *in, uint8_t *out, long n)
{
    for (long i = 0; i < n; ++i) out[i] = oracle_f32_to_e4m3(in[i]);
}

/* -------------------------------------------------------------------------
 * Placement (Sec. 5.3 "Placement before preparation"; Sec. 5.1 storage blocks).
 * Request r takes the next ceil(T_r / B) ids of free_pages, in batch order.
 * src_slot[p] = pool slot (page * B + offset) holding the cached row that lands
 * at position p, -1 when no cached unit covers p.  fresh_idx[p] = index into the
 * recompute list when p is recomputed, else -1.
 * Returns 0, or a negative number for a batch that has no valid layout.
 * ------------------------------------------------------------------------- */
int oracle_placement(int batch, const int32_t *seq_len, const int32_t *unit_off,
                     const int32_t *unit_len, const int32_t *unit_target_pos,
                     const int32_t *unit_page_off, const int32_t *unit_pages,
                     const int32_t *recompute_off, const int32_t *recompute_pos,
                     const int32_t *free_pages, int n_free, int page_size,
                     const int32_t *unit_src_offset /* nullable: 0 */,
                     int32_t *page_off, int32_t *pages, int32_t *src_slot, int32_t *fresh_idx)
{
    int next_free = 0;
    long tok_base = 0;
    page_off[0] = 0;
    for (int r = 0; r < batch; ++r) {
        int T = seq_len[r];
        int need = (T + page_size - 1) / page_size;
        if (next_free + need > n_free) return -1;
        for (int k = 0; k < need; ++k) pages[page_off[r] + k] = free_pages[next_free + k];
        next_free += need;
        page_off[r + 1] = page_off[r] + need;
        for (int p = 0; p < T; ++p) { src_slot[tok_base + p] = -1; fresh_idx[tok_base + p] = -1; }
        for (int u = unit_off[r]; u < unit_off[r + 1]; ++u) {
            int cached = unit_page_off[u + 1] > unit_page_off[u];
            for (int i = 0; i < unit_len[u]; ++i) {
                int p = unit_target_pos[u] + i;
                if (p < 0 || p >= T) return -2;
                if (!cached) continue;
                if (src_slot[tok_base + p] != -1) return -3;            /* two units on one position */
                int si = i + (unit_src_offset ? unit_src_offset[u] : 0);   /* token index inside the source pages */
                src_slot[tok_base + p] = unit_pages[unit_page_off[u] + si / page_size] * page_size + si % page_size;
            }
        }
        for (int j = recompute_off[r]; j < recompute_off[r + 1]; ++j) {
            int p = recompute_pos[j];
            if (p < 0 || p >= T) return -4;
            if (j > recompute_off[r] && recompute_pos[j - 1] >= p) return -5;
            fresh_idx[tok_base + p] = j;
        }
        for (int p = 0; p < T; ++p)
            if (src_slot[tok_base + p] < 0 && fresh_idx[tok_base + p] < 0) return -6;   /* nobody supplies p */
        tok_base += T;
    }
    return 0;
}

/* -------------------------------------------------------------------------
 * Rotary embedding of one head vector by delta positions (Sec. 2.2).
 * Pair m has frequency w_m = theta^(-2m/D) (or inv_freq[m] when given).
 * pairing 0: pair m = (x[m], x[m + D/2]); pairing 1: pair m = (x[2m], x[2m+1]).
 * (a, b) -> (a cos(delta w) - b sin(delta w),  b cos(delta w) + a sin(delta w)).
 * ------------------------------------------------------------------------- */
void oracle_rope_rotate(const double *x, double *out, int D, double delta, double theta,
                        const double *inv_freq, int pairing)
{
    int half = D / 2;
    for (int m = 0; m < half; ++m) {
        double w = inv_freq ? inv_freq[m] : pow(theta, -2.0 * (double)m / (double)D);
        double ang = delta * w;
        double c = cos(ang), s = sin(ang);
        int ia = pairing ? 2 * m : m;
        int ib = pairing ? 2 * m + 1 : m + half;
        double a = x[ia], b = x[ib];
        out[ia] = a * c - b * s;
        out[ib] = b * c + a * s;
    }
}

/* -------------------------------------------------------------------------
 * Assembled K and V of request r (Sec. 5.3 "Preparing cache hits", "Completing
 * prefill").  For every position p < T:
 *   recomputed position j  -> K = k_new[j], V = v_new[j] (bit copies); with fresh_k_raw the fresh keys
 *                             are un-rotated projections and K = k_new[j] rotated for position p
 *                             (Sec. 5.3 "Completing prefill", Sec. 6.1), a bit copy only at p = 0;
 *   otherwise, cached unit u at offset i = p - target_pos(u):
 *        V = pool row (bit copy: values carry no rotation),
 *        K = pool row rotated by delta = (target_pos(u) + tstride(u) * i) - (cached_pos(u) + stride(u) * i),
 *            tstride = 1 unless given (0 = every token rotated for position target_pos(u): the form in
 *            which a freshly computed unit is retained when target_pos = 0, Sec. 5.3 / 6.1);
 *        the unit's token i sits at source slot (src_offset(u) + i) of its pages (src_offset 0 unless given).
 * k_asm is fp64 and left unrounded.  k_bits / k_exact: rows whose result is a bit
 * copy (recomputed rows and delta == 0) are given as bf16 bits with k_exact = 1.
 * ------------------------------------------------------------------------- */
/* Nearest bf16 (8 significant bits, float's exponent range), ties to even, of a double: ONE rounding
 * of the exact value.  Written with frexp / nearbyint (the default rounding mode is to-nearest-even). */
uint16_t oracle_f64_to_bf16_rne(double x)
{
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x), m, q;
    int e, prec = 8;
    float f;
    uint32_t u;
    if (isnan(x)) return 0x7fc0;
    if (a == 0.0) return sign;
    if (isinf(x)) return sign | 0x7f80;
    m = frexp(a, &e);                       /* a = m * 2^e, 0.5 <= m < 1 */
    if (e < -125) prec = 8 - (-125 - e);    /* below 2^-126 the spacing is fixed at 2^-133 */
    if (prec < 0) return sign;
    q = nearbyint(ldexp(m, prec));          /* integer with at most `prec` bits (or 2^prec after a carry) */
    a = ldexp(q, e - prec);
    if (a >= ldexp(1.0, 128)) return sign | 0x7f80;
    f = (float)a;                           /* exact: a has at most 8 significant bits */
    memcpy(&u, &f, sizeof u);
    return sign | (uint16_t)(u >> 16);
}

/* 8-bit source pools (src_fmt 1; this build's extension, see oracle_e4m3_*): a stored code c
 * stands for c * scale.  The product of a code (4 significant bits) and a float scale (24) is exact
 * in fp64.  The 16-bit row that reaches the destination is that exact product rounded ONCE to
 * nearest-even bf16, for V and for keys whose shift is 0; rotated keys are computed from the exact
 * product in fp64 and left unrounded like every other rotated key. */
int oracle_assemble_ex(int r, const int32_t *seq_len, const int32_t *unit_off,
                    const int32_t *unit_len, const int32_t *unit_cached_pos,
                    const int32_t *unit_cached_stride, const int32_t *unit_target_pos,
                    const int32_t *unit_page_off, const int32_t *unit_pages,
                    const int32_t *recompute_off, const int32_t *recompute_pos,
                    int page_size, int H_kv, int D, double theta, const double *inv_freq, int pairing,
                    const void *k_pool_any, const void *v_pool_any,
                    const uint16_t *k_new, const uint16_t *v_new,
                    const int32_t *unit_src_offset /* nullable */, const int32_t *unit_target_stride /* nullable */,
                    int src_fmt, float k_scale, float v_scale, int fresh_k_raw,
                    double *k_asm, uint16_t *v_asm, uint16_t *k_bits, uint8_t *k_exact, int32_t *delta_out);

int oracle_assemble(int r, const int32_t *seq_len, const int32_t *unit_off,
                    const int32_t *unit_len, const int32_t *unit_cached_pos,
                    const int32_t *unit_cached_stride, const int32_t *unit_target_pos,
                    const int32_t *unit_page_off, const int32_t *unit_pages,
                    const int32_t *recompute_off, const int32_t *recompute_pos,
                    int page_size, int H_kv, int D, double theta, const double *inv_freq, int pairing,
                    const uint16_t *k_pool, const uint16_t *v_pool,
                    const uint16_t *k_new, const uint16_t *v_new,
                    const int32_t *unit_src_offset /* nullable */, const int32_t *unit_target_stride /* nullable */,
                    double *k_asm, uint16_t *v_asm, uint16_t *k_bits, uint8_t *k_exact, int32_t *delta_out)
{
    return oracle_assemble_ex(r, seq_len, unit_off, unit_len, unit_cached_pos, unit_cached_stride, unit_target_pos,
                              unit_page_off, unit_pages, recompute_off, recompute_pos, page_size, H_kv, D, theta,
                              inv_freq, pairing, k_pool, v_pool, k_new, v_new, unit_src_offset, unit_target_stride,
                              0, 1.0f, 1.0f, 0, k_asm, v_asm, k_bits, k_exact, delta_out);
}

int oracle_assemble_ex(int r, const int32_t *seq_len, const int32_t *unit_off,
                    const int32_t *unit_len, const int32_t *unit_cached_pos,
                    const int32_t *unit_cached_stride, const int32_t *unit_target_pos,
                    const int32_t *unit_page_off, const int32_t *unit_pages,
                    const int32_t *recompute_off, const int32_t *recompute_pos,
                    int page_size, int H_kv, int D, double theta, const double *inv_freq, int pairing,
                    const void *k_pool_any, const void *v_pool_any,
                    const uint16_t *k_new, const uint16_t *v_new,
                    const int32_t *unit_src_offset /* nullable */, const int32_t *unit_target_stride /* nullable */,
                    int src_fmt, float k_scale, float v_scale, int fresh_k_raw,
                    double *k_asm, uint16_t *v_asm, uint16_t *k_bits, uint8_t *k_exact, int32_t *delta_out)
{
    const uint16_t *k_pool = (const uint16_t *)k_pool_any, *v_pool = (const uint16_t *)v_pool_any;
    const uint8_t *k_pool8 = (const uint8_t *)k_pool_any, *v_pool8 = (const uint8_t *)v_pool_any;
    int T = seq_len[r];
    size_t row = (size_t)H_kv * D;
    uint8_t *have = (uint8_t *)calloc((size_t)T + 1, 1);
    double *tmp = (double *)malloc(sizeof(double) * D);
    for (int p = 0; p < T; ++p) { k_exact[p] = 0; delta_out[p] = 0; }
    for (int u = unit_off[r]; u < unit_off[r + 1]; ++u) {
        if (unit_page_off[u + 1] <= unit_page_off[u]) continue;
        for (int i = 0; i < unit_len[u]; ++i) {
            int p = unit_target_pos[u] + i;
            int si = i + (unit_src_offset ? unit_src_offset[u] : 0);
            size_t slot = (size_t)unit_pages[unit_page_off[u] + si / page_size] * page_size + si % page_size;
            int tstride = unit_target_stride ? unit_target_stride[u] : 1;
            int delta = (unit_target_pos[u] + tstride * i) - (unit_cached_pos[u] + unit_cached_stride[u] * i);
            delta_out[p] = delta;
            if (src_fmt == 0) memcpy(v_asm + (size_t)p * row, v_pool + slot * row, row * sizeof(uint16_t));
            else
                for (size_t e = 0; e < row; ++e)
                    v_asm[(size_t)p * row + e] = oracle_f64_to_bf16_rne(oracle_e4m3_to_double(v_pool8[slot * row + e]) * (double)v_scale);
            for (int h = 0; h < H_kv; ++h) {
                double *dst = k_asm + (size_t)p * row + (size_t)h * D;
                for (int d = 0; d < D; ++d)
                    tmp[d] = src_fmt == 0 ? bf16_to_double(k_pool[slot * row + (size_t)h * D + d])
                                          : oracle_e4m3_to_double(k_pool8[slot * row + (size_t)h * D + d]) * (double)k_scale;
                oracle_rope_rotate(tmp, dst, D, (double)delta, theta, inv_freq, pairing);
            }
            if (delta == 0) {
                k_exact[p] = 1;
                if (src_fmt == 0) memcpy(k_bits + (size_t)p * row, k_pool + slot * row, row * sizeof(uint16_t));
                else
                    for (size_t e = 0; e < row; ++e)
                        k_bits[(size_t)p * row + e] = oracle_f64_to_bf16_rne(oracle_e4m3_to_double(k_pool8[slot * row + e]) * (double)k_scale);
            }
            have[p] = 1;
        }
    }
    for (int j = recompute_off[r]; j < recompute_off[r + 1]; ++j) {
        int p = recompute_pos[j];
        memcpy(v_asm + (size_t)p * row, v_new + (size_t)j * row, row * sizeof(uint16_t));
        memcpy(k_bits + (size_t)p * row, k_new + (size_t)j * row, row * sizeof(uint16_t));
        if (fresh_k_raw && p != 0) {
            /* the fresh keys were handed over BEFORE rotation (Sec. 6.1: pre-RoPE keys are captured):
             * the request's own row is the key rotated for its position p, in fp64, unrounded */
            for (int h = 0; h < H_kv; ++h) {
                for (int d = 0; d < D; ++d) tmp[d] = bf16_to_double(k_new[(size_t)j * row + (size_t)h * D + d]);
                oracle_rope_rotate(tmp, k_asm + (size_t)p * row + (size_t)h * D, D, (double)p, theta, inv_freq, pairing);
            }
            k_exact[p] = 0;
            delta_out[p] = p;
        } else {
            for (size_t e = 0; e < row; ++e) k_asm[(size_t)p * row + e] = bf16_to_double(k_new[(size_t)j * row + e]);
            k_exact[p] = 1;
            delta_out[p] = 0;
        }
        have[p] = 1;
    }
    int missing = 0;
    for (int p = 0; p < T; ++p) missing += !have[p];
    free(have);
    free(tmp);
    return missing ? -1 : 0;
}

/* -------------------------------------------------------------------------
 * Attention rows (Sec. 5.3 "Completing prefill").  Row i is query token row_q[i]
 * (index into q [n_q][H_q][D]) with head row_h[i] at position row_pos[i]; it
 * reads kv head row_h[i] / g (g = H_q / H_kv):
 *     s_t = scale * <q, K[t]>            t = 0 .. pos
 *     O   = sum_t softmax(s)_t V[t]
 *     LSE = log sum_t exp(s_t)
 * ------------------------------------------------------------------------- */
static void attention_row(const double *qd, int p, int kvh, int H_kv, int D, double scale,
                          const double *k_asm, const uint16_t *v_asm, double *o, double *lse)
{
    size_t row = (size_t)H_kv * D;
    double *s = (double *)malloc(sizeof(double) * ((size_t)p + 1));
    double mx = -INFINITY;
    for (int t = 0; t <= p; ++t) {
        const double *kv = k_asm + (size_t)t * row + (size_t)kvh * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += qd[d] * kv[d];
        s[t] = acc * scale;
        if (s[t] > mx) mx = s[t];
    }
    double denom = 0.0;
    for (int t = 0; t <= p; ++t) { s[t] = exp(s[t] - mx); denom += s[t]; }
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int t = 0; t <= p; ++t) {
        const uint16_t *vv = v_asm + (size_t)t * row + (size_t)kvh * D;
        double w = s[t] / denom;
        for (int d = 0; d < D; ++d) o[d] += w * bf16_to_double(vv[d]);
    }
    *lse = mx + log(denom);
    free(s);
}

void oracle_attention_rows(int T, int H_q, int H_kv, int D, double scale,
                           const double *k_asm, const uint16_t *v_asm, const uint16_t *q,
                           int n_rows, const int32_t *row_q, const int32_t *row_h, const int32_t *row_pos,
                           double *out, double *lse)
{
    int g = H_q / H_kv;
    (void)T;
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < n_rows; ++i) {
        int h = row_h[i];
        const uint16_t *qv = q + ((size_t)row_q[i] * H_q + h) * D;
        double *qd = (double *)malloc(sizeof(double) * D);
        for (int d = 0; d < D; ++d) qd[d] = bf16_to_double(qv[d]);
        attention_row(qd, row_pos[i], h / g, H_kv, D, scale, k_asm, v_asm, out + (size_t)i * D, lse + i);
        free(qd);
    }
}

/* The same rows with the queries given as doubles [n_q][H_q][D] (queries that are not bf16 numbers: the
 * decoded values of 8-bit codes times a scale - this build's 8-bit-key attention, which the paper does
 * not have). */
void oracle_attention_rows_qf64(int T, int H_q, int H_kv, int D, double scale,
                                const double *k_asm, const uint16_t *v_asm, const double *q,
                                int n_rows, const int32_t *row_q, const int32_t *row_h, const int32_t *row_pos,
                                double *out, double *lse)
{
    int g = H_q / H_kv;
    (void)T;
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < n_rows; ++i) {
        int h = row_h[i];
        attention_row(q + ((size_t)row_q[i] * H_q + h) * D, row_pos[i], h / g, H_kv, D, scale, k_asm, v_asm,
                      out + (size_t)i * D, lse + i);
    }
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
