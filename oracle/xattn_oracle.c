/*
 * TEST INFRASTRUCTURE -- not part of the product.
 *
 * Plain fp64 CPU oracle for the cross-decoder attention of the decoder-decoder
 * architecture ("You Only Cache Once", Section 2.2, the cross-decoder equation
 * block: Y = Attention(Q^l, K^, V^) + X, with "standard multi-head attention",
 * causal masking and grouped-query attention).
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code with the CUDA path.
 *
 * What it computes is the textbook definition, written out:
 *
 *   for sequence i, query head h (KV head c = h / G, G = Hq / Hkv), query row t:
 *     n_vis = clamp(N_i - T + t + 1, 0, N_i)          (causal, bottom-right aligned:
 *                                                      the cache already holds the T
 *                                                      new positions, a row sees itself)
 *     s_j   = scale * sum_e Q[i,h,t,e] * K[i,c,j,e]   for j < n_vis
 *     m     = max_j s_j
 *     p_j   = exp(s_j - m)
 *     O     = sum_j p_j V[i,c,j,:] / sum_j p_j
 *     LSE   = m + log(sum_j p_j)                       (natural log)
 *     n_vis = 0  ->  O = 0, LSE = -inf
 *
 * Two passes over the keys (max, then sums); no tiling, no online rescaling.
 *
 * Optional sliding window (Section 3.2, the window causal mask B_ij = 0 iff
 * i - C < j <= i, -inf otherwise): with window C > 0 the row at absolute position
 * i = N_i - T + t sees only the keys j with i - C < j <= i, i.e. the C most recent
 * ones, itself included.  C = 0 means no window (plain causal).
 *
 * Layout (the same bits the GPU reads): Q is [B, Hq, T, d] bf16.  K and V are
 * packed buffers of bf16; sequence i starts at token offset cu[i]; inside a
 * sequence the order is [Hkv, N_i, d] (head-major), the distance between heads
 * being kv_head_stride elements (0 means tight: N_i * d).
 *   element(i, c, j, e) = cu[i] * Hkv * d + c * head_stride_i + j * d + e
 *
 * Optional 8-bit cache (Section 1 assumes 8-bit K/V quantisation when it sizes a cache): K and V may be given
 * as FP8 E4M3 bytes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; exponent field 0 is
 * subnormal m/8 * 2^-6; 0x7F / 0xFF are NaN; no infinities) with one fp32 scale per KV head:
 * the value of an element is scale[c] * e4m3(byte).  Everything else is unchanged.
 *
 * Pins (tests/test_oracle_pins.py): single key, identical keys -> prefix means,
 * permutation invariance, split + merge = unsplit, brute force without max
 * subtraction, two-key logistic closed form, affine map of V, key shift,
 * GQA = MHA with repeated heads, chunk row = decode call, a library fp64
 * softmax-attention on small shapes.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

typedef struct {
    int32_t B, Hq, Hkv, d, T;
    double scale;
    const uint16_t *Q, *K, *V;
    const int32_t *cu;
    const int32_t *kv_len;
    int64_t kv_head_stride;
    int32_t window;
    /* 8-bit cache: when K8 is set, K and V above are unused */
    const uint8_t *K8, *V8;
    const float *k_scale, *v_scale;   /* [Hkv] */
} problem_t;

/* FP8 E4M3 byte -> value, from the format's definition. */
double oracle_e4m3_to_f64(uint8_t b)
{
    int sign = b >> 7, ex = (b >> 3) & 15, man = b & 7;
    double v;
    if (ex == 15 && man == 7) return NAN;
    if (ex == 0) v = ldexp((double)man / 8.0, -6);
    else v = ldexp(1.0 + (double)man / 8.0, ex - 7);
    return sign ? -v : v;
}

/* Element idx (in elements from the start of the packed buffer) of K (which = 0) or V (1). */
static double kv_val(const problem_t *p, int which, int c, int64_t idx)
{
    if (p->K8) {
        const uint8_t *buf = which ? p->V8 : p->K8;
        const float *sc = which ? p->v_scale : p->k_scale;
        return (double)sc[c] * oracle_e4m3_to_f64(buf[idx]);
    }
    return bf16_bits_to_f64((which ? p->V : p->K)[idx]);
}

static int64_t kv_base(const problem_t *p, int i, int c)
{
    int64_t hs = p->kv_head_stride ? p->kv_head_stride : (int64_t)p->kv_len[i] * p->d;
    return (int64_t)p->cu[i] * p->Hkv * p->d + (int64_t)c * hs;
}

static int64_t visible_keys(const problem_t *p, int i, int t)
{
    int64_t n = (int64_t)p->kv_len[i] - p->T + t + 1;
    if (n < 0) n = 0;
    if (n > p->kv_len[i]) n = p->kv_len[i];
    return n;
}

/* First key of the row's window: the mask keeps i - C < j, so the lowest kept j is
 * i - C + 1 (never below 0); without a window every key from 0 on is kept. */
static int64_t first_visible(const problem_t *p, int i, int t)
{
    if (p->window <= 0) return 0;
    int64_t pos = (int64_t)p->kv_len[i] - p->T + t;   /* absolute position of the query row */
    int64_t lo = pos - p->window + 1;
    return lo < 0 ? 0 : lo;
}

/* Attention of one query row over keys [j0, j1) of its KV head (already
 * clipped to the visible range by the caller).  scores is scratch of length
 * >= j1 - j0.  Writes d outputs and the log-sum-exp. */
static void row_over_range(const problem_t *p, int i, int h, int t,
                           int64_t j0, int64_t j1, double *scores,
                           double *out, double *lse)
{
    const int d = p->d;
    const int G = p->Hq / p->Hkv;
    const int c = h / G;
    const uint16_t *q = p->Q + (((int64_t)i * p->Hq + h) * p->T + t) * d;
    const int64_t kvb = kv_base(p, i, c);

    for (int e = 0; e < d; ++e) out[e] = 0.0;
    if (j1 <= j0) {
        *lse = -INFINITY;
        return;
    }
    double m = -INFINITY;
    for (int64_t j = j0; j < j1; ++j) {
        double s = 0.0;
        for (int e = 0; e < d; ++e) s += bf16_bits_to_f64(q[e]) * kv_val(p, 0, c, kvb + j * d + e);
        s *= p->scale;
        scores[j - j0] = s;
        if (s > m) m = s;
    }
    double denom = 0.0;
    for (int64_t j = j0; j < j1; ++j) {
        double w = exp(scores[j - j0] - m);
        denom += w;
        for (int e = 0; e < d; ++e) out[e] += w * kv_val(p, 1, c, kvb + j * d + e);
    }
    for (int e = 0; e < d; ++e) out[e] /= denom;
    *lse = m + log(denom);
}

static double resolve_scale(double scale, int d)
{
    return scale != 0.0 ? scale : 1.0 / sqrt((double)d);
}

static int check_shape(int B, int Hq, int Hkv, int d, int T)
{
    if (B < 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || T <= 0) return -1;
    if (Hq % Hkv) return -1;
    return 0;
}

/* Full output: O [B, Hq, T, d] and LSE [B, Hq, T], both fp64. */
int oracle_xattn(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t T, double scale,
                 const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                 const int32_t *cu, const int32_t *kv_len, int64_t kv_head_stride, int32_t window,
                 double *O, double *LSE)
{
    if (check_shape(B, Hq, Hkv, d, T) || window < 0) return -1;
    problem_t p = {B, Hq, Hkv, d, T, resolve_scale(scale, d), Q, K, V, cu, kv_len, kv_head_stride, window};
    int64_t max_len = 1;
    for (int i = 0; i < B; ++i)
        if (kv_len[i] > max_len) max_len = kv_len[i];
    int failed = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)max_len);
        if (!scores) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int i = 0; i < B; ++i)
            for (int h = 0; h < Hq; ++h) {
                if (!scores) continue;
                for (int t = 0; t < T; ++t) {
                    int64_t row = ((int64_t)i * Hq + h) * T + t;
                    row_over_range(&p, i, h, t, first_visible(&p, i, t), visible_keys(&p, i, t), scores,
                                   O + row * d, LSE + row);
                }
            }
        free(scores);
    }
    return failed ? -2 : 0;
}

/* Selected rows only: row r is (rows_b[r], rows_h[r], rows_t[r]); O [n_rows, d], LSE [n_rows]. */
int oracle_xattn_rows(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t T, double scale,
                      const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                      const int32_t *cu, const int32_t *kv_len, int64_t kv_head_stride, int32_t window,
                      int64_t n_rows, const int32_t *rows_b, const int32_t *rows_h,
                      const int32_t *rows_t, double *O, double *LSE)
{
    if (check_shape(B, Hq, Hkv, d, T) || window < 0) return -1;
    problem_t p = {B, Hq, Hkv, d, T, resolve_scale(scale, d), Q, K, V, cu, kv_len, kv_head_stride, window};
    for (int64_t r = 0; r < n_rows; ++r)
        if (rows_b[r] < 0 || rows_b[r] >= B || rows_h[r] < 0 || rows_h[r] >= Hq ||
            rows_t[r] < 0 || rows_t[r] >= T)
            return -1;
    int64_t max_len = 1;
    for (int i = 0; i < B; ++i)
        if (kv_len[i] > max_len) max_len = kv_len[i];
    int failed = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)max_len);
        if (!scores) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            if (!scores) continue;
            int i = rows_b[r], t = rows_t[r];
            row_over_range(&p, i, rows_h[r], t, first_visible(&p, i, t), visible_keys(&p, i, t), scores,
                           O + r * d, LSE + r);
        }
        free(scores);
    }
    return failed ? -2 : 0;
}

/* Merge of per-piece results by their log-sum-exp:
 *   LSE = log sum_s exp(LSE_s),  O = sum_s exp(LSE_s - LSE) O_s,
 * pieces with LSE_s = -inf carry no weight; all empty -> O = 0, LSE = -inf. */
static void merge_pieces(int S, int d, const double *po, const double *plse,
                         double *out, double *lse)
{
    double m = -INFINITY;
    for (int s = 0; s < S; ++s)
        if (plse[s] > m) m = plse[s];
    for (int e = 0; e < d; ++e) out[e] = 0.0;
    if (m == -INFINITY) {
        *lse = -INFINITY;
        return;
    }
    double denom = 0.0;
    for (int s = 0; s < S; ++s)
        if (plse[s] != -INFINITY) denom += exp(plse[s] - m);
    double total = m + log(denom);
    for (int s = 0; s < S; ++s) {
        if (plse[s] == -INFINITY) continue;
        double w = exp(plse[s] - total);
        for (int e = 0; e < d; ++e) out[e] += w * po[(int64_t)s * d + e];
    }
    *lse = total;
}

/* The same attention computed piecewise: the key axis is cut at the n_cuts
 * ascending positions cuts[] (absolute key indices, shared by all rows); every
 * piece [cuts[k], cuts[k+1]) (plus the ends) is evaluated on its own and the
 * pieces are merged by log-sum-exp.  Used to check "split + merge = unsplit". */
int oracle_xattn_split_merge(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t T, double scale,
                             const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                             const int32_t *cu, const int32_t *kv_len, int64_t kv_head_stride, int32_t window,
                             int32_t n_cuts, const int64_t *cuts, double *O, double *LSE)
{
    if (check_shape(B, Hq, Hkv, d, T) || n_cuts < 0 || window < 0) return -1;
    for (int k = 1; k < n_cuts; ++k)
        if (cuts[k] < cuts[k - 1]) return -1;
    problem_t p = {B, Hq, Hkv, d, T, resolve_scale(scale, d), Q, K, V, cu, kv_len, kv_head_stride, window};
    int64_t max_len = 1;
    for (int i = 0; i < B; ++i)
        if (kv_len[i] > max_len) max_len = kv_len[i];
    const int S = n_cuts + 1;
    double *scores = (double *)malloc(sizeof(double) * (size_t)max_len);
    double *po = (double *)malloc(sizeof(double) * (size_t)S * d);
    double *plse = (double *)malloc(sizeof(double) * (size_t)S);
    if (!scores || !po || !plse) {
        free(scores); free(po); free(plse);
        return -2;
    }
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hq; ++h)
            for (int t = 0; t < T; ++t) {
                int64_t n_vis = visible_keys(&p, i, t), n_lo = first_visible(&p, i, t);
                for (int s = 0; s < S; ++s) {
                    int64_t j0 = s == 0 ? 0 : cuts[s - 1];
                    int64_t j1 = s == n_cuts ? n_vis : cuts[s];
                    if (j0 < n_lo) j0 = n_lo;
                    if (j1 > n_vis) j1 = n_vis;
                    if (j0 > n_vis) j0 = n_vis;
                    row_over_range(&p, i, h, t, j0, j1, scores, po + (int64_t)s * d, plse + s);
                }
                int64_t row = ((int64_t)i * Hq + h) * T + t;
                merge_pieces(S, d, po, plse, O + row * d, LSE + row);
            }
    free(scores); free(po); free(plse);
    return 0;
}

/* Stand-alone merge of given partial results (fp32 as the GPU API takes them):
 * part_o [rows, S, d], part_lse [rows, S] (natural log, -inf = empty piece). */
int oracle_combine(int64_t rows, int32_t S, int32_t d, const float *part_o,
                   const float *part_lse, double *O, double *LSE)
{
    if (rows < 0 || S <= 0 || d <= 0) return -1;
    double *po = (double *)malloc(sizeof(double) * (size_t)S * d);
    double *plse = (double *)malloc(sizeof(double) * (size_t)S);
    if (!po || !plse) {
        free(po); free(plse);
        return -2;
    }
    for (int64_t r = 0; r < rows; ++r) {
        for (int s = 0; s < S; ++s) {
            plse[s] = (double)part_lse[r * S + s];
            for (int e = 0; e < d; ++e) po[(int64_t)s * d + e] = (double)part_o[(r * S + s) * d + e];
        }
        merge_pieces(S, d, po, plse, O + r * d, LSE + r);
    }
    free(po); free(plse);
    return 0;
}

/* The same definition over an 8-bit cache: K8, V8 hold E4M3 bytes in the packed head-major
 * layout (strides in elements as before), k_scale / v_scale one fp32 factor per KV head. */
int oracle_xattn_fp8(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t T, double scale,
                     const uint16_t *Q, const uint8_t *K8, const uint8_t *V8,
                     const float *k_scale, const float *v_scale,
                     const int32_t *cu, const int32_t *kv_len, int64_t kv_head_stride, int32_t window,
                     double *O, double *LSE)
{
    if (check_shape(B, Hq, Hkv, d, T) || window < 0) return -1;
    problem_t p = {B, Hq, Hkv, d, T, resolve_scale(scale, d), Q, NULL, NULL, cu, kv_len, kv_head_stride, window,
                   K8, V8, k_scale, v_scale};
    int64_t max_len = 1;
    for (int i = 0; i < B; ++i)
        if (kv_len[i] > max_len) max_len = kv_len[i];
    int failed = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)max_len);
        if (!scores) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int i = 0; i < B; ++i)
            for (int h = 0; h < Hq; ++h) {
                if (!scores) continue;
                for (int t = 0; t < T; ++t) {
                    int64_t row = ((int64_t)i * Hq + h) * T + t;
                    row_over_range(&p, i, h, t, first_visible(&p, i, t), visible_keys(&p, i, t), scores,
                                   O + row * d, LSE + row);
                }
            }
        free(scores);
    }
    return failed ? -2 : 0;
}

