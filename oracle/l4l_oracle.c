/*
 * CPU oracle for causal attention (prefill, decode) and the KV-cache copy.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT. It is a slow, plain restatement of
 * the definition of scaled-dot-product softmax attention in fp64, read from the same
 * bf16 inputs the GPU path gets. It shares no code with the CUDA kernels and must be
 * used only by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * What it follows. The paper (appendix, "Transformer attention") names the two
 * phase-specialised kernels but prints no formula: a prefill kernel for q_len > 1
 * that derives the KV head from the grouped-query structure and applies the causal
 * mask in the score update, and a decode kernel for q_len = 1 that serves one KV
 * head's whole query-head group from a populated cache. Both are exact
 * reformulations (online softmax, tiling) of ordinary softmax attention, so the
 * oracle is that definition written out:
 *
 *   s_j   = scale * sum_d q[d] * k_j[d]            (keys j = 0 .. n-1)
 *   p_j   = exp(s_j - max_j s_j)
 *   o[d]  = sum_j p_j * v_j[d] / sum_j p_j
 *   lse   = max_j s_j + log(sum_j p_j)
 *
 * Readings where the paper is silent (declared choices):
 *   - query head h uses KV head h / (Hq / Hkv) (consecutive query heads share a KV head);
 *   - prefill is causal with square alignment: query i sees keys 0..i of its sequence;
 *   - decode has no mask: the current token is already in the cache, the query sees
 *     all kv_len tokens;
 *   - n = 0 keys gives o = 0 and lse = -inf;
 *   - q, k, v are [B, S, H, D] token-major, the cache is [B, Hkv, Lmax, D]; all dense.
 *
 * No tiling, no online softmax, no reordering: one function, attend_row(), is the
 * definition; everything else is loops that call it or copy 16-bit words.
 * Parallelism is OpenMP over independent output rows only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE binary32; widening is exact. */
static double bf16_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int l4l_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Softmax attention of ONE query row over n keys (the definition above).
 *   q        : D bf16 values
 *   k, v     : row j at k + j*k_stride, v + j*v_stride (strides in elements), D values each
 *   p        : scratch of n doubles
 *   out      : D doubles;  lse : 1 double (may be NULL)
 */
static void attend_row(const uint16_t *q, const uint16_t *k, int64_t k_stride,
                       const uint16_t *v, int64_t v_stride, int n, int D,
                       double scale, double *p, double *out, double *lse)
{
    if (n <= 0) {
        for (int d = 0; d < D; ++d) out[d] = 0.0;
        if (lse) *lse = -INFINITY;
        return;
    }
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        double dot = 0.0;
        for (int d = 0; d < D; ++d)
            dot += bf16_to_f64(q[d]) * bf16_to_f64(k[(int64_t)j * k_stride + d]);
        p[j] = scale * dot;
        if (p[j] > m) m = p[j];
    }
    double l = 0.0;
    for (int j = 0; j < n; ++j) {
        p[j] = exp(p[j] - m);
        l += p[j];
    }
    for (int d = 0; d < D; ++d) {
        double acc = 0.0;
        for (int j = 0; j < n; ++j)
            acc += p[j] * bf16_to_f64(v[(int64_t)j * v_stride + d]);
        out[d] = acc / l;
    }
    if (lse) *lse = m + log(l);
}

/*
 * Causal prefill, every valid row.
 *   q        [B, S, Hq, D]  bf16 bits      k, v  [B, S, Hkv, D] bf16 bits
 *   seq_len  [B]            tokens per sequence (<= S)
 *   out      [B, S, Hq, D]  fp64; rows i >= seq_len[b] are left untouched
 *   lse      [B, Hq, S]     fp64 or NULL; same rule
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int l4l_oracle_prefill(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       const int32_t *seq_len, int B, int S, int Hq, int Hkv, int D,
                       double scale, double *out, double *lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    int fail = 0;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(S > 0 ? S : 1));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 8)
        for (int b = 0; b < B; ++b) {
            for (int i = 0; i < S; ++i) {
                if (!p || i >= seq_len[b]) continue;
                for (int h = 0; h < Hq; ++h) {
                    const int g = h / G;
                    const uint16_t *qrow = q + (((int64_t)b * S + i) * Hq + h) * D;
                    const uint16_t *kb = k + (((int64_t)b * S) * Hkv + g) * D;
                    const uint16_t *vb = v + (((int64_t)b * S) * Hkv + g) * D;
                    attend_row(qrow, kb, (int64_t)Hkv * D, vb, (int64_t)Hkv * D,
                               i + 1, D, scale, p,
                               out + (((int64_t)b * S + i) * Hq + h) * D,
                               lse ? lse + ((int64_t)b * Hq + h) * S + i : NULL);
                }
            }
        }
        free(p);
    }
    return fail ? -1 : 0;
}

/*
 * Causal prefill of a LIST of rows (for sizes where every row would take too long).
 *   rows     [n_rows, 3]    (b, i, h) triples, each with i < seq_len[b]
 *   out      [n_rows, D]    lse [n_rows] or NULL
 */
int l4l_oracle_prefill_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                            const int32_t *seq_len, int B, int S, int Hq, int Hkv, int D,
                            double scale, const int32_t *rows, int n_rows,
                            double *out, double *lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    int fail = 0;
    for (int r = 0; r < n_rows; ++r) {
        int b = rows[3 * r], i = rows[3 * r + 1], h = rows[3 * r + 2];
        if (b < 0 || b >= B || h < 0 || h >= Hq || i < 0 || i >= seq_len[b]) return -1;
    }
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(S > 0 ? S : 1));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_rows; ++r) {
            if (!p) continue;
            const int b = rows[3 * r], i = rows[3 * r + 1], h = rows[3 * r + 2];
            const int g = h / G;
            attend_row(q + (((int64_t)b * S + i) * Hq + h) * D,
                       k + (((int64_t)b * S) * Hkv + g) * D, (int64_t)Hkv * D,
                       v + (((int64_t)b * S) * Hkv + g) * D, (int64_t)Hkv * D,
                       i + 1, D, scale, p, out + (int64_t)r * D, lse ? lse + r : NULL);
        }
        free(p);
    }
    return fail ? -1 : 0;
}

/*
 * Prefill of a chunk of new tokens over a populated cache (q_len > 1 AND a populated cache, the regime
 * between the paper's two phases), bottom-right causal alignment: row i of the chunk is the token at
 * absolute position past[b] + i and sees cache slots 0 .. past[b] + i. The chunk's own K/V are expected in
 * the cache already (slots past[b] .. past[b] + q_len[b] - 1).
 *   q        [B, S, Hq, D]        cache_k, cache_v  [B, Hkv, Lmax, D]
 *   out      [B, S, Hq, D] fp64; rows i >= q_len[b] are left untouched     lse [B, Hq, S] or NULL
 */
int l4l_oracle_prefill_chunk(const uint16_t *q, const uint16_t *cache_k, const uint16_t *cache_v,
                             const int32_t *past, const int32_t *q_len, int B, int S, int Hq, int Hkv, int D,
                             int Lmax, double scale, double *out, double *lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    for (int b = 0; b < B; ++b)
        if (past[b] < 0 || q_len[b] < 0 || q_len[b] > S || past[b] + q_len[b] > Lmax) return -1;
    const int G = Hq / Hkv;
    int fail = 0;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(Lmax > 0 ? Lmax : 1));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 8)
        for (int b = 0; b < B; ++b) {
            for (int i = 0; i < S; ++i) {
                if (!p || i >= q_len[b]) continue;
                for (int h = 0; h < Hq; ++h) {
                    const int g = h / G;
                    const int64_t base = ((int64_t)b * Hkv + g) * Lmax * D;
                    attend_row(q + (((int64_t)b * S + i) * Hq + h) * D, cache_k + base, D, cache_v + base, D,
                               past[b] + i + 1, D, scale, p, out + (((int64_t)b * S + i) * Hq + h) * D,
                               lse ? lse + ((int64_t)b * Hq + h) * S + i : NULL);
                }
            }
        }
        free(p);
    }
    return fail ? -1 : 0;
}

/* Round an fp64 value to bf16: to nearest, ties to even; overflow goes to infinity, NaN stays NaN. */
static uint16_t f64_to_bf16(double x)
{
    float f;
    uint32_t u;
    if (x != x) return 0x7FC0;
    if (x != 0.0 && !isinf(x)) {
        int e;
        (void)frexp(fabs(x), &e);                                 /* |x| = m 2^e with 0.5 <= m < 1 */
        /* spacing of the bf16 values around |x|: 8 significant bits, subnormals below 2^-126 */
        const double quantum = ldexp(1.0, (e - 8 < -133) ? -133 : e - 8);
        const double r = nearbyint(fabs(x) / quantum) * quantum; /* ties to even (default rounding mode) */
        x = x < 0 ? -r : r;                                       /* now exactly a bf16 value, or 2^128 */
    }
    f = (float)x;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(u >> 16);
}

/* Exposed for the tests that pin the rounding against a library conversion. */
void l4l_oracle_round_bf16(const double *x, uint16_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = f64_to_bf16(x[i]);
}

/*
 * Rotary position embedding with optional per-head RMS normalisation, for ONE head row.
 * Half-split convention: element i < D/2 is paired with element i + D/2;
 *     y[i]       = x[i] cos_i - x[i + D/2] sin_i,     y[i + D/2] = x[i + D/2] cos_i + x[i] sin_i
 * and, before that, when w != NULL:  x[d] <- x[d] / sqrt(mean_d x[d]^2 + eps) * w[d].
 * Everything in fp64; `y` receives the unrounded result.
 */
static void rope_row(const uint16_t *x, int D, const float *cosr, const float *sinr, const float *w, double eps,
                     double *y)
{
    double xs[256];
    double ss = 0.0;
    for (int d = 0; d < D; ++d) {
        xs[d] = bf16_to_f64(x[d]);
        ss += xs[d] * xs[d];
    }
    if (w) {
        const double r = 1.0 / sqrt(ss / D + eps);
        for (int d = 0; d < D; ++d) xs[d] = xs[d] * r * (double)w[d];
    }
    const int H = D / 2;
    for (int i = 0; i < H; ++i) {
        const double c = (double)cosr[i], sn = (double)sinr[i];
        y[i] = xs[i] * c - xs[i + H] * sn;
        y[i + H] = xs[i + H] * c + xs[i] * sn;
    }
}

/*
 * Rotary embedding (+ optional RMS normalisation) of the new tokens' q and k, fused with the cache
 * update: token t < n_new[b] of sequence b sits at position P = pos[b] + t; its q rows are replaced
 * by their rotated values, its rotated k rows and its v rows (bit for bit) go to cache slot P.
 * Tokens with P outside [0, min(Lmax, n_pos)) are skipped.
 *   q [B,T,Hq,D] in/out (bf16 bits)   k_new, v_new [B,T,Hkv,D]   caches [B,Hkv,Lmax,D] in/out
 *   cos, sin [n_pos, D/2] fp32        q_w, k_w [D] fp32 or NULL
 *   q_exact [B,T,Hq,D], k_exact [B,T,Hkv,D]: the unrounded fp64 results (or NULL); skipped rows untouched
 */
int l4l_oracle_rope_kv_append(uint16_t *q, const uint16_t *k_new, const uint16_t *v_new, uint16_t *cache_k,
                              uint16_t *cache_v, const int32_t *pos, const int32_t *n_new, int B, int T, int Hq,
                              int Hkv, int D, int Lmax, const float *cosv, const float *sinv, int n_pos,
                              const float *q_w, const float *k_w, double eps, double *q_exact, double *k_exact)
{
    if (D <= 0 || D > 256 || (D & 1)) return -1;
    const int lim = Lmax < n_pos ? Lmax : n_pos;
    double y[256];
    for (int b = 0; b < B; ++b) {
        const int n = n_new ? n_new[b] : T;
        for (int t = 0; t < T && t < n; ++t) {
            const int64_t P = (int64_t)pos[b] + t;
            if (P < 0 || P >= lim) continue;
            const float *cr = cosv + P * (D / 2), *sr = sinv + P * (D / 2);
            for (int h = 0; h < Hq; ++h) {
                uint16_t *row = q + (((int64_t)b * T + t) * Hq + h) * D;
                rope_row(row, D, cr, sr, q_w, eps, y);
                for (int d = 0; d < D; ++d) {
                    row[d] = f64_to_bf16(y[d]);
                    if (q_exact) q_exact[(((int64_t)b * T + t) * Hq + h) * D + d] = y[d];
                }
            }
            for (int g = 0; g < Hkv; ++g) {
                const int64_t src = (((int64_t)b * T + t) * Hkv + g) * D;
                const int64_t dst = (((int64_t)b * Hkv + g) * Lmax + P) * D;
                rope_row(k_new + src, D, cr, sr, k_w, eps, y);
                for (int d = 0; d < D; ++d) {
                    cache_k[dst + d] = f64_to_bf16(y[d]);
                    if (k_exact) k_exact[src + d] = y[d];
                }
                memcpy(cache_v + dst, v_new + src, sizeof(uint16_t) * (size_t)D);
            }
        }
    }
    return 0;
}

/*
 * Decode: one query token per sequence over the populated cache (no mask).
 *   q        [B, Hq, D]           cache_k, cache_v  [B, Hkv, Lmax, D]
 *   kv_len   [B]   valid tokens, the current one included (<= Lmax)
 *   out      [B, Hq, D] fp64      lse [B, Hq] fp64 or NULL
 */
int l4l_oracle_decode(const uint16_t *q, const uint16_t *cache_k, const uint16_t *cache_v,
                      const int32_t *kv_len, int B, int Hq, int Hkv, int D, int Lmax,
                      double scale, double *out, double *lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    int fail = 0;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(Lmax > 0 ? Lmax : 1));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int b = 0; b < B; ++b) {
            for (int h = 0; h < Hq; ++h) {
                if (!p) continue;
                const int g = h / G;
                const int64_t base = ((int64_t)b * Hkv + g) * Lmax * D;
                attend_row(q + ((int64_t)b * Hq + h) * D, cache_k + base, D,
                           cache_v + base, D, kv_len[b], D, scale, p,
                           out + ((int64_t)b * Hq + h) * D,
                           lse ? lse + (int64_t)b * Hq + h : NULL);
            }
        }
        free(p);
    }
    return fail ? -1 : 0;
}

/* ------------------------------------------------------------------------------------------------
 * Second workload: the gated linear recurrence of the RecurrentGemma block (RG-LRU), which the paper's
 * appendix lists as an accepted kernel that fuses "sigmoid, softplus-derived recurrent gating, reset
 * handling, normalization, and the recurrent scan" with the state carried through the sequence and
 * the final state written once. The paper prints no formula; this is the published recurrence of that
 * block, per sequence b, channel c, step t (all in fp64 here):
 *     i_t = sigmoid(gate_x[b,t,c])                      input gate
 *     r_t = sigmoid(gate_a[b,t,c])                      recurrence gate
 *     log a_t = -8 * r_t * softplus(a_param[c])
 *     a_t = exp(log a_t),   m_t = sqrt(1 - a_t^2)       (m_t keeps the state's variance bounded)
 *     at a reset step (position[b,t] == 0):  a_t = 0, m_t = 1
 *     h_t = a_t * h_{t-1} + m_t * i_t * x[b,t,c]
 *     y[b,t,c] = h_t
 * x, gate_x, gate_a: bf16 bits [B, T, W]; a_param: fp32 [W]; position: int32 [B, T] or NULL (no resets);
 * state: fp64 [B, W] in/out (h before the first step / after step seq_len[b]-1); seq_len [B] or NULL (= T).
 * y: fp64 [B, T, W]; rows t >= seq_len[b] untouched.
 */
int l4l_oracle_rglru(const uint16_t *x, const uint16_t *gate_x, const uint16_t *gate_a, const float *a_param,
                     const int32_t *position, const int32_t *seq_len, double *state, double *y, int B, int T, int W)
{
    for (int b = 0; b < B; ++b) {
        const int L = seq_len ? seq_len[b] : T;
        if (L < 0 || L > T) return -1;
        for (int c = 0; c < W; ++c) {
            const double sp = log1p(exp((double)a_param[c]));        /* softplus */
            double h = state[(int64_t)b * W + c];
            for (int t = 0; t < L; ++t) {
                const int64_t idx = ((int64_t)b * T + t) * W + c;
                const double in_gate = 1.0 / (1.0 + exp(-bf16_to_f64(gate_x[idx])));
                const double rec_gate = 1.0 / (1.0 + exp(-bf16_to_f64(gate_a[idx])));
                double a = exp(-8.0 * rec_gate * sp);
                double m = sqrt(1.0 - a * a);
                if (position && position[(int64_t)b * T + t] == 0) {
                    a = 0.0;
                    m = 1.0;
                }
                h = a * h + m * in_gate * bf16_to_f64(x[idx]);
                y[idx] = h;
            }
            state[(int64_t)b * W + c] = h;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * fp8 (e4m3) cache. The format: 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is
 * subnormal (m/8 * 2^-6); there are no infinities; exponent 15 with mantissa 7 is NaN; the largest
 * finite value is 1.75 * 2^8 = 448.
 */
static double e4m3_to_f64(uint8_t c)
{
    const int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    v = (e == 0) ? ldexp((double)m / 8.0, -6) : ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* fp32 value -> e4m3: nearest, ties to even, saturating at +-448 (NaN -> 0x7F). Brute force over the 127
 * non-negative finite codes: the nearest one wins, a tie goes to the even code. */
static uint8_t f32_to_e4m3(float y)
{
    uint8_t best = 0;
    double bd = INFINITY;
    const double a = fabs((double)y);
    if (y != y) return 0x7F;
    for (int c = 0; c < 0x7F; ++c) {
        const double d = fabs(e4m3_to_f64((uint8_t)c) - a);
        if (d < bd || (d == bd && (c & 1) == 0)) { bd = d; best = (uint8_t)c; }
    }
    return (uint8_t)(best | (signbit(y) ? 0x80 : 0));
}

void l4l_oracle_e4m3_decode(const uint8_t *c, double *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = e4m3_to_f64(c[i]);
}

void l4l_oracle_e4m3_encode(const float *x, uint8_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_e4m3(x[i]);
}

/*
 * Cache update of an fp8 cache: slot write_pos[b] + t of (b, kv head g) receives the e4m3 code of
 * fp32(x) / scale[g], the division rounded to fp32 (the precision the decision is defined in), for the
 * new tokens' k and v. Out-of-range slots: error (the caller tests the drop rule separately).
 *   cache_k8, cache_v8 [B, Hkv, Lmax, D] bytes, in/out      k_new, v_new [B, T, Hkv, D] bf16 bits
 */
int l4l_oracle_kv_append_fp8(uint8_t *cache_k8, uint8_t *cache_v8, const uint16_t *k_new, const uint16_t *v_new,
                             const int32_t *pos, const int32_t *n_new, const float *k_scale, const float *v_scale,
                             int B, int T, int Hkv, int D, int Lmax)
{
    for (int b = 0; b < B; ++b) {
        const int n = n_new ? n_new[b] : T;
        for (int t = 0; t < n && t < T; ++t) {
            const int64_t slot = (int64_t)pos[b] + t;
            if (slot < 0 || slot >= Lmax) continue;
            for (int g = 0; g < Hkv; ++g)
                for (int d = 0; d < D; ++d) {
                    const int64_t src = (((int64_t)b * T + t) * Hkv + g) * D + d;
                    const int64_t dst = (((int64_t)b * Hkv + g) * Lmax + slot) * D + d;
                    const volatile float qk = (float)bf16_to_f64(k_new[src]) / k_scale[g];
                    const volatile float qv = (float)bf16_to_f64(v_new[src]) / v_scale[g];
                    cache_k8[dst] = f32_to_e4m3(qk);
                    cache_v8[dst] = f32_to_e4m3(qv);
                }
        }
    }
    return 0;
}

/*
 * Decode over an fp8 cache: the definition of attend_row() written out once more over the values the
 * bytes stand for, k_j[d] = e4m3(cache_k8[j][d]) * k_scale[g] (and the same for v), in fp64.
 */
int l4l_oracle_decode_fp8(const uint16_t *q, const uint8_t *cache_k8, const uint8_t *cache_v8, const int32_t *kv_len,
                          const float *k_scale, const float *v_scale, int B, int Hq, int Hkv, int D, int Lmax,
                          double scale, double *out, double *lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        if (kv_len[b] < 0 || kv_len[b] > Lmax) return -1;
    int fail = 0;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(Lmax > 0 ? Lmax : 1));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int b = 0; b < B; ++b) {
            for (int h = 0; h < Hq; ++h) {
                if (!p) continue;
                const int g = h / G, n = kv_len[b];
                const uint16_t *qr = q + ((int64_t)b * Hq + h) * D;
                const uint8_t *kb = cache_k8 + ((int64_t)b * Hkv + g) * Lmax * D;
                const uint8_t *vb = cache_v8 + ((int64_t)b * Hkv + g) * Lmax * D;
                double *o = out + ((int64_t)b * Hq + h) * D;
                const double ks = (double)k_scale[g], vs = (double)v_scale[g];
                if (n <= 0) {
                    for (int d = 0; d < D; ++d) o[d] = 0.0;
                    if (lse) lse[(int64_t)b * Hq + h] = -INFINITY;
                    continue;
                }
                double m = -INFINITY, l = 0.0;
                for (int j = 0; j < n; ++j) {
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += bf16_to_f64(qr[d]) * (e4m3_to_f64(kb[(int64_t)j * D + d]) * ks);
                    p[j] = scale * dot;
                    if (p[j] > m) m = p[j];
                }
                for (int j = 0; j < n; ++j) {
                    p[j] = exp(p[j] - m);
                    l += p[j];
                }
                for (int d = 0; d < D; ++d) {
                    double acc = 0.0;
                    for (int j = 0; j < n; ++j) acc += p[j] * (e4m3_to_f64(vb[(int64_t)j * D + d]) * vs);
                    o[d] = acc / l;
                }
                if (lse) lse[(int64_t)b * Hq + h] = m + log(l);
            }
        }
        free(p);
    }
    return fail ? -1 : 0;
}

/*
 * Cache copy. Writes n_new[b] tokens of k_new / v_new ([B, T, Hkv, D]) into the cache
 * ([B, Hkv, Lmax, D]) at slots pos[b] .. pos[b]+n_new[b]-1, as raw 16-bit words.
 * Everything else in the cache is left as it was. The prefill cache write is the case
 * pos = 0, n_new = seq_len; the decode-step append is the case T = 1, n_new = 1.
 * Returns -1 if a write would fall outside [0, Lmax).
 */
int l4l_oracle_kv_append(uint16_t *cache_k, uint16_t *cache_v, const uint16_t *k_new,
                         const uint16_t *v_new, const int32_t *pos, const int32_t *n_new,
                         int B, int T, int Hkv, int D, int Lmax)
{
    for (int b = 0; b < B; ++b)
        if (n_new[b] < 0 || n_new[b] > T || pos[b] < 0 || pos[b] + n_new[b] > Lmax) return -1;
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < n_new[b]; ++r)
            for (int g = 0; g < Hkv; ++g)
                for (int d = 0; d < D; ++d) {
                    const int64_t src = (((int64_t)b * T + r) * Hkv + g) * D + d;
                    const int64_t dst = (((int64_t)b * Hkv + g) * Lmax + pos[b] + r) * D + d;
                    cache_k[dst] = k_new[src];
                    cache_v[dst] = v_new[src];
                }
    return 0;
}
