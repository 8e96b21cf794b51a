/*
 * fp64 CPU oracle for the GTA (Grouped-head latenT Attention) operator.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * operator computes.  It shares no code, header, table or helper with the CUDA
 * library and is never on the product path: only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may build, load or call it.
 *
 * What it follows (paper section / equation):
 *   - grouping of Q, K and the latent C into n_q / n_k / n_c groups and the head
 *     maps q(i), k(i), c(i): Sec. 3.2 "Input projections and grouping";
 *   - value decoder  V_i = C_{c(i)} W_{P,i} (.) Sigmoid(x_t W_{G,i}): Sec. 3.2,
 *     the "Nonlinear value decoder" equation;
 *   - attention  Softmax(Q K^T / sqrt(d_h)) V_i  and its inference
 *     reformulation (Softmax(.) C W_P) (.) Sigmoid(x_t W_G): Sec. 3.3;
 *   - the token-level causal form, sum over k = 1..t inclusive: App. B.1.1;
 *   - decode over cached keys / latents, cache = (n_k d_h + n_c d_l) N: App. B.1.3.
 *
 * Readings taken where the paper leaves a choice (all listed in the design notes):
 *   - head maps are contiguous blocks: q(i) = floor(i n_q / n_h),
 *     k(i) = floor(q(i) n_k / n_q), c(i) = floor(q(i) n_c / n_q);
 *   - the gate uses the hidden state of the QUERY token of the output row and is
 *     passed through a sigmoid (main text); the appendix drops the sigmoid;
 *   - the causal sum includes the diagonal;
 *   - the output projection W_O and RoPE are outside the operator.
 *
 * Everything is computed in double.  Inputs may be stored as fp32, bf16 (raw
 * 16-bit patterns) or fp64 and are widened exactly, element by element.
 * Layouts (row-major, innermost last):
 *   q   [B, n_q, N, d_h]     k [B, n_k, N, d_h]     c [B, n_c, N, d_l]
 *   x   [B, N, H]            w_p [n_h, d_l, d_h]    w_g [H, n_h*d_h]
 *   out [B, R, n_h, d_h]  (R = N, or the number of sampled rows)
 *
 * Parity pins (tests, CPU only): reduction to textbook multi-head attention,
 * rows of the softmax sum to one, causality, decode == last prefill row,
 * brute force against an independent einsum restatement, equality of the
 * definition form and the reformulated form, uniform-attention and one-hot
 * closed forms, head sharing inside a group, batch independence.  The paper
 * prints no worked numeric example, so absolute values have no printed pin.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { GTA_ORACLE_F32 = 0, GTA_ORACLE_BF16 = 1, GTA_ORACLE_F64 = 2 };

typedef struct {
    int32_t batch;      /* B   */
    int32_t seq;        /* N   (prefill) */
    int32_t d_model;    /* H   */
    int32_t n_heads;    /* n_h */
    int32_t n_q;        /* query / attention-map groups */
    int32_t n_k;        /* key groups    */
    int32_t n_c;        /* latent groups */
    int32_t d_h;        /* head dim      */
    int32_t d_l;        /* latent dim    */
    int32_t causal;     /* 1: keys j <= t only; 0: all keys */
    double  scale;      /* 0 => 1/sqrt(d_h) */
} gta_oracle_shape;

/* ---- exact widening of one stored element to double ---- */
static double load_elem(const void *p, int dtype, size_t i)
{
    if (dtype == GTA_ORACLE_F32) return (double)((const float *)p)[i];
    if (dtype == GTA_ORACLE_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)p)[i] << 16; /* bf16 = top half of fp32 */
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return ((const double *)p)[i];
}

static double *widen(const void *p, int dtype, size_t n)
{
    double *d = (double *)malloc((n ? n : 1) * sizeof(double));
    if (!d) return NULL;
    for (size_t i = 0; i < n; ++i) d[i] = load_elem(p, dtype, i);
    return d;
}

static int head_to_q(const gta_oracle_shape *s, int i) { return (int)(((long)i * s->n_q) / s->n_heads); }
static int q_to_k(const gta_oracle_shape *s, int g)    { return (int)(((long)g * s->n_k) / s->n_q); }
static int q_to_c(const gta_oracle_shape *s, int g)    { return (int)(((long)g * s->n_c) / s->n_q); }

static double softmax_scale(const gta_oracle_shape *s)
{
    return s->scale != 0.0 ? s->scale : 1.0 / sqrt((double)s->d_h);
}

static int shape_ok(const gta_oracle_shape *s)
{
    if (s->batch < 0 || s->seq < 0 || s->d_model < 1 || s->n_heads < 1 || s->n_q < 1 ||
        s->n_k < 1 || s->n_c < 1 || s->d_h < 1 || s->d_l < 1) return 0;
    if (s->n_heads % s->n_q || s->n_q % s->n_k || s->n_q % s->n_c) return 0;
    return 1;
}

/*
 * Softmax probabilities of one query vector against n_keys keys (Sec. 3.3):
 *   p_j = exp(s_j - max) / sum_j exp(s_j - max),  s_j = scale * <qv, K_j>.
 */
static void softmax_row(const double *qv, const double *keys, int n_keys, int d_h,
                        double scale, double *p)
{
    double m = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
        double dot = 0.0;
        for (int d = 0; d < d_h; ++d) dot += qv[d] * keys[(size_t)j * d_h + d];
        p[j] = scale * dot;
        if (p[j] > m) m = p[j];
    }
    double sum = 0.0;
    for (int j = 0; j < n_keys; ++j) { p[j] = exp(p[j] - m); sum += p[j]; }
    for (int j = 0; j < n_keys; ++j) p[j] /= sum;
}

/* gate_e = Sigmoid( sum_h x[h] * W_G[h, col0 + e] )   (Sec. 3.2, decoder equation) */
static void gate_row(const double *xrow, const double *w_g, int H, int w_g_cols, int col0,
                     int d_h, double *gate)
{
    for (int e = 0; e < d_h; ++e) gate[e] = 0.0;
    for (int h = 0; h < H; ++h) {
        const double xv = xrow[h];
        const double *wrow = w_g + (size_t)h * w_g_cols + col0;
        for (int e = 0; e < d_h; ++e) gate[e] += xv * wrow[e];
    }
    for (int e = 0; e < d_h; ++e) gate[e] = 1.0 / (1.0 + exp(-gate[e]));
}

/*
 * One output row of one head in the REFORMULATED form (Sec. 3.3, second equation):
 *   o_lat = sum_j p_j C_j ;  out = (o_lat W_{P,i}) (.) gate
 */
static void head_row_reformulated(const double *qv, const double *keys, const double *lat,
                                  int n_keys, int d_h, int d_l, double scale,
                                  const double *xrow, const double *w_p_i, const double *w_g,
                                  int H, int w_g_cols, int col0,
                                  double *p, double *o_lat, double *gate, double *out)
{
    if (n_keys <= 0) { for (int e = 0; e < d_h; ++e) out[e] = 0.0; return; }
    softmax_row(qv, keys, n_keys, d_h, scale, p);
    for (int l = 0; l < d_l; ++l) o_lat[l] = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        const double pj = p[j];
        const double *cj = lat + (size_t)j * d_l;
        for (int l = 0; l < d_l; ++l) o_lat[l] += pj * cj[l];
    }
    gate_row(xrow, w_g, H, w_g_cols, col0, d_h, gate);
    for (int e = 0; e < d_h; ++e) out[e] = 0.0;
    for (int l = 0; l < d_l; ++l) {
        const double ol = o_lat[l];
        const double *wrow = w_p_i + (size_t)l * d_h;
        for (int e = 0; e < d_h; ++e) out[e] += ol * wrow[e];
    }
    for (int e = 0; e < d_h; ++e) out[e] *= gate[e];
}

/*
 * One output row of one head in the DEFINITION form (decoder equation of Sec. 3.2
 * followed by the first equation of Sec. 3.3): the gated value matrix
 *   V^{(t)}[j, e] = (sum_l C[j, l] W_P[l, e]) * gate_t[e]
 * is materialised for every key j and then averaged with the probabilities.
 */
static void head_row_definition(const double *qv, const double *keys, const double *lat,
                                int n_keys, int d_h, int d_l, double scale,
                                const double *xrow, const double *w_p_i, const double *w_g,
                                int H, int w_g_cols, int col0,
                                double *p, double *vmat, double *gate, double *out)
{
    if (n_keys <= 0) { for (int e = 0; e < d_h; ++e) out[e] = 0.0; return; }
    gate_row(xrow, w_g, H, w_g_cols, col0, d_h, gate);
    for (int j = 0; j < n_keys; ++j) {
        for (int e = 0; e < d_h; ++e) {
            double v = 0.0;
            for (int l = 0; l < d_l; ++l) v += lat[(size_t)j * d_l + l] * w_p_i[(size_t)l * d_h + e];
            vmat[(size_t)j * d_h + e] = v * gate[e];
        }
    }
    softmax_row(qv, keys, n_keys, d_h, scale, p);
    for (int e = 0; e < d_h; ++e) {
        double acc = 0.0;
        for (int j = 0; j < n_keys; ++j) acc += p[j] * vmat[(size_t)j * d_h + e];
        out[e] = acc;
    }
}

static int prefill_impl(const gta_oracle_shape *s, int dtype, const void *q, const void *k,
                        const void *c, const void *x, const void *w_p, const void *w_g,
                        const int32_t *rows, int n_rows, double *out, int n_threads,
                        int definition_form)
{
    if (!shape_ok(s) || !out) return 1;
    const int B = s->batch, N = s->seq, H = s->d_model, nh = s->n_heads;
    const int dh = s->d_h, dl = s->d_l;
    const int R = rows ? n_rows : N;
    if (B == 0 || N == 0 || R == 0) return 0;
    for (int r = 0; rows && r < n_rows; ++r) if (rows[r] < 0 || rows[r] >= N) return 1;

    double *Q = widen(q, dtype, (size_t)B * s->n_q * N * dh);
    double *K = widen(k, dtype, (size_t)B * s->n_k * N * dh);
    double *C = widen(c, dtype, (size_t)B * s->n_c * N * dl);
    double *X = widen(x, dtype, (size_t)B * N * H);
    double *WP = widen(w_p, dtype, (size_t)nh * dl * dh);
    double *WG = widen(w_g, dtype, (size_t)H * nh * dh);
    int rc = (Q && K && C && X && WP && WG) ? 0 : 2;
    const double scale = softmax_scale(s);
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
    if (rc == 0) {
        const long work = (long)B * R * nh;
        int failed = 0;
#pragma omp parallel
        {
            double *p = (double *)malloc((size_t)N * sizeof(double));
            double *tmp = (double *)malloc((definition_form ? (size_t)N * dh : (size_t)dl) * sizeof(double));
            double *gate = (double *)malloc((size_t)dh * sizeof(double));
            const int have_scratch = p && tmp && gate;
            if (!have_scratch) {
#pragma omp atomic write
                failed = 1;
            }
#pragma omp for schedule(dynamic, 4)
            for (long w = 0; w < work; ++w) {
                if (!have_scratch) continue;
                const int i = (int)(w % nh);
                const int r = (int)((w / nh) % R);
                const int b = (int)(w / ((long)nh * R));
                const int t = rows ? rows[r] : r;
                const int g = head_to_q(s, i), kg = q_to_k(s, g), cg = q_to_c(s, g);
                const int n_keys = s->causal ? t + 1 : N;
                const double *qv = Q + (((size_t)b * s->n_q + g) * N + t) * dh;
                const double *keys = K + ((size_t)b * s->n_k + kg) * N * dh;
                const double *lat = C + ((size_t)b * s->n_c + cg) * N * dl;
                const double *xrow = X + ((size_t)b * N + t) * H;
                const double *wpi = WP + (size_t)i * dl * dh;
                double *o = out + (((size_t)b * R + r) * nh + i) * dh;
                if (definition_form)
                    head_row_definition(qv, keys, lat, n_keys, dh, dl, scale, xrow, wpi, WG, H,
                                        nh * dh, i * dh, p, tmp, gate, o);
                else
                    head_row_reformulated(qv, keys, lat, n_keys, dh, dl, scale, xrow, wpi, WG, H,
                                          nh * dh, i * dh, p, tmp, gate, o);
            }
            free(p); free(tmp); free(gate);
        }
        if (failed) rc = 2;
    }
    free(Q); free(K); free(C); free(X); free(WP); free(WG);
    return rc;
}

/*
 * Causal (or full) prefill, reformulated form.  rows == NULL: every row, out is
 * [B, N, n_h, d_h]; otherwise only the n_rows listed positions, out is
 * [B, n_rows, n_h, d_h].  Returns 0 on success.
 */
int gta_oracle_prefill(const gta_oracle_shape *s, int dtype, const void *q, const void *k,
                       const void *c, const void *x, const void *w_p, const void *w_g,
                       const int32_t *rows, int n_rows, double *out, int n_threads)
{
    return prefill_impl(s, dtype, q, k, c, x, w_p, w_g, rows, n_rows, out, n_threads, 0);
}

/* Same result through the definition form (gated V materialised per query row). */
int gta_oracle_prefill_definition(const gta_oracle_shape *s, int dtype, const void *q,
                                  const void *k, const void *c, const void *x, const void *w_p,
                                  const void *w_g, const int32_t *rows, int n_rows, double *out,
                                  int n_threads)
{
    return prefill_impl(s, dtype, q, k, c, x, w_p, w_g, rows, n_rows, out, n_threads, 1);
}

/*
 * Attention probabilities of every query group: probs [B, n_q, N, N], entries with
 * j > t are 0 when causal.  For small shapes (row-sum and causality checks).
 */
int gta_oracle_probs(const gta_oracle_shape *s, int dtype, const void *q, const void *k,
                     double *probs)
{
    if (!shape_ok(s) || !probs) return 1;
    const int B = s->batch, N = s->seq, dh = s->d_h;
    double *Q = widen(q, dtype, (size_t)B * s->n_q * N * dh);
    double *K = widen(k, dtype, (size_t)B * s->n_k * N * dh);
    if (!Q || !K) { free(Q); free(K); return 2; }
    const double scale = softmax_scale(s);
    for (int b = 0; b < B; ++b)
        for (int g = 0; g < s->n_q; ++g)
            for (int t = 0; t < N; ++t) {
                const int n_keys = s->causal ? t + 1 : N;
                double *row = probs + (((size_t)b * s->n_q + g) * N + t) * N;
                for (int j = 0; j < N; ++j) row[j] = 0.0;
                softmax_row(Q + (((size_t)b * s->n_q + g) * N + t) * dh,
                            K + ((size_t)b * s->n_k + q_to_k(s, g)) * N * dh, n_keys, dh, scale, row);
            }
    free(Q); free(K);
    return 0;
}

/*
 * One decode step (App. B.1.3): sequence b's new token, whose key and latent are
 * already the last of seq_lens[b] cached entries, attends every cached entry.
 *   q [B, n_q, d_h]   k_cache [B, n_k, S_cap, d_h]   c_cache [B, n_c, S_cap, d_l]
 *   x_t [B, H]        out [B, n_h, d_h]              seq_lens [B] (includes the new token)
 * A sequence with seq_lens[b] == 0 yields zeros.
 */
int gta_oracle_decode(const gta_oracle_shape *s, int dtype, const void *q, const void *k_cache,
                      const void *c_cache, const int32_t *seq_lens, int S_cap, const void *x_t,
                      const void *w_p, const void *w_g, double *out, int n_threads)
{
    if (!shape_ok(s) || !out || !seq_lens || S_cap < 0) return 1;
    const int B = s->batch, H = s->d_model, nh = s->n_heads, dh = s->d_h, dl = s->d_l;
    for (int b = 0; b < B; ++b) if (seq_lens[b] < 0 || seq_lens[b] > S_cap) return 1;
    if (B == 0) return 0;
    double *Q = widen(q, dtype, (size_t)B * s->n_q * dh);
    double *X = widen(x_t, dtype, (size_t)B * H);
    double *WP = widen(w_p, dtype, (size_t)nh * dl * dh);
    double *WG = widen(w_g, dtype, (size_t)H * nh * dh);
    int rc = (Q && X && WP && WG) ? 0 : 2;
    const double scale = softmax_scale(s);
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
    if (rc == 0) {
        int failed = 0;
        const long work = (long)B * nh;
#pragma omp parallel for schedule(dynamic, 1)
        for (long w = 0; w < work; ++w) {
            const int i = (int)(w % nh), b = (int)(w / nh);
            const int len = seq_lens[b];
            const int g = head_to_q(s, i), kg = q_to_k(s, g), cg = q_to_c(s, g);
            const size_t k_off = ((size_t)b * s->n_k + kg) * S_cap * dh;
            const size_t c_off = ((size_t)b * s->n_c + cg) * S_cap * dl;
            double *keys = (double *)malloc(((size_t)len * dh + 1) * sizeof(double));
            double *lat = (double *)malloc(((size_t)len * dl + 1) * sizeof(double));
            double *p = (double *)malloc(((size_t)len + 1) * sizeof(double));
            double *o_lat = (double *)malloc((size_t)dl * sizeof(double));
            double *gate = (double *)malloc((size_t)dh * sizeof(double));
            if (!keys || !lat || !p || !o_lat || !gate) {
#pragma omp atomic write
                failed = 1;
            } else {
                for (size_t e = 0; e < (size_t)len * dh; ++e) keys[e] = load_elem(k_cache, dtype, k_off + e);
                for (size_t e = 0; e < (size_t)len * dl; ++e) lat[e] = load_elem(c_cache, dtype, c_off + e);
                head_row_reformulated(Q + ((size_t)b * s->n_q + g) * dh, keys, lat, len, dh, dl, scale,
                                      X + (size_t)b * H, WP + (size_t)i * dl * dh, WG, H, nh * dh,
                                      i * dh, p, o_lat, gate, out + ((size_t)b * nh + i) * dh);
            }
            free(keys); free(lat); free(p); free(o_lat); free(gate);
        }
        if (failed) rc = 2;
    }
    free(Q); free(X); free(WP); free(WG);
    return rc;
}

/*
 * Cache append (Sec. 3.3 / App. B.1.3: the caches hold K and C of every past token).
 * Byte copy, no arithmetic:  for each sequence b with len_b + n_new <= S_cap,
 *   k_cache[b, :, len_b + n, :] = k_new[b, :, n, :]   (n = 0..n_new-1), likewise c,
 *   then len_b += n_new.
 * A sequence that would overflow is left untouched (cache and length) and
 * *overflowed is set to 1.  elem_size is the storage size of one element in bytes.
 *   k_new [B, n_k, n_new, d_h]   c_new [B, n_c, n_new, d_l]
 */
int gta_oracle_cache_append(const gta_oracle_shape *s, int elem_size, void *k_cache, void *c_cache,
                            int S_cap, const void *k_new, const void *c_new, int n_new,
                            int32_t *seq_lens, int32_t *overflowed)
{
    if (!shape_ok(s) || elem_size < 1 || S_cap < 0 || n_new < 0 || !seq_lens) return 1;
    const size_t krow = (size_t)s->d_h * elem_size, crow = (size_t)s->d_l * elem_size;
    if (overflowed) *overflowed = 0;
    for (int b = 0; b < s->batch; ++b) {
        const int len = seq_lens[b];
        if (len < 0 || len + n_new > S_cap) { if (overflowed) *overflowed = 1; continue; }
        for (int g = 0; g < s->n_k; ++g)
            for (int n = 0; n < n_new; ++n)
                memcpy((char *)k_cache + (((size_t)b * s->n_k + g) * S_cap + len + n) * krow,
                       (const char *)k_new + (((size_t)b * s->n_k + g) * n_new + n) * krow, krow);
        for (int g = 0; g < s->n_c; ++g)
            for (int n = 0; n < n_new; ++n)
                memcpy((char *)c_cache + (((size_t)b * s->n_c + g) * S_cap + len + n) * crow,
                       (const char *)c_new + (((size_t)b * s->n_c + g) * n_new + n) * crow, crow);
        seq_lens[b] = len + n_new;
    }
    return 0;
}

/*
 * Closed-form costs of Table 3 (GTA row) and App. B.1.2 / B.1.3, in the paper's
 * units (multiply-accumulate counts and cache elements, no factor 2):
 *   attention  n_q (d_h + d_l) N^2        cache  (n_k d_h + n_c d_l) N
 */
double gta_oracle_attention_cost(const gta_oracle_shape *s)
{
    return (double)s->n_q * ((double)s->d_h + s->d_l) * (double)s->seq * (double)s->seq;
}

double gta_oracle_cache_elems(const gta_oracle_shape *s)
{
    return ((double)s->n_k * s->d_h + (double)s->n_c * s->d_l) * (double)s->seq;
}

int gta_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
