/*
 * fp64 CPU oracle for one decode step of Grouped Value Attention with decoupled RoPE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition the CUDA library is checked
 * against.  It is deliberately slow and unblocked: two-pass softmax, no tiling, no split-KV, pages
 * resolved by direct indexing.  It shares no code, header, table or constant with the CUDA path and
 * must never be called from it.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may load it.
 *
 * Notation follows the paper (row vectors).  d_v = value width (paper d_h), d_c = content-key
 * width (paper d_n), d_r = RoPE width, g(h) = h / (H/G).
 *
 *   rope      : x R_p^T with R_p block-diagonal 2x2 rotations, angle p * base^(-2i/d_r)
 *               (Section 3.3, Eq. krope; the pairing/frequency convention is this build's reading)
 *   absorb    : q~_h = q_h^nope M_h^T                     (Section 3.2, Eq. absorb; Algorithm 1)
 *   append    : V_{1:t,g} <- [V_{1:t-1,g}; v_{t,g}],  k^rope_t = (.)R_t^T appended   (Algorithm 1)
 *   decode    : s_j = q~_h v_{j,g(h)}^T + q^rope_h (k^rope_j)^T ;  o_h = softmax(s/sqrt(d_qk)) V_{g(h)}
 *               with d_qk = d_c + d_r                     (Section 3.3 score equation; Algorithm 1)
 *   gqa       : matched GQA decode over cached K and V    (Section 2, GQA; Section 3.4)
 *   prefill   : ordinary causal attention whose scores are the content term plus the positional term, keys formed explicitly:
 *               K_h = V_g(h) M_h (Eq. kvm), k_j = [K_h,j ; k^rope_j], q_i = [q^nope_i ; q^rope_i R_i^T]
 *               (Section 3.3; the sentence after Algorithm 1 on training / multi-token attention)
 *
 * All arithmetic is double precision.  Cache pools are read in their storage type (bf16 bit
 * patterns or float32) and widened exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_E4M3 2   /* 8-bit float: 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinity, 0x7F / 0xFF = NaN, largest finite 448 */

/* ---- storage <-> double ---------------------------------------------------------------------- */
/* value of an e4m3 code, exactly */
double oracle_e4m3_to_double(uint8_t c) {
    int e = (c >> 3) & 15, m = c & 7;
    double v;
    if ((c & 0x7F) == 0x7F) return NAN;
    v = e == 0 ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return (c & 0x80) ? -v : v;
}

static double load_elem(const void *pool, int dtype, int64_t idx) {
    if (dtype == ORACLE_E4M3) return oracle_e4m3_to_double(((const uint8_t *)pool)[idx]);
    if (dtype == ORACLE_BF16) {
        uint32_t u = ((uint32_t)((const uint16_t *)pool)[idx]) << 16;
        float f;
        memcpy(&f, &u, 4);
        return (double)f;
    }
    return (double)((const float *)pool)[idx];
}

/* Round a double to bfloat16, nearest with ties to even, straight from the fp64 value (no
 * intermediate float rounding).  Works on the value, not on bit tricks shared with anyone:
 * scale into [2^7, 2^8) so that the 8 significant bits of bf16 are the integer part, round the
 * integer with nearbyint (default rounding mode = ties-to-even), scale back (exact). */
uint16_t oracle_bf16_from_double(double x) {
    if (x != x) return 0x7FC0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80);
    int e;
    (void)frexp(a, &e);        /* a = m * 2^e, m in [0.5, 1)  => a in [2^(e-1), 2^e) */
    int exp_unb = e - 1;        /* floor(log2 a) */
    if (exp_unb < -126) exp_unb = -126;   /* subnormal bf16: fixed quantum 2^-133 */
    double q = ldexp(a, 7 - exp_unb);     /* in [128, 256) for normals */
    double r = nearbyint(q);              /* ties-to-even */
    double y = ldexp(r, exp_unb - 7);     /* exact */
    if (y >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80); /* rounded past the largest finite bf16 */
    float f = (float)y;                   /* exact: y has at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* Round a double to e4m3, nearest with ties to even, straight from the fp64 value; magnitudes beyond the largest finite
 * value 448 saturate to it (there is no infinity to round to), NaN stays NaN.  Same construction as above: scale so
 * that the representable numbers near |x| are the integers (quantum 2^(e-3) for |x| in [2^e, 2^(e+1)), fixed quantum
 * 2^-9 below the smallest normal 2^-6), round with nearbyint, scale back, then read off exponent and mantissa. */
uint8_t oracle_e4m3_from_double(double x) {
    if (x != x) return 0x7F;
    uint8_t sign = signbit(x) ? 0x80 : 0;
    double a = fabs(x);
    if (a > 448.0) return (uint8_t)(sign | 0x7E);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);
    int exp_unb = e - 1;                       /* floor(log2 a) */
    if (exp_unb < -6) exp_unb = -6;            /* subnormal range: quantum 2^-9 */
    double r = nearbyint(ldexp(a, 3 - exp_unb));   /* in [8, 16] for normals, [0, 8] for subnormals */
    double y = ldexp(r, exp_unb - 3);          /* exact */
    if (y == 0.0) return sign;
    if (y < ldexp(1.0, -6)) return (uint8_t)(sign | (uint8_t)r);          /* subnormal: mantissa = r */
    (void)frexp(y, &e);
    exp_unb = e - 1;                           /* rounding may have carried into the next binade */
    int m = (int)(ldexp(y, 3 - exp_unb) - 8.0);
    return (uint8_t)(sign | ((exp_unb + 7) << 3) | m);
}

static void store_elem(void *pool, int dtype, int64_t idx, double x) {
    if (dtype == ORACLE_E4M3)
        ((uint8_t *)pool)[idx] = oracle_e4m3_from_double(x);
    else if (dtype == ORACLE_BF16)
        ((uint16_t *)pool)[idx] = oracle_bf16_from_double(x);
    else
        ((float *)pool)[idx] = (float)x;  /* IEEE nearest-even conversion */
}

/* ---- RoPE: y = x R_p^T, pairs (2i, 2i+1), theta_i = base^(-2i/d_r) ---------------------------- */
void oracle_rope(const double *x, int d_r, double pos, double base, double *y) {
    for (int i = 0; i < d_r / 2; ++i) {
        double theta = pow(base, -2.0 * (double)i / (double)d_r);
        double a = pos * theta;
        double c = cos(a), s = sin(a);
        double x0 = x[2 * i], x1 = x[2 * i + 1];
        y[2 * i] = x0 * c - x1 * s;
        y[2 * i + 1] = x0 * s + x1 * c;
    }
}

/* ---- absorb: q_abs[b,h,0:d_v] = q_c[b,h,:] M_h^T ; q_abs[b,h,d_v:] = rope(q_r[b,h,:], q_pos[b]) --
 * M is [H][d_v][d_c] row-major (M_h in R^{d_h x d_n}), so (q M_h^T)[i] = sum_j q[j] M_h[i][j].   */
void oracle_absorb(const double *q_c, const double *q_r, const double *M, const int32_t *q_pos,
                   int B, int H, int d_v, int d_c, int d_r, double base, double *q_abs) {
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *dst = q_abs + ((int64_t)b * H + h) * (d_v + d_r);
            const double *q = q_c + ((int64_t)b * H + h) * d_c;
            const double *Mh = M + (int64_t)h * d_v * d_c;
            for (int i = 0; i < d_v; ++i) {
                double acc = 0.0;
                for (int j = 0; j < d_c; ++j) acc += q[j] * Mh[(int64_t)i * d_c + j];
                dst[i] = acc;
            }
            oracle_rope(q_r + ((int64_t)b * H + h) * d_r, d_r, (double)q_pos[b], base, dst + d_v);
        }
}

/* physical page of logical page j of sequence b; block_table == NULL means contiguous */
static int64_t page_of(const int32_t *block_table, int max_pages, int b, int j) {
    return block_table ? (int64_t)block_table[(int64_t)b * max_pages + j] : (int64_t)b * max_pages + j;
}

/* ---- append: write the new token's G value rows and its rotated positional key -----------------
 * v_pool [num_pages][G][P][d_v], kr_pool [num_pages][P][d_r].  v_new [B][G][d_v], kr_new [B][d_r]
 * (unrotated), pos [B].  Returns 0, or 1+b for the first sequence whose position lies outside its block table or whose page id is out of range
 * (that sequence and the ones after it are not written). */
int oracle_append(void *v_pool, void *kr_pool, int dtype, const int32_t *block_table, int num_pages,
                  int max_pages, int P, int G, int d_v, int d_r, double base, const double *v_new,
                  const double *kr_new, const int32_t *pos, int B) {
    double *rot = (double *)malloc(sizeof(double) * (size_t)d_r);
    int rc = 0;
    for (int b = 0; b < B && !rc; ++b) {
        int t = pos[b];
        if (t < 0 || t / P >= max_pages) { rc = 1 + b; break; }   /* position outside the block table: no lookup */
        int64_t page = page_of(block_table, max_pages, b, t / P);
        int slot = t % P;
        if (page < 0 || page >= num_pages) { rc = 1 + b; break; }
        for (int g = 0; g < G; ++g)
            for (int i = 0; i < d_v; ++i)
                store_elem(v_pool, dtype, ((page * G + g) * P + slot) * d_v + i,
                           v_new[((int64_t)b * G + g) * d_v + i]);
        oracle_rope(kr_new + (int64_t)b * d_r, d_r, (double)t, base, rot);
        for (int k = 0; k < d_r; ++k) store_elem(kr_pool, dtype, (page * P + slot) * d_r + k, rot[k]);
    }
    free(rot);
    return rc;
}

/* ---- decode: plain two-pass softmax attention over the paged GVA cache ---------------------------
 * q_abs [B][H][d_v+d_r] (absorbed content query, then rotated positional query), out [B][H][d_v],
 * lse [B][H] = log sum_j exp(scale * s_j).  seq_len == 0 gives out = 0, lse = -inf.            */
void oracle_decode(const void *v_pool, const void *kr_pool, int dtype, const int32_t *block_table,
                   int max_pages, int P, const int32_t *seq_lens, const double *q_abs, double scale,
                   int B, int H, int G, int d_v, int d_r, double *out, double *lse) {
    int hpg = H / G;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            int g = h / hpg;
            int T = seq_lens[b];
            const double *q = q_abs + ((int64_t)b * H + h) * (d_v + d_r);
            double *o = out + ((int64_t)b * H + h) * d_v;
            for (int i = 0; i < d_v; ++i) o[i] = 0.0;
            if (T <= 0) { if (lse) lse[(int64_t)b * H + h] = -INFINITY; continue; }
            double *s = (double *)malloc(sizeof(double) * (size_t)T);
            double m = -INFINITY;
            for (int t = 0; t < T; ++t) {
                int64_t page = page_of(block_table, max_pages, b, t / P);
                int slot = t % P;
                int64_t vrow = ((page * G + g) * P + slot) * d_v;
                int64_t krow = (page * P + slot) * d_r;
                double acc = 0.0;
                for (int i = 0; i < d_v; ++i) acc += q[i] * load_elem(v_pool, dtype, vrow + i);
                for (int k = 0; k < d_r; ++k) acc += q[d_v + k] * load_elem(kr_pool, dtype, krow + k);
                s[t] = acc * scale;
                if (s[t] > m) m = s[t];
            }
            double L = 0.0;
            for (int t = 0; t < T; ++t) { s[t] = exp(s[t] - m); L += s[t]; }
            for (int t = 0; t < T; ++t) {
                int64_t page = page_of(block_table, max_pages, b, t / P);
                int slot = t % P;
                int64_t vrow = ((page * G + g) * P + slot) * d_v;
                double p = s[t] / L;
                for (int i = 0; i < d_v; ++i) o[i] += p * load_elem(v_pool, dtype, vrow + i);
            }
            if (lse) lse[(int64_t)b * H + h] = m + log(L);
            free(s);
        }
}

/* ---- softmax weights of one (b, h) row, for invariant checks (sum to one, flat case) ------------- */
void oracle_decode_weights(const void *v_pool, const void *kr_pool, int dtype, const int32_t *block_table,
                           int max_pages, int P, const int32_t *seq_lens, const double *q_abs, double scale,
                           int H, int G, int d_v, int d_r, int b, int h, double *p) {
    int g = h / (H / G);
    int T = seq_lens[b];
    const double *q = q_abs + ((int64_t)b * H + h) * (d_v + d_r);
    double m = -INFINITY;
    for (int t = 0; t < T; ++t) {
        int64_t page = page_of(block_table, max_pages, b, t / P);
        int slot = t % P;
        double acc = 0.0;
        for (int i = 0; i < d_v; ++i) acc += q[i] * load_elem(v_pool, dtype, ((page * G + g) * P + slot) * d_v + i);
        for (int k = 0; k < d_r; ++k) acc += q[d_v + k] * load_elem(kr_pool, dtype, (page * P + slot) * d_r + k);
        p[t] = acc * scale;
        if (p[t] > m) m = p[t];
    }
    double L = 0.0;
    for (int t = 0; t < T; ++t) { p[t] = exp(p[t] - m); L += p[t]; }
    for (int t = 0; t < T; ++t) p[t] /= L;
}

/* ---- matched GQA decode: s_j = q_h K_{j,g(h)}^T / sqrt(d_h), o_h = softmax(s) V_{g(h)} -----------
 * k_pool, v_pool [num_pages][G][P][d_h]; q [B][H][d_h] already rotated; K cached already rotated. */
void oracle_gqa_decode(const void *k_pool, const void *v_pool, int dtype, const int32_t *block_table,
                       int max_pages, int P, const int32_t *seq_lens, const double *q, double scale,
                       int B, int H, int G, int d_h, double *out, double *lse) {
    int hpg = H / G;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            int g = h / hpg;
            int T = seq_lens[b];
            const double *qq = q + ((int64_t)b * H + h) * d_h;
            double *o = out + ((int64_t)b * H + h) * d_h;
            for (int i = 0; i < d_h; ++i) o[i] = 0.0;
            if (T <= 0) { if (lse) lse[(int64_t)b * H + h] = -INFINITY; continue; }
            double *s = (double *)malloc(sizeof(double) * (size_t)T);
            double m = -INFINITY;
            for (int t = 0; t < T; ++t) {
                int64_t page = page_of(block_table, max_pages, b, t / P);
                int64_t row = ((page * G + g) * P + (t % P)) * d_h;
                double acc = 0.0;
                for (int i = 0; i < d_h; ++i) acc += qq[i] * load_elem(k_pool, dtype, row + i);
                s[t] = acc * scale;
                if (s[t] > m) m = s[t];
            }
            double L = 0.0;
            for (int t = 0; t < T; ++t) { s[t] = exp(s[t] - m); L += s[t]; }
            for (int t = 0; t < T; ++t) {
                int64_t page = page_of(block_table, max_pages, b, t / P);
                int64_t row = ((page * G + g) * P + (t % P)) * d_h;
                double p = s[t] / L;
                for (int i = 0; i < d_h; ++i) o[i] += p * load_elem(v_pool, dtype, row + i);
            }
            if (lse) lse[(int64_t)b * H + h] = m + log(L);
            free(s);
        }
}

/* ---- the projections around the attention (Algorithm 1: q_t = x_t W_Q, v_t = x_t W_V, x_t W_r; then
 * then the concatenated heads through the output projection) ------------------------------------------
 * Plain matrix product y[b][n] = sum_k x[b][k] W[k][n], fp64. */
void oracle_matmul(const double *x, const double *W, int B, int K, int N, double *y) {
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += x[(int64_t)b * K + k] * W[(int64_t)k * N + n];
            y[(int64_t)b * N + n] = acc;
        }
}

/* Weight absorption: because M_h is fixed at inference, q~_h = (x W_Q^{nope,h}) M_h^T = x (W_Q^{nope,h} M_h^T)
 * (Eq. absorb applied to the projection).  W_q_nope [d_model][H][d_c], M [H][d_v][d_c] ->
 * W_abs [d_model][H][d_v] with W_abs[m][h][i] = sum_j W_q_nope[m][h][j] M[h][i][j]. */
void oracle_fold_maps(const double *W_q_nope, const double *M, int d_model, int H, int d_v, int d_c, double *W_abs) {
    for (int m = 0; m < d_model; ++m)
        for (int h = 0; h < H; ++h)
            for (int i = 0; i < d_v; ++i) {
                double acc = 0.0;
                for (int j = 0; j < d_c; ++j)
                    acc += W_q_nope[((int64_t)m * H + h) * d_c + j] * M[((int64_t)h * d_v + i) * d_c + j];
                W_abs[((int64_t)m * H + h) * d_v + i] = acc;
            }
}

/* ---- prefill / chunked prefill: causal attention with content + positional scores ------------------
 * Several query tokens per sequence.  Sequence b has ctx_lens[b] tokens cached before the chunk and
 * q_lens = cu_q[b+1] - cu_q[b] new tokens whose value rows and rotated positional keys are ALREADY in
 * the cache (appended first, as in Algorithm 1); query token i of sequence b sits at position
 * t = ctx_lens[b] + i and attends to positions 0..t.  Nothing is absorbed here: the content keys are
 * formed explicitly, K_h = V_g(h) M_h (Eq. kvm), and the score is the full-key dot product
 *   s_ij = q^nope_i . K_h,j + (q^rope_i R_t^T) . k^rope_j,   o_i = softmax_j<=t(s_ij / sqrt(d_qk)) V_g(h).
 * q_c [n_q][H][d_c], q_r [n_q][H][d_r] unrotated, M [H][d_v][d_c]; out [n_q][H][d_v], lse [n_q][H]. */
void oracle_prefill(const void *v_pool, const void *kr_pool, int dtype, const int32_t *block_table,
                    int max_pages, int P, const int32_t *cu_q, const int32_t *ctx_lens, const double *q_c,
                    const double *q_r, const double *M, double base, double scale, int B, int H, int G,
                    int d_v, int d_c, int d_r, double *out, double *lse) {
    int hpg = H / G;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            int g = h / hpg;
            int n_q = cu_q[b + 1] - cu_q[b];
            int T = ctx_lens[b] + n_q;                     /* tokens in the cache after the chunk's append */
            if (n_q <= 0) continue;
            /* explicit keys of this head: K[j][:] = v_j M_h  (d_c wide), and the value rows widened */
            double *K = (double *)malloc(sizeof(double) * (size_t)T * (size_t)d_c);
            double *V = (double *)malloc(sizeof(double) * (size_t)T * (size_t)d_v);
            double *R = (double *)malloc(sizeof(double) * (size_t)T * (size_t)(d_r > 0 ? d_r : 1));
            double *s = (double *)malloc(sizeof(double) * (size_t)T);
            double *qrot = (double *)malloc(sizeof(double) * (size_t)(d_r > 0 ? d_r : 1));
            for (int j = 0; j < T; ++j) {
                int64_t page = page_of(block_table, max_pages, b, j / P);
                int slot = j % P;
                for (int i = 0; i < d_v; ++i) V[(int64_t)j * d_v + i] = load_elem(v_pool, dtype, ((page * G + g) * P + slot) * d_v + i);
                for (int k = 0; k < d_r; ++k) R[(int64_t)j * d_r + k] = load_elem(kr_pool, dtype, (page * P + slot) * d_r + k);
                for (int c = 0; c < d_c; ++c) {
                    double acc = 0.0;
                    for (int i = 0; i < d_v; ++i) acc += V[(int64_t)j * d_v + i] * M[((int64_t)h * d_v + i) * d_c + c];
                    K[(int64_t)j * d_c + c] = acc;
                }
            }
            for (int i = 0; i < n_q; ++i) {
                int64_t row = (int64_t)(cu_q[b] + i) * H + h;
                int t = ctx_lens[b] + i;
                const double *qc = q_c + row * d_c;
                oracle_rope(q_r + row * d_r, d_r, (double)t, base, qrot);
                double m = -INFINITY;
                for (int j = 0; j <= t; ++j) {
                    double acc = 0.0;
                    for (int c = 0; c < d_c; ++c) acc += qc[c] * K[(int64_t)j * d_c + c];
                    for (int k = 0; k < d_r; ++k) acc += qrot[k] * R[(int64_t)j * d_r + k];
                    s[j] = acc * scale;
                    if (s[j] > m) m = s[j];
                }
                double L = 0.0;
                for (int j = 0; j <= t; ++j) { s[j] = exp(s[j] - m); L += s[j]; }
                double *o = out + row * d_v;
                for (int d = 0; d < d_v; ++d) o[d] = 0.0;
                for (int j = 0; j <= t; ++j) {
                    double p = s[j] / L;
                    for (int d = 0; d < d_v; ++d) o[d] += p * V[(int64_t)j * d_v + d];
                }
                if (lse) lse[row] = m + log(L);
            }
            free(K); free(V); free(R); free(s); free(qrot);
        }
}

/* Append of a chunk: token i of sequence b (i < cu_q[b+1]-cu_q[b]) is written at position ctx_lens[b] + i,
 * exactly as oracle_append writes one token (Algorithm 1's append lines, once per new token).
 * v_new [n_q][G][d_v], kr_new [n_q][d_r] unrotated.  Returns 0, or 1+b for the first sequence with a position outside its block table or a bad page id. */
int oracle_append_chunk(void *v_pool, void *kr_pool, int dtype, const int32_t *block_table, int num_pages,
                        int max_pages, int P, int G, int d_v, int d_r, double base, const double *v_new,
                        const double *kr_new, const int32_t *cu_q, const int32_t *ctx_lens, int B) {
    double *rot = (double *)malloc(sizeof(double) * (size_t)(d_r > 0 ? d_r : 1));
    int rc = 0;
    for (int b = 0; b < B && !rc; ++b)
        for (int i = 0; i < cu_q[b + 1] - cu_q[b]; ++i) {
            int64_t n = cu_q[b] + i;
            int t = ctx_lens[b] + i;
            if (t < 0 || t / P >= max_pages) { rc = 1 + b; break; }   /* position outside the block table: no lookup */
            int64_t page = page_of(block_table, max_pages, b, t / P);
            int slot = t % P;
            if (page < 0 || page >= num_pages) { rc = 1 + b; break; }
            for (int g = 0; g < G; ++g)
                for (int d = 0; d < d_v; ++d)
                    store_elem(v_pool, dtype, ((page * G + g) * P + slot) * d_v + d, v_new[(n * G + g) * d_v + d]);
            oracle_rope(kr_new + n * d_r, d_r, (double)t, base, rot);
            for (int k = 0; k < d_r; ++k) store_elem(kr_pool, dtype, (page * P + slot) * d_r + k, rot[k]);
        }
    free(rot);
    return rc;
}

#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
void oracle_set_threads(int n) { omp_set_num_threads(n); }
#else
int oracle_num_threads(void) { return 1; }
void oracle_set_threads(int n) { (void)n; }
#endif
