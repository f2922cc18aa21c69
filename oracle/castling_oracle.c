/*
 * CPU oracle for the inference-time linear-angular attention core of
 * Castling-ViT (arXiv 2211.10526).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, float64 statement of
 * what the attention core computes, written from the paper's equations so that
 * a reader can check it against them by eye.  It shares no code with the CUDA
 * library and must never be called from the product path; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What is computed, per batch b and head h, for N = gridH*gridW tokens of
 * width d (row-major [B,H,N,d] tensors, token t = y*gridW + x):
 *
 *   q^_t = q_t / max(||q_t||_2, eps),  k^_t likewise        (Sec. 3.1 text before
 *                                                            Eq. 3; text after Eq. 8;
 *                                                            last sentence of Sec. 3.2.1)
 *   Sim(t,j) = 1/2 + (q^_t . k^_j)/pi                       (Eq. 8, "linear-angular terms")
 *   A_t      = sum_j Sim(t,j) v_j                           (Eq. 9, H = Sim(Q,K) V)
 *            = 1/2 sum_j v_j + (1/pi) q^_t (K^^T V)         (Eq. 9, re-associated as in
 *                                                            the "kernel-based linear
 *                                                            attention" paragraph of Sec. 3.1)
 *   C_t[ch]  = bias[ch] + sum_{dy,dx} w[ch][dy+r][dx+r] V[y+dy][x+dx][ch]
 *                                                           (Eq. 9, M_DW V: depthwise
 *                                                            convolution of the value
 *                                                            tokens on the token grid)
 *   out_t    = A_t + C_t                                    (Eq. 9 with the sparse softmax
 *                                                            term identically zero at
 *                                                            inference, Sec. 3.2.2)
 *
 * Readings taken where the paper is silent or prints something else:
 * the 1/2 term is the token SUM of V (Eq. 8 adds 1/2 to every pair (t,j));
 * there is no row-sum denominator and no 1/sqrt(d); V is not normalised;
 * the convolution is a cross-correlation with zero "same" padding, stride 1,
 * one filter per head-channel ch = h*d + j, with an optional bias.
 *
 * Pins (tests/test_oracle_pins.py): brute force over the explicit N x N
 * similarity matrix against the re-associated form, the arccos series of
 * Eq. 8, closed forms for constant V, equal keys, d = 1, delta / shift / box
 * filters, an explicit M_DW matrix, scale invariance and linearity.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif

/* ---- Eq. 5: the exact angular kernel on a cosine x in [-1, 1] ---------- */
double castling_oracle_angular_exact(double x)
{
    return 1.0 - acos(x) / M_PI;
}

/* ---- Eq. 8: 1/2 + x/pi + (1/pi) sum_{k=1..kmax} c_k x^(2k+1),
 *      c_k = (2k)! / (2^(2k) (k!)^2 (2k+1)).  kmax = 0 is the kept part. -- */
double castling_oracle_angular_series_coeff(int k)
{
    /* (2k)! / (2^(2k) (k!)^2) built as a running product of (2i-1)/(2i) */
    double c = 1.0;
    for (int i = 1; i <= k; ++i) c *= (2.0 * i - 1.0) / (2.0 * i);
    return c / (2.0 * k + 1.0);
}

double castling_oracle_angular_series(double x, int kmax)
{
    double sum = 0.5 + x / M_PI;
    for (int k = 1; k <= kmax; ++k)
        sum += castling_oracle_angular_series_coeff(k) * pow(x, 2 * k + 1) / M_PI;
    return sum;
}

/* ---- helpers ------------------------------------------------------------ */
static double l2norm(const double* x, int d)
{
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    return sqrt(ss);
}

/* unit row: x / max(||x||, eps) */
static void unit_row(const double* x, int d, double eps, double* xhat)
{
    double nrm = l2norm(x, d);
    if (nrm < eps) nrm = eps;
    for (int i = 0; i < d; ++i) xhat[i] = x[i] / nrm;
}

/* Depthwise convolution of V on the token grid for one (b,h): Eq. 9, M_DW V.
 * conv[t][j] = bias[h*d+j] + sum w[h*d+j][dy+r][dx+r] * V[(y+dy)*gridW + x+dx][j],
 * terms outside the grid contribute zero. */
static void dwconv_head(const double* v, const double* w, const double* bias, int h,
                        int gridH, int gridW, int d, int ksize, double* conv)
{
    const int r = (ksize - 1) / 2;
    for (int y = 0; y < gridH; ++y)
        for (int x = 0; x < gridW; ++x)
            for (int j = 0; j < d; ++j) {
                const int ch = h * d + j;
                double acc = bias ? bias[ch] : 0.0;
                for (int dy = -r; dy <= r; ++dy)
                    for (int dx = -r; dx <= r; ++dx) {
                        const int yy = y + dy, xx = x + dx;
                        if (yy < 0 || yy >= gridH || xx < 0 || xx >= gridW) continue;
                        acc += w[((size_t)ch * ksize + (dy + r)) * ksize + (dx + r)]
                             * v[((size_t)yy * gridW + xx) * d + j];
                    }
                conv[((size_t)y * gridW + x) * d + j] = acc;
            }
}

/* ---- the re-associated (linear in N) form -------------------------------
 * Processes heads bh in [bh_begin, bh_end) of the flattened B*H index so a
 * caller may split the work over threads.  Returns 0, or -1 on bad arguments
 * or allocation failure. */
int castling_oracle_forward(const double* q, const double* k, const double* v,
                            const double* w, const double* bias, double* out,
                            int B, int H, int gridH, int gridW, int d, int ksize,
                            double eps, int bh_begin, int bh_end)
{
    if (!q || !k || !v || !w || !out) return -1;
    if (B <= 0 || H <= 0 || gridH <= 0 || gridW <= 0 || d <= 0) return -1;
    if (ksize <= 0 || (ksize & 1) == 0) return -1;
    if (bh_begin < 0 || bh_end > B * H || bh_begin > bh_end) return -1;
    const int N = gridH * gridW;
    double* S = (double*)malloc(sizeof(double) * d * d);   /* K^^T V, d x d */
    double* vsum = (double*)malloc(sizeof(double) * d);    /* sum_j v_j     */
    double* xhat = (double*)malloc(sizeof(double) * d);
    double* conv = (double*)malloc(sizeof(double) * (size_t)N * d);
    if (!S || !vsum || !xhat || !conv) { free(S); free(vsum); free(xhat); free(conv); return -1; }

    for (int bh = bh_begin; bh < bh_end; ++bh) {
        const int h = bh % H;
        const size_t base = (size_t)bh * N * d;
        const double* qh = q + base; const double* kh = k + base; const double* vh = v + base;
        double* oh = out + base;

        /* state: S[i][j] = sum_n k^_n[i] v_n[j];  vsum[j] = sum_n v_n[j] */
        memset(S, 0, sizeof(double) * d * d);
        memset(vsum, 0, sizeof(double) * d);
        for (int n = 0; n < N; ++n) {
            unit_row(kh + (size_t)n * d, d, eps, xhat);
            for (int i = 0; i < d; ++i)
                for (int j = 0; j < d; ++j)
                    S[i * d + j] += xhat[i] * vh[(size_t)n * d + j];
            for (int j = 0; j < d; ++j) vsum[j] += vh[(size_t)n * d + j];
        }

        dwconv_head(vh, w, bias, h, gridH, gridW, d, ksize, conv);

        /* apply: out_t = 1/2 vsum + (1/pi) q^_t S + conv_t */
        for (int t = 0; t < N; ++t) {
            unit_row(qh + (size_t)t * d, d, eps, xhat);
            for (int j = 0; j < d; ++j) {
                double lin = 0.0;
                for (int i = 0; i < d; ++i) lin += xhat[i] * S[i * d + j];
                oh[(size_t)t * d + j] = 0.5 * vsum[j] + lin / M_PI + conv[(size_t)t * d + j];
            }
        }
    }
    free(S); free(vsum); free(xhat); free(conv);
    return 0;
}

/* ---- leading tokens that are not on the grid (class / distillation tokens) ----
 * Reading taken where the paper is silent: a sequence may start with `prefix` tokens that
 * have no grid position.  They attend and are attended to like every other token (they
 * enter S, the token sum and get an output row from Eq. 9's attention terms), but the
 * depthwise convolution (and its bias) is defined on the 2-D grid only: it reads and
 * writes the gridH*gridW tokens that follow the prefix and contributes nothing to the
 * prefix rows.  prefix = 0 is castling_oracle_forward. */
int castling_oracle_forward_prefix(const double* q, const double* k, const double* v,
                                   const double* w, const double* bias, double* out,
                                   int B, int H, int prefix, int gridH, int gridW, int d, int ksize,
                                   double eps, int bh_begin, int bh_end)
{
    if (!q || !k || !v || !w || !out) return -1;
    if (B <= 0 || H <= 0 || prefix < 0 || gridH <= 0 || gridW <= 0 || d <= 0) return -1;
    if (ksize <= 0 || (ksize & 1) == 0) return -1;
    if (bh_begin < 0 || bh_end > B * H || bh_begin > bh_end) return -1;
    const int G = gridH * gridW, T = prefix + G;           /* T tokens per sequence */
    double* state = (double*)malloc(sizeof(double) * d * d);
    double* tok_sum = (double*)malloc(sizeof(double) * d);
    double* u = (double*)malloc(sizeof(double) * d);
    double* grid_conv = (double*)malloc(sizeof(double) * (size_t)G * d);
    if (!state || !tok_sum || !u || !grid_conv) { free(state); free(tok_sum); free(u); free(grid_conv); return -1; }

    for (int bh = bh_begin; bh < bh_end; ++bh) {
        const int h = bh % H;
        const size_t base = (size_t)bh * T * d;
        const double* qp = q + base; const double* kp = k + base; const double* vp = v + base;
        double* op = out + base;

        memset(state, 0, sizeof(double) * d * d);
        memset(tok_sum, 0, sizeof(double) * d);
        for (int m = 0; m < T; ++m) {                      /* every token, prefix included */
            unit_row(kp + (size_t)m * d, d, eps, u);
            for (int a = 0; a < d; ++a)
                for (int c = 0; c < d; ++c)
                    state[a * d + c] += u[a] * vp[(size_t)m * d + c];
            for (int c = 0; c < d; ++c) tok_sum[c] += vp[(size_t)m * d + c];
        }

        dwconv_head(vp + (size_t)prefix * d, w, bias, h, gridH, gridW, d, ksize, grid_conv);  /* grid tokens only */

        for (int m = 0; m < T; ++m) {
            unit_row(qp + (size_t)m * d, d, eps, u);
            for (int c = 0; c < d; ++c) {
                double dot = 0.0;
                for (int a = 0; a < d; ++a) dot += u[a] * state[a * d + c];
                const double on_grid = (m >= prefix) ? grid_conv[(size_t)(m - prefix) * d + c] : 0.0;
                op[(size_t)m * d + c] = tok_sum[c] / 2.0 + dot / M_PI + on_grid;
            }
        }
    }
    free(state); free(tok_sum); free(u); free(grid_conv);
    return 0;
}

/* ---- the definition written out: explicit N x N similarity matrix -------
 * Sim[t][j] = 1/2 + (q^_t . k^_j)/pi (Eq. 8), A = Sim V (Eq. 9), plus the
 * depthwise convolution.  O(N^2 d); for small N only. */
int castling_oracle_forward_bruteforce(const double* q, const double* k, const double* v,
                                       const double* w, const double* bias, double* out,
                                       int B, int H, int gridH, int gridW, int d, int ksize,
                                       double eps)
{
    if (!q || !k || !v || !w || !out) return -1;
    if (B <= 0 || H <= 0 || gridH <= 0 || gridW <= 0 || d <= 0) return -1;
    if (ksize <= 0 || (ksize & 1) == 0) return -1;
    const int N = gridH * gridW;
    double* qhat = (double*)malloc(sizeof(double) * (size_t)N * d);
    double* khat = (double*)malloc(sizeof(double) * (size_t)N * d);
    double* sim  = (double*)malloc(sizeof(double) * (size_t)N * N);
    double* conv = (double*)malloc(sizeof(double) * (size_t)N * d);
    if (!qhat || !khat || !sim || !conv) { free(qhat); free(khat); free(sim); free(conv); return -1; }

    for (int bh = 0; bh < B * H; ++bh) {
        const int h = bh % H;
        const size_t base = (size_t)bh * N * d;
        const double* vh = v + base;
        for (int t = 0; t < N; ++t) {
            unit_row(q + base + (size_t)t * d, d, eps, qhat + (size_t)t * d);
            unit_row(k + base + (size_t)t * d, d, eps, khat + (size_t)t * d);
        }
        for (int t = 0; t < N; ++t)
            for (int j = 0; j < N; ++j) {
                double dot = 0.0;
                for (int i = 0; i < d; ++i) dot += qhat[(size_t)t * d + i] * khat[(size_t)j * d + i];
                sim[(size_t)t * N + j] = 0.5 + dot / M_PI;
            }
        dwconv_head(vh, w, bias, h, gridH, gridW, d, ksize, conv);
        for (int t = 0; t < N; ++t)
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int j = 0; j < N; ++j) acc += sim[(size_t)t * N + j] * vh[(size_t)j * d + c];
                out[base + (size_t)t * d + c] = acc + conv[(size_t)t * d + c];
            }
    }
    free(qhat); free(khat); free(sim); free(conv);
    return 0;
}

/* The explicit similarity matrix of one head, for inspection by the pins:
 * sim[t][j] = 1/2 + (q^_t . k^_j)/pi, N x N. */
int castling_oracle_similarity(const double* q, const double* k, double* sim, int N, int d, double eps)
{
    if (!q || !k || !sim || N <= 0 || d <= 0) return -1;
    double* qh = (double*)malloc(sizeof(double) * d);
    double* kh = (double*)malloc(sizeof(double) * d);
    if (!qh || !kh) { free(qh); free(kh); return -1; }
    for (int t = 0; t < N; ++t) {
        unit_row(q + (size_t)t * d, d, eps, qh);
        for (int j = 0; j < N; ++j) {
            unit_row(k + (size_t)j * d, d, eps, kh);
            double dot = 0.0;
            for (int i = 0; i < d; ++i) dot += qh[i] * kh[i];
            sim[(size_t)t * N + j] = 0.5 + dot / M_PI;
        }
    }
    free(qh); free(kh);
    return 0;
}

/* ==== variants of the attention beyond the inference-time core ==================================
 *
 * (a) Row-sum normalisation.  Kernel-based linear attention as Sec. 3.1 states it (Eq. 3) divides
 *     row t by phi(Q_t) . sum_j phi(K_j), i.e. by the sum of that row's similarities; Eq. 9 prints
 *     no such denominator, so the core above has none.  With the kept kernel of Eq. 8 the row sum
 *     is  sum_j (1/2 + q^_t.k^_j/pi) = T/2 + q^_t . (sum_j k^_j)/pi  over the T tokens of the
 *     sequence, and the normalised attention term is A_t divided by it.  The depthwise convolution
 *     is added afterwards, unchanged.
 * (b) The exact angular kernel, Sim = 1 - arccos(q^.k^)/pi (Eq. 4-5), in place of its kept part.
 * (c) The auxiliary branch of training, Mask_eps(Softmax_j(q^_t . k^_j)) (Eq. 10, Sec. 3.2.2),
 *     Mask_eps(x) = x if x > eps else 0, added to the attention weights.  Readings taken: the
 *     softmax runs over the keys of one query, on the cosines of the unit rows (Sec. 3.2.1, last
 *     sentence: the normalisation is inserted into the sparse branch as well), without 1/sqrt(d)
 *     (Eq. 10 has none) and without renormalising what survives the mask.
 * (b) and (c) have no re-associated form: they are written with the explicit T x T weight matrix.
 */

/* (a), linear in the number of tokens.  prefix leading tokens are off the grid, as in
 * castling_oracle_forward_prefix; prefix = 0 is the plain grid. */
int castling_oracle_forward_rownorm(const double* q, const double* k, const double* v,
                                    const double* w, const double* bias, double* out,
                                    int B, int H, int prefix, int gridH, int gridW, int d, int ksize,
                                    double eps, int bh_begin, int bh_end)
{
    if (!q || !k || !v || !w || !out) return -1;
    if (B <= 0 || H <= 0 || prefix < 0 || gridH <= 0 || gridW <= 0 || d <= 0) return -1;
    if (ksize <= 0 || (ksize & 1) == 0) return -1;
    if (bh_begin < 0 || bh_end > B * H || bh_begin > bh_end) return -1;
    const int G = gridH * gridW, T = prefix + G;
    double* kv = (double*)malloc(sizeof(double) * d * d);     /* sum_j k^_j^T v_j */
    double* vtot = (double*)malloc(sizeof(double) * d);       /* sum_j v_j        */
    double* ktot = (double*)malloc(sizeof(double) * d);       /* sum_j k^_j       */
    double* u = (double*)malloc(sizeof(double) * d);
    double* gconv = (double*)malloc(sizeof(double) * (size_t)G * d);
    if (!kv || !vtot || !ktot || !u || !gconv) { free(kv); free(vtot); free(ktot); free(u); free(gconv); return -1; }

    for (int bh = bh_begin; bh < bh_end; ++bh) {
        const int h = bh % H;
        const size_t base = (size_t)bh * T * d;
        const double* qp = q + base; const double* kp = k + base; const double* vp = v + base;
        double* op = out + base;
        memset(kv, 0, sizeof(double) * d * d);
        memset(vtot, 0, sizeof(double) * d);
        memset(ktot, 0, sizeof(double) * d);
        for (int m = 0; m < T; ++m) {
            unit_row(kp + (size_t)m * d, d, eps, u);
            for (int a = 0; a < d; ++a) {
                ktot[a] += u[a];
                for (int c = 0; c < d; ++c) kv[a * d + c] += u[a] * vp[(size_t)m * d + c];
            }
            for (int c = 0; c < d; ++c) vtot[c] += vp[(size_t)m * d + c];
        }
        const double* vgrid = vp + (size_t)prefix * d;        /* the convolution sees the grid tokens only */
        dwconv_head(vgrid, w, bias, h, gridH, gridW, d, ksize, gconv);
        for (int m = 0; m < T; ++m) {
            unit_row(qp + (size_t)m * d, d, eps, u);
            double rowsum = 0.5 * T;                           /* sum_j (1/2 + q^_m.k^_j/pi) */
            for (int a = 0; a < d; ++a) rowsum += u[a] * ktot[a] / M_PI;
            for (int c = 0; c < d; ++c) {
                double num = 0.5 * vtot[c];
                for (int a = 0; a < d; ++a) num += u[a] * kv[a * d + c] / M_PI;
                const double on_grid = (m >= prefix) ? gconv[(size_t)(m - prefix) * d + c] : 0.0;
                op[(size_t)m * d + c] = num / rowsum + on_grid;
            }
        }
    }
    free(kv); free(vtot); free(ktot); free(u); free(gconv);
    return 0;
}

/* The explicit weight matrix of one head, weights[t][j], T x T, for (a)-(c):
 *   kernel   0: 1/2 + x/pi (Eq. 8, kept part);  1: 1 - arccos(x)/pi (Eq. 5);  x = q^_t . k^_j
 *   rownorm  != 0: every row of that is divided by its sum (Eq. 3)
 *   sparse   != 0: Mask_sparse_eps(Softmax_j(x)) (Eq. 10) is added afterwards */
int castling_oracle_attention_weights(const double* q, const double* k, double* weights, int T, int d,
                                      double eps, int kernel, int rownorm, int sparse, double sparse_eps)
{
    if (!q || !k || !weights || T <= 0 || d <= 0 || kernel < 0 || kernel > 1) return -1;
    double* qu = (double*)malloc(sizeof(double) * (size_t)T * d);
    double* ku = (double*)malloc(sizeof(double) * (size_t)T * d);
    double* cosine = (double*)malloc(sizeof(double) * T);
    if (!qu || !ku || !cosine) { free(qu); free(ku); free(cosine); return -1; }
    for (int t = 0; t < T; ++t) {
        unit_row(q + (size_t)t * d, d, eps, qu + (size_t)t * d);
        unit_row(k + (size_t)t * d, d, eps, ku + (size_t)t * d);
    }
    for (int t = 0; t < T; ++t) {
        double* row = weights + (size_t)t * T;
        double total = 0.0;
        for (int j = 0; j < T; ++j) {
            double x = 0.0;
            for (int i = 0; i < d; ++i) x += qu[(size_t)t * d + i] * ku[(size_t)j * d + i];
            cosine[j] = x;
            if (kernel == 0) {
                row[j] = 0.5 + x / M_PI;
            } else {
                const double xc = x > 1.0 ? 1.0 : (x < -1.0 ? -1.0 : x);   /* rounding may leave [-1, 1] */
                row[j] = castling_oracle_angular_exact(xc);
            }
            total += row[j];
        }
        if (rownorm)
            for (int j = 0; j < T; ++j) row[j] /= total;
        if (sparse) {
            double z = 0.0;
            for (int j = 0; j < T; ++j) z += exp(cosine[j]);
            for (int j = 0; j < T; ++j) {
                const double p = exp(cosine[j]) / z;
                if (p > sparse_eps) row[j] += p;
            }
        }
    }
    free(qu); free(ku); free(cosine);
    return 0;
}

/* out = weights . V + DWConv(V) with the weight matrix above; grid tokens only (no leading tokens).
 * O(T^2 d) per head. */
int castling_oracle_forward_matrix(const double* q, const double* k, const double* v,
                                   const double* w, const double* bias, double* out,
                                   int B, int H, int gridH, int gridW, int d, int ksize, double eps,
                                   int kernel, int rownorm, int sparse, double sparse_eps,
                                   int bh_begin, int bh_end)
{
    if (!q || !k || !v || !w || !out) return -1;
    if (B <= 0 || H <= 0 || gridH <= 0 || gridW <= 0 || d <= 0) return -1;
    if (ksize <= 0 || (ksize & 1) == 0) return -1;
    if (bh_begin < 0 || bh_end > B * H || bh_begin > bh_end) return -1;
    const int T = gridH * gridW;
    double* wt = (double*)malloc(sizeof(double) * (size_t)T * T);
    double* conv = (double*)malloc(sizeof(double) * (size_t)T * d);
    if (!wt || !conv) { free(wt); free(conv); return -1; }
    int rc = 0;
    for (int bh = bh_begin; bh < bh_end && rc == 0; ++bh) {
        const int h = bh % H;
        const size_t base = (size_t)bh * T * d;
        rc = castling_oracle_attention_weights(q + base, k + base, wt, T, d, eps, kernel, rownorm, sparse, sparse_eps);
        if (rc) break;
        dwconv_head(v + base, w, bias, h, gridH, gridW, d, ksize, conv);
        for (int t = 0; t < T; ++t)
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int j = 0; j < T; ++j) acc += wt[(size_t)t * T + j] * v[base + (size_t)j * d + c];
                out[base + (size_t)t * d + c] = acc + conv[(size_t)t * d + c];
            }
    }
    free(wt); free(conv);
    return rc;
}

/* Softmax_j(q^_t . k^_j) of one head, T x T: lets a test pick a mask threshold that lies in a gap
 * of these values, so that the comparison with an fp32 implementation does not hinge on ties. */
int castling_oracle_softmax_probs(const double* q, const double* k, double* probs, int T, int d, double eps)
{
    if (!q || !k || !probs || T <= 0 || d <= 0) return -1;
    double* qu = (double*)malloc(sizeof(double) * d);
    double* ku = (double*)malloc(sizeof(double) * (size_t)T * d);
    if (!qu || !ku) { free(qu); free(ku); return -1; }
    for (int j = 0; j < T; ++j) unit_row(k + (size_t)j * d, d, eps, ku + (size_t)j * d);
    for (int t = 0; t < T; ++t) {
        unit_row(q + (size_t)t * d, d, eps, qu);
        double z = 0.0;
        for (int j = 0; j < T; ++j) {
            double x = 0.0;
            for (int i = 0; i < d; ++i) x += qu[i] * ku[(size_t)j * d + i];
            probs[(size_t)t * T + j] = exp(x);
            z += exp(x);
        }
        for (int j = 0; j < T; ++j) probs[(size_t)t * T + j] /= z;
    }
    free(qu); free(ku);
    return 0;
}
