/*
 * CPU oracle for the Based sequence-mixing hot path (arXiv 2402.18668).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, fp64 restatement of
 * the paper's definitions, used only to check the CUDA library and to time a
 * CPU baseline.  It shares no code with the CUDA path and the product never
 * calls it.
 *
 * What it implements, and where the paper defines it:
 *   oracle_phi                  2nd-order Taylor feature map: Eq. (3) of Sec. 4.1
 *                               with the scale factors of the TaylorExp module in
 *                               the App. B.1 PyTorch listing (x / d'^(1/4) and
 *                               (x (x) x) / (sqrt(2) sqrt(d'))).
 *   oracle_linattn_quadratic    causal linear attention in its "attention" form,
 *                               left-hand side of Eq. (2), Sec. 4.1: every (i, j<=i)
 *                               pair visited explicitly.  This is the authority.
 *   oracle_linattn_row          one output row of the same definition.
 *   oracle_linattn_recurrent    recurrent form (KV-state / K-state recurrences and
 *                               Eq. (2b) of Sec. 4.1; update-then-read order of the
 *                               App. B.2 step() listing).  L = 1 is one decode step.
 *   oracle_swa                  exact softmax attention, Eq. (1) of Sec. 2,
 *                               restricted to the causal window
 *                               {k_{i-w+1}, ..., k_i} of Sec. 4.2.
 *   oracle_swa_decode_step      one generation step of the same sliding-window attention on a
 *                               rolling cache of the last w keys and values (the PyTorch
 *                               sliding-window listing and Algorithm 3 of App. B.2, plus the
 *                               cache update the paper's benchmark leaves out).
 *   oracle_linattn_quadratic_ld the quadratic form again with long double
 *                               accumulators (adequacy check of fp64 on tiny inputs).
 *   oracle_linattn_numerator    the numerator alone, sum_{j<=i} phi(q_i).phi(k_j) v_j: what Algorithm 1
 *                               and the kernel micro-benchmarks of App. "IO Aware Implementations" (their
 *                               captions say they time the numerator) compute.
 *   oracle_linattn_backward     gradients of the definition form (left-hand side of Eq. (2)) with respect
 *                               to q, k, v for a given gradient of the output; the paper calls prefill
 *                               "the forward pass during training" but prints no backward algorithm, so
 *                               this is the chain rule applied to the definition, pair by pair.
 *   oracle_psi, oracle_state_to_sym, oracle_linattn_recurrent_sym
 *                               the same recurrences on the symmetric feature set whose size
 *                               the appendix "Computing Recurrent State Size" counts,
 *                               1 + 3d'/2 + d'^2/2 features: the product x_m x_n is kept once
 *                               per unordered pair.  psi(q).psi(k) = phi(q).phi(k), so outputs
 *                               are those of the full form; the symmetric state is the full
 *                               state with each (m,n),(n,m) pair of rows folded into one.
 *
 *   oracle_baseconv_gate        the gated short convolution at the core of the BaseConv layer of
 *                               App. "Extended Architecture Details" (paragraph "Convolution"):
 *                               z = a (.) SiLU(h * g + b2), h * g a causal depthwise convolution
 *                               of width w (the paper suggests 3); the three projections around
 *                               it are plain matrix products and are not part of this function.
 *   oracle_baseconv_gate_step   the same for one new token, from the last w-1 rows of g.
 *
 * Parity pins: every function above is pinned by tests/test_oracle_*.py
 * (closed forms, special cases, library softmax attention, the Taylor remainder
 * bound, brute force in extended precision).  Nothing here is "parity unpinned".
 *
 * Layouts (row-major, last index contiguous), all double:
 *   q, k : [B, H, L, dp]      v, y : [B, H, L, dv]
 *   S    : [B, H, D, dv]      z    : [B, H, D]        D = 1 + dp + dp*dp
 * Feature order inside D: index 0 the constant, 1..dp the linear terms,
 * 1 + dp + m*dp + n the (m, n) product.
 * Symmetric form: Ds = 1 + dp + dp(dp+1)/2; index 0 the constant, 1..dp the linear terms, then
 * the pairs m <= n in row-major order of the upper triangle: (0,0), (0,1), ..., (0,dp-1), (1,1), ...
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_EPS 1e-12 /* the eps of the App. B listings, added to the denominator */

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int oracle_feature_dim(int dp) { return 1 + dp + dp * dp; }

/* phi(x) = [1, x / d'^(1/4), vec(x x^T) / (sqrt 2 * sqrt d')] */
void oracle_phi(const double *x, int dp, double *out) {
    const double rd = sqrt((double)dp);
    const double rrd = sqrt(rd);
    const double r2 = sqrt(2.0);
    out[0] = 1.0;
    for (int m = 0; m < dp; ++m) out[1 + m] = x[m] / rrd;
    for (int m = 0; m < dp; ++m)
        for (int n = 0; n < dp; ++n) out[1 + dp + m * dp + n] = (x[m] * x[n] / r2) / rd;
}

/* The similarity phi(q).phi(k) in closed form: 1 + s/sqrt(d') + s^2/(2 d'), s = q.k */
static double taylor_weight(const double *qi, const double *kj, int dp) {
    double s = 0.0;
    for (int m = 0; m < dp; ++m) s += qi[m] * kj[m];
    return 1.0 + s / sqrt((double)dp) + s * s / (2.0 * (double)dp);
}

/* One output row i of one head, straight from the definition. */
void oracle_linattn_row(const double *q, const double *k, const double *v, int L, int dp, int dv,
                        int i, double *y_row) {
    (void)L;
    double den = 0.0;
    for (int c = 0; c < dv; ++c) y_row[c] = 0.0;
    for (int j = 0; j <= i; ++j) {
        const double w = taylor_weight(q + (size_t)i * dp, k + (size_t)j * dp, dp);
        den += w;
        for (int c = 0; c < dv; ++c) y_row[c] += w * v[(size_t)j * dv + c];
    }
    for (int c = 0; c < dv; ++c) y_row[c] /= (den + ORACLE_EPS);
}

/*
 * Quadratic definition for all heads.  S and z (nullable together) receive the
 * final state sum_j phi(k_j) v_j^T and sum_j phi(k_j), accumulated directly.
 */
void oracle_linattn_quadratic(const double *q, const double *k, const double *v, double *y, double *S,
                              double *z, int B, int H, int L, int dp, int dv) {
    const int D = oracle_feature_dim(dp);
    const long nh = (long)B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < nh; ++bh) {
        const double *qh = q + (size_t)bh * L * dp;
        const double *kh = k + (size_t)bh * L * dp;
        const double *vh = v + (size_t)bh * L * dv;
        double *yh = y + (size_t)bh * L * dv;
        for (int i = 0; i < L; ++i) oracle_linattn_row(qh, kh, vh, L, dp, dv, i, yh + (size_t)i * dv);
        if (S && z) {
            double *Sh = S + (size_t)bh * D * dv;
            double *zh = z + (size_t)bh * D;
            double *f = (double *)malloc(sizeof(double) * (size_t)D);
            memset(Sh, 0, sizeof(double) * (size_t)D * dv);
            memset(zh, 0, sizeof(double) * (size_t)D);
            for (int j = 0; j < L; ++j) {
                oracle_phi(kh + (size_t)j * dp, dp, f);
                for (int a = 0; a < D; ++a) {
                    zh[a] += f[a];
                    for (int c = 0; c < dv; ++c) Sh[(size_t)a * dv + c] += f[a] * vh[(size_t)j * dv + c];
                }
            }
            free(f);
        }
    }
}

/*
 * Recurrent form.  S, z are read as the initial state and overwritten with the
 * final one.  Per token: S += phi(k) v^T; z += phi(k); then
 * y = phi(q) S / (phi(q) z + eps).
 */
void oracle_linattn_recurrent(const double *q, const double *k, const double *v, double *y, double *S,
                              double *z, int B, int H, int L, int dp, int dv) {
    const int D = oracle_feature_dim(dp);
    const long nh = (long)B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < nh; ++bh) {
        const double *qh = q + (size_t)bh * L * dp;
        const double *kh = k + (size_t)bh * L * dp;
        const double *vh = v + (size_t)bh * L * dv;
        double *yh = y + (size_t)bh * L * dv;
        double *Sh = S + (size_t)bh * D * dv;
        double *zh = z + (size_t)bh * D;
        double *f = (double *)malloc(sizeof(double) * (size_t)D);
        double *g = (double *)malloc(sizeof(double) * (size_t)D);
        for (int i = 0; i < L; ++i) {
            oracle_phi(kh + (size_t)i * dp, dp, f);
            for (int a = 0; a < D; ++a) {
                zh[a] += f[a];
                for (int c = 0; c < dv; ++c) Sh[(size_t)a * dv + c] += f[a] * vh[(size_t)i * dv + c];
            }
            oracle_phi(qh + (size_t)i * dp, dp, g);
            double den = 0.0;
            for (int a = 0; a < D; ++a) den += g[a] * zh[a];
            for (int c = 0; c < dv; ++c) {
                double num = 0.0;
                for (int a = 0; a < D; ++a) num += g[a] * Sh[(size_t)a * dv + c];
                yh[(size_t)i * dv + c] = num / (den + ORACLE_EPS);
            }
        }
        free(f);
        free(g);
    }
}

/* Sliding-window softmax attention: query i sees keys max(0, i-w+1) .. i. */
void oracle_swa(const double *q, const double *k, const double *v, double *y, int B, int H, int L, int d,
                int w, double scale) {
    const long nh = (long)B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < nh; ++bh) {
        const double *qh = q + (size_t)bh * L * d;
        const double *kh = k + (size_t)bh * L * d;
        const double *vh = v + (size_t)bh * L * d;
        double *yh = y + (size_t)bh * L * d;
        double *p = (double *)malloc(sizeof(double) * (size_t)(w > 0 ? w : 1));
        for (int i = 0; i < L; ++i) {
            const int lo = (i - w + 1 > 0) ? i - w + 1 : 0;
            double mx = -INFINITY;
            for (int j = lo; j <= i; ++j) {
                double s = 0.0;
                for (int m = 0; m < d; ++m) s += qh[(size_t)i * d + m] * kh[(size_t)j * d + m];
                p[j - lo] = s * scale;
                if (p[j - lo] > mx) mx = p[j - lo];
            }
            double sum = 0.0;
            for (int j = lo; j <= i; ++j) {
                p[j - lo] = exp(p[j - lo] - mx);
                sum += p[j - lo];
            }
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int j = lo; j <= i; ++j) acc += p[j - lo] * vh[(size_t)j * d + c];
                yh[(size_t)i * d + c] = acc / sum;
            }
        }
        free(p);
    }
}

/*
 * One decode step on a rolling window cache.  kc, vc: [B, H, w, d]; the token at absolute
 * position t is kept in slot t % w.  The new k, v (position pos) are written first, then the
 * query attends over the cached positions max(0, pos-w+1) .. pos (softmax does not depend on
 * the slot order).  q, k, v, y: [B, H, d].
 */
void oracle_swa_decode_step(const double *q, const double *k, const double *v, double *kc, double *vc, double *y,
                            int B, int H, int d, int w, int pos, double scale) {
    const long nh = (long)B * H;
    const int nvalid = (pos + 1 < w) ? pos + 1 : w;
#pragma omp parallel for schedule(static)
    for (long bh = 0; bh < nh; ++bh) {
        double *kh = kc + (size_t)bh * w * d;
        double *vh = vc + (size_t)bh * w * d;
        const int slot = pos % w;
        for (int m = 0; m < d; ++m) {
            kh[(size_t)slot * d + m] = k[(size_t)bh * d + m];
            vh[(size_t)slot * d + m] = v[(size_t)bh * d + m];
        }
        double *p = (double *)malloc(sizeof(double) * (size_t)w);
        double mx = -INFINITY;
        for (int j = 0; j < nvalid; ++j) {          /* before the ring is full, slots 0..pos are the valid ones */
            double s = 0.0;
            for (int m = 0; m < d; ++m) s += q[(size_t)bh * d + m] * kh[(size_t)j * d + m];
            p[j] = s * scale;
            if (p[j] > mx) mx = p[j];
        }
        double sum = 0.0;
        for (int j = 0; j < nvalid; ++j) {
            p[j] = exp(p[j] - mx);
            sum += p[j];
        }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int j = 0; j < nvalid; ++j) acc += p[j] * vh[(size_t)j * d + c];
            y[(size_t)bh * d + c] = acc / sum;
        }
        free(p);
    }
}

/* Quadratic definition, one head, long double accumulation (tiny inputs only). */
void oracle_linattn_quadratic_ld(const double *q, const double *k, const double *v, double *y, int L,
                                 int dp, int dv) {
    for (int i = 0; i < L; ++i) {
        long double den = 0.0L;
        long double *num = (long double *)calloc((size_t)dv, sizeof(long double));
        for (int j = 0; j <= i; ++j) {
            long double s = 0.0L;
            for (int m = 0; m < dp; ++m) s += (long double)q[(size_t)i * dp + m] * (long double)k[(size_t)j * dp + m];
            const long double w = 1.0L + s / sqrtl((long double)dp) + s * s / (2.0L * (long double)dp);
            den += w;
            for (int c = 0; c < dv; ++c) num[c] += w * (long double)v[(size_t)j * dv + c];
        }
        for (int c = 0; c < dv; ++c) y[(size_t)i * dv + c] = (double)(num[c] / (den + (long double)ORACLE_EPS));
        free(num);
    }
}

/* ---- symmetric feature set (appendix "Computing Recurrent State Size") ------------------- */

int oracle_feature_dim_sym(int dp) { return 1 + dp + dp * (dp + 1) / 2; }

/*
 * psi(x): constant and linear terms as in phi; one feature per unordered pair {m, n}:
 * x_m^2 / (sqrt 2 sqrt d') on the diagonal and x_m x_n / sqrt d' off it (the two equal
 * entries (m,n), (n,m) of phi, each x_m x_n / (sqrt 2 sqrt d'), merged into one of sqrt 2 times
 * the size, which keeps the inner product).
 */
void oracle_psi(const double *x, int dp, double *out) {
    const double rd = sqrt((double)dp);
    const double rrd = sqrt(rd);
    const double r2 = sqrt(2.0);
    int at = 0;
    out[at++] = 1.0;
    for (int m = 0; m < dp; ++m) out[at++] = x[m] / rrd;
    for (int m = 0; m < dp; ++m)
        for (int n = m; n < dp; ++n) out[at++] = (m == n) ? (x[m] * x[m] / r2) / rd : (x[m] * x[n]) / rd;
}

/*
 * Fold a full state (D rows) into the symmetric one (Ds rows): constant and linear rows are
 * copied, the diagonal rows too, and rows (m,n), (n,m) become (row_mn + row_nm) / sqrt 2.
 * `width` is dv for the KV-state and 1 for the K-state.
 */
void oracle_state_to_sym(const double *full, double *sym, long nheads, int dp, int width) {
    const int D = oracle_feature_dim(dp), Ds = oracle_feature_dim_sym(dp);
    const double r2 = sqrt(2.0);
    for (long h = 0; h < nheads; ++h) {
        const double *f = full + (size_t)h * D * width;
        double *s = sym + (size_t)h * Ds * width;
        for (int a = 0; a <= dp; ++a)
            for (int c = 0; c < width; ++c) s[(size_t)a * width + c] = f[(size_t)a * width + c];
        int at = 1 + dp;
        for (int m = 0; m < dp; ++m)
            for (int n = m; n < dp; ++n, ++at)
                for (int c = 0; c < width; ++c) {
                    const double a = f[(size_t)(1 + dp + m * dp + n) * width + c];
                    const double b = f[(size_t)(1 + dp + n * dp + m) * width + c];
                    s[(size_t)at * width + c] = (m == n) ? a : (a + b) / r2;
                }
    }
}

/* The recurrent form on the symmetric state: S [B,H,Ds,dv], z [B,H,Ds]; otherwise as above. */
void oracle_linattn_recurrent_sym(const double *q, const double *k, const double *v, double *y, double *S,
                                  double *z, int B, int H, int L, int dp, int dv) {
    const int D = oracle_feature_dim_sym(dp);
    const long nh = (long)B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < nh; ++bh) {
        const double *qh = q + (size_t)bh * L * dp;
        const double *kh = k + (size_t)bh * L * dp;
        const double *vh = v + (size_t)bh * L * dv;
        double *yh = y + (size_t)bh * L * dv;
        double *Sh = S + (size_t)bh * D * dv;
        double *zh = z + (size_t)bh * D;
        double *f = (double *)malloc(sizeof(double) * (size_t)D);
        double *g = (double *)malloc(sizeof(double) * (size_t)D);
        for (int i = 0; i < L; ++i) {
            oracle_psi(kh + (size_t)i * dp, dp, f);
            for (int a = 0; a < D; ++a) {
                zh[a] += f[a];
                for (int c = 0; c < dv; ++c) Sh[(size_t)a * dv + c] += f[a] * vh[(size_t)i * dv + c];
            }
            oracle_psi(qh + (size_t)i * dp, dp, g);
            double den = 0.0;
            for (int a = 0; a < D; ++a) den += g[a] * zh[a];
            for (int c = 0; c < dv; ++c) {
                double num = 0.0;
                for (int a = 0; a < D; ++a) num += g[a] * Sh[(size_t)a * dv + c];
                yh[(size_t)i * dv + c] = num / (den + ORACLE_EPS);
            }
        }
        free(f);
        free(g);
    }
}

/* ---- gated short convolution of the BaseConv layer (App. "Extended Architecture Details") ---- */

static double silu(double x) { return x / (1.0 + exp(-x)); }

/*
 * a, g, out: [B, N, C]; h: [w, C] (h[0] is the tap on the current token, h[j] on the token j
 * steps back); b2: [C].  out[b,i,c] = a[b,i,c] * SiLU(sum_{j<w, j<=i} h[j,c] g[b,i-j,c] + b2[c]).
 */
void oracle_baseconv_gate(const double *a, const double *g, const double *h, const double *b2, double *out,
                          int B, int N, int C, int w) {
#pragma omp parallel for schedule(static)
    for (long bi = 0; bi < (long)B * N; ++bi) {
        const long b = bi / N, i = bi % N;
        for (int c = 0; c < C; ++c) {
            double acc = b2[c];
            for (int j = 0; j < w && j <= i; ++j) acc += h[(size_t)j * C + c] * g[((size_t)b * N + (i - j)) * C + c];
            out[(size_t)bi * C + c] = a[(size_t)bi * C + c] * silu(acc);
        }
    }
}

/*
 * One token: a, g, out [B, C]; state [B, w-1, C] holds the previous rows of g, state[b,j] = g of
 * the token j+1 steps back (zeros before the sequence start); it is shifted and g stored in slot 0.
 */
void oracle_baseconv_gate_step(const double *a, const double *g, const double *h, const double *b2, double *state,
                               double *out, int B, int C, int w) {
    for (int b = 0; b < B; ++b) {
        double *st = state + (size_t)b * (w - 1) * C;
        for (int c = 0; c < C; ++c) {
            double acc = b2[c] + h[c] * g[(size_t)b * C + c];
            for (int j = 1; j < w; ++j) acc += h[(size_t)j * C + c] * st[(size_t)(j - 1) * C + c];
            out[(size_t)b * C + c] = a[(size_t)b * C + c] * silu(acc);
            for (int j = w - 2; j >= 1; --j) st[(size_t)j * C + c] = st[(size_t)(j - 1) * C + c];
            if (w > 1) st[c] = g[(size_t)b * C + c];
        }
    }
}

/* ---- numerator only (Algorithm 1 stops here; the micro-benchmark figures time this) ---------- */
void oracle_linattn_numerator(const double *q, const double *k, const double *v, double *y, int B, int H, int L,
                              int dp, int dv) {
    const long nh = (long)B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < nh; ++bh) {
        const double *qh = q + (size_t)bh * L * dp;
        const double *kh = k + (size_t)bh * L * dp;
        const double *vh = v + (size_t)bh * L * dv;
        double *yh = y + (size_t)bh * L * dv;
        for (int i = 0; i < L; ++i) {
            for (int c = 0; c < dv; ++c) yh[(size_t)i * dv + c] = 0.0;
            for (int j = 0; j <= i; ++j) {
                const double w = taylor_weight(qh + (size_t)i * dp, kh + (size_t)j * dp, dp);
                for (int c = 0; c < dv; ++c) yh[(size_t)i * dv + c] += w * vh[(size_t)j * dv + c];
            }
        }
    }
}

/* ---- backward of the definition form ------------------------------------------------------ */
/*
 * y_i = N_i / D_i,  N_i = sum_{j<=i} w_ij v_j,  D_i = sum_{j<=i} w_ij + eps,
 * w_ij = 1 + s_ij / sqrt(d') + s_ij^2 / (2 d'),  s_ij = q_i . k_j.
 * With G_i the gradient of the loss with respect to y_i:
 *   dN_i = G_i / D_i (a vector),  dD_i = -(G_i . y_i) / D_i (a scalar),
 *   dw_ij = dN_i . v_j + dD_i,  ds_ij = dw_ij (1 / sqrt(d') + s_ij / d'),
 *   dv_j = sum_{i>=j} w_ij dN_i,  dq_i = sum_{j<=i} ds_ij k_j,  dk_j = sum_{i>=j} ds_ij q_i.
 * numerator_only != 0: y_i = N_i (dN_i = G_i, dD_i = 0).
 */
void oracle_linattn_backward(const double *q, const double *k, const double *v, const double *dout, double *dq,
                             double *dk, double *dv, int B, int H, int L, int dp, int dvw, int numerator_only) {
    const long nh = (long)B * H;
    const double rd = sqrt((double)dp);
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < nh; ++bh) {
        const double *qh = q + (size_t)bh * L * dp, *kh = k + (size_t)bh * L * dp;
        const double *vh = v + (size_t)bh * L * dvw, *gh = dout + (size_t)bh * L * dvw;
        double *dqh = dq + (size_t)bh * L * dp, *dkh = dk + (size_t)bh * L * dp, *dvh = dv + (size_t)bh * L * dvw;
        double *dN = (double *)malloc(sizeof(double) * (size_t)dvw);
        double *num = (double *)malloc(sizeof(double) * (size_t)dvw);
        memset(dqh, 0, sizeof(double) * (size_t)L * dp);
        memset(dkh, 0, sizeof(double) * (size_t)L * dp);
        memset(dvh, 0, sizeof(double) * (size_t)L * dvw);
        for (int i = 0; i < L; ++i) {
            /* forward quantities of row i */
            double den = ORACLE_EPS;
            for (int c = 0; c < dvw; ++c) num[c] = 0.0;
            for (int j = 0; j <= i; ++j) {
                const double w = taylor_weight(qh + (size_t)i * dp, kh + (size_t)j * dp, dp);
                den += w;
                for (int c = 0; c < dvw; ++c) num[c] += w * vh[(size_t)j * dvw + c];
            }
            double dD = 0.0;
            for (int c = 0; c < dvw; ++c) {
                const double g = gh[(size_t)i * dvw + c];
                if (numerator_only) dN[c] = g;
                else {
                    dN[c] = g / den;
                    dD -= g * (num[c] / den) / den;
                }
            }
            for (int j = 0; j <= i; ++j) {
                double sij = 0.0;
                for (int m = 0; m < dp; ++m) sij += qh[(size_t)i * dp + m] * kh[(size_t)j * dp + m];
                const double w = 1.0 + sij / rd + sij * sij / (2.0 * (double)dp);
                double dw = dD;
                for (int c = 0; c < dvw; ++c) {
                    dw += dN[c] * vh[(size_t)j * dvw + c];
                    dvh[(size_t)j * dvw + c] += w * dN[c];
                }
                const double ds = dw * (1.0 / rd + sij / (double)dp);
                for (int m = 0; m < dp; ++m) {
                    dqh[(size_t)i * dp + m] += ds * kh[(size_t)j * dp + m];
                    dkh[(size_t)j * dp + m] += ds * qh[(size_t)i * dp + m];
                }
            }
        }
        free(dN);
        free(num);
    }
}
