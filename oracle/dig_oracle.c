/*
 * fp64 CPU oracle for the DiG token-mixer hot path (arxiv 2405.18428).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or helper
 * with the CUDA path, and the product never calls it.
 *
 * What is written out here
 *   - gate transform        alpha = sigmoid(x)^(1/tau), kept as a = log(alpha)      (Eq. gate_gla)
 *   - GLA recurrence        S_t = diag(alpha_t) S_{t-1} + k_t^T v_t,  o_t = q_t S_t (Eq. attn_gla,
 *                           with the value-channel gate beta fixed to 1)
 *   - its reverse-mode derivative (not printed in the paper; derived from Eq. attn_gla)
 *   - the four scan orders of the block-by-block scanning scheme (Algorithm 1 / Algorithm 4:
 *     flip and transpose of the reshaped token matrix), materialised as index arrays
 *   - the 3x3 depthwise convolution of the SREM module (Algorithm 1, "DWConv2d(reshape2d(z))"),
 *     evaluated on the re-oriented token matrix by explicit gather / conv / scatter, and its
 *     reverse-mode derivative
 *   - the recurrence started from a given state and returning the final state (the paper starts
 *     from zero and drops it; this is what splitting a sequence into pieces needs), with the
 *     matching terms of the derivative
 *   - the recurrence with the full gate G_t = alpha_t^T beta_t of Eq. gate_gla (value-channel decay
 *     beta as well), and its derivative
 *   - the output gate z = Swish(r) (.) LN(o) that follows the recurrence (Eq. attn_gla, the line
 *     forming Y_t before the projection W_O), and its reverse-mode derivative
 *
 * Everything is token-by-token and element-by-element: no chunking, no blocking, no fused forms.
 * Tensors are dense row-major doubles with layout [B][L][H][d]; L = grid_h*grid_w and the
 * canonical token index is y*grid_w + x.
 *
 * Pins (tests/test_oracle_*.py): brute-force parallel form, reduction to causal linear
 * attention (Eq. attn_simple) when alpha == 1, constant-decay closed form, fast-decay limit,
 * permutation bijectivity and the four-block cycle, central finite differences for the
 * backward pass, the suffix-sum gate-gradient identity, identity-initialised convolution,
 * convolution against hand-evaluated corner / edge / interior counts; for the convolution's
 * derivative: central finite differences, the adjoint identity <dy, conv(x)> = <dx, x>, and
 * dw of an identity-initialised filter on a one-pixel image; for the output gate: a library
 * layer-norm and silu on the same rows, zero-mean / unit-variance and shift-scale invariance of
 * the normalisation, Swish's values at 0 and far from 0, central finite differences of the
 * derivative, and do summing to zero over a row when the affine part is absent; for the state
 * arguments: a sequence cut in two and chained through the state equals the uncut one (values and
 * all gradients), the final state of a constant-decay sequence in closed form, finite differences;
 * for the value-channel gate: beta == 1 gives the alpha-only recurrence back, the parallel form
 * o_t = sum_{s<=t} (q_t e^{Lam_t} . k_s e^{-Lam_s}) v_s e^{M_t - M_s} written out in numpy, finite
 * differences, and the suffix-sum identity d(log beta)_t = sum_{s>=t} (o_s do_s - v_s dv_s).
 * Not pinned by the paper: whether DWConv2d carries a bias (the argument is optional).
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

/* direction codes: 0 row-major forward, 1 row-major reverse, 2 column-major forward,
 * 3 column-major reverse */

/* perm[p] = canonical token visited at scan position p.
 * Built the way Algorithm 1 builds the orders: start from the row-major sequence; "flip"
 * reverses a sequence; "transpose" reshapes to 2-D, transposes and flattens. */
int dig_oracle_perm(int direction, int grid_h, int grid_w, long long *perm)
{
    const long long L = (long long)grid_h * grid_w;
    if (direction < 0 || direction > 3 || grid_h <= 0 || grid_w <= 0) return 1;
    long long *seq = (long long *)malloc(sizeof(long long) * (size_t)L);
    if (!seq) return 2;
    for (long long t = 0; t < L; ++t) seq[t] = t;           /* row-major forward */
    if (direction == 2 || direction == 3) {
        /* transpose(reshape2d(seq)): new matrix has grid_w rows and grid_h columns */
        for (int x = 0; x < grid_w; ++x)
            for (int y = 0; y < grid_h; ++y)
                perm[(long long)x * grid_h + y] = seq[(long long)y * grid_w + x];
        memcpy(seq, perm, sizeof(long long) * (size_t)L);
    }
    if (direction == 1 || direction == 3) {
        for (long long p = 0; p < L; ++p) perm[p] = seq[L - 1 - p];  /* flip */
    } else {
        memcpy(perm, seq, sizeof(long long) * (size_t)L);
    }
    free(seq);
    return 0;
}

/* a = log(sigmoid(x)^(1/tau)) = logsigmoid(x)/tau, per head temperature.  (Eq. gate_gla) */
int dig_oracle_gate(const double *x, const double *tau_per_head, double *a,
                    long long B, long long L, int H, int d_k)
{
    for (long long bl = 0; bl < B * L; ++bl)
        for (int h = 0; h < H; ++h)
            for (int c = 0; c < d_k; ++c) {
                const size_t i = ((size_t)bl * H + h) * d_k + c;
                const double z = x[i];
                /* log(1/(1+e^-z)), written so that neither branch overflows */
                const double ls = (z >= 0.0) ? -log1p(exp(-z)) : z - log1p(exp(z));
                a[i] = ls / tau_per_head[h];
            }
    return 0;
}

static size_t tok_off(long long b, long long t, int h, long long L, int H, int d)
{
    return (((size_t)b * L + t) * H + h) * (size_t)d;
}

/* Forward recurrence (Eq. attn_gla), one (b,h) pair at a time, in scan order.
 * s_in (may be NULL = zero, the paper's case): state before the first scan position, [B][H][d_k][d_v];
 * s_out (may be NULL): receives the state after the last scan position, same layout. */
static int gla_fwd_impl(const double *q, const double *k, const double *v, const double *a, const double *bg,
                        double *out, const double *s_in, double *s_out, int B, int H, int grid_h, int grid_w,
                        int d_k, int d_v, int direction, int threads)
{
    const long long L = (long long)grid_h * grid_w;
    long long *perm = (long long *)malloc(sizeof(long long) * (size_t)L);
    if (!perm) return 2;
    if (dig_oracle_perm(direction, grid_h, grid_w, perm)) { free(perm); return 1; }
    int err = 0;
    (void)threads;
#ifdef _OPENMP
#pragma omp parallel for num_threads(threads > 0 ? threads : 1) schedule(dynamic, 1)
#endif
    for (int bh = 0; bh < B * H; ++bh) {
        const int b = bh / H, h = bh % H;
        double *S = (double *)calloc((size_t)d_k * d_v, sizeof(double));
        if (!S) { err = 2; continue; }
        if (s_in) memcpy(S, s_in + (size_t)bh * d_k * d_v, sizeof(double) * (size_t)d_k * d_v);
        for (long long p = 0; p < L; ++p) {
            const long long t = perm[p];
            const double *qt = q + tok_off(b, t, h, L, H, d_k);
            const double *kt = k + tok_off(b, t, h, L, H, d_k);
            const double *at = a + tok_off(b, t, h, L, H, d_k);
            const double *vt = v + tok_off(b, t, h, L, H, d_v);
            double *ot = out + tok_off(b, t, h, L, H, d_v);
            const double *bt = bg ? bg + tok_off(b, t, h, L, H, d_v) : NULL;
            for (int c = 0; c < d_k; ++c) {
                const double al = exp(at[c]);
                for (int e = 0; e < d_v; ++e) {         /* S'_{t-1} = G_t . S_{t-1}, G_t = alpha_t^T beta_t; S_t = S' + k^T v */
                    const double be = bt ? exp(bt[e]) : 1.0;
                    S[(size_t)c * d_v + e] = al * be * S[(size_t)c * d_v + e] + kt[c] * vt[e];
                }
            }
            for (int e = 0; e < d_v; ++e) {             /* o_t = q_t S_t */
                double acc = 0.0;
                for (int c = 0; c < d_k; ++c) acc += qt[c] * S[(size_t)c * d_v + e];
                ot[e] = acc;
            }
        }
        if (s_out) memcpy(s_out + (size_t)bh * d_k * d_v, S, sizeof(double) * (size_t)d_k * d_v);
        free(S);
    }
    free(perm);
    return err;
}

int dig_oracle_gla_fwd(const double *q, const double *k, const double *v, const double *a,
                       double *out, int B, int H, int grid_h, int grid_w, int d_k, int d_v,
                       int direction, int threads)
{
    return gla_fwd_impl(q, k, v, a, NULL, out, NULL, NULL, B, H, grid_h, grid_w, d_k, d_v, direction, threads);
}

/* The same recurrence started from a given state and returning the final one: what a caller needs to
 * split a sequence into pieces (the paper always starts from zero and drops the final state). */
int dig_oracle_gla_fwd_state(const double *q, const double *k, const double *v, const double *a,
                             const double *s_in, double *out, double *s_out, int B, int H, int grid_h,
                             int grid_w, int d_k, int d_v, int direction, int threads)
{
    return gla_fwd_impl(q, k, v, a, NULL, out, s_in, s_out, B, H, grid_h, grid_w, d_k, d_v, direction, threads);
}

/* Reverse-mode derivative of the recurrence above.
 *   dS_t  = q_t^T do_t + diag(alpha_{t+1}) dS_{t+1}          (dS past the end is 0)
 *   dq_t  = S_t do_t^T,  dk_t = dS_t v_t^T,  dv_t = k_t dS_t
 *   da_t[c] = alpha_t[c] * sum_e dS_t[c,e] S_{t-1}[c,e]
 * S_{t-1} and S_t are re-created from checkpoints of the forward state taken every SEG
 * positions, so memory stays small at long L.
 * With a start state s_in (NULL = zero) the forward sweep starts from it; ds_out (NULL = zero) is the
 * gradient with respect to the final state and seeds dS; ds_in (may be NULL) receives the gradient
 * with respect to s_in, which is dS after the first position has handed it on. */
static int gla_bwd_impl(const double *q, const double *k, const double *v, const double *a, const double *bg,
                        const double *dout, const double *s_in, const double *ds_out, double *dq, double *dk,
                        double *dv, double *da, double *db, double *ds_in, int B, int H, int grid_h, int grid_w,
                        int d_k, int d_v, int direction, int threads)
{
    enum { SEG = 64 };
    const long long L = (long long)grid_h * grid_w;
    const size_t SZ = (size_t)d_k * d_v;
    const long long nseg = (L + SEG - 1) / SEG;
    long long *perm = (long long *)malloc(sizeof(long long) * (size_t)L);
    if (!perm) return 2;
    if (dig_oracle_perm(direction, grid_h, grid_w, perm)) { free(perm); return 1; }
    int err = 0;
    (void)threads;
#ifdef _OPENMP
#pragma omp parallel for num_threads(threads > 0 ? threads : 1) schedule(dynamic, 1)
#endif
    for (int bh = 0; bh < B * H; ++bh) {
        const int b = bh / H, h = bh % H;
        double *ckpt = (double *)malloc(sizeof(double) * SZ * (size_t)nseg);   /* state entering each segment */
        double *seg = (double *)malloc(sizeof(double) * SZ * (SEG + 1));       /* seg[j] = state before local step j */
        double *dS = (double *)calloc(SZ, sizeof(double));
        if (!ckpt || !seg || !dS) { err = 2; free(ckpt); free(seg); free(dS); continue; }
        if (ds_out) memcpy(dS, ds_out + SZ * (size_t)bh, sizeof(double) * SZ);
        /* forward sweep, storing checkpoints */
        {
            double *S = (double *)calloc(SZ, sizeof(double));
            if (s_in) memcpy(S, s_in + SZ * (size_t)bh, sizeof(double) * SZ);
            for (long long p = 0; p < L; ++p) {
                if (p % SEG == 0) memcpy(ckpt + SZ * (size_t)(p / SEG), S, sizeof(double) * SZ);
                const long long t = perm[p];
                const double *kt = k + tok_off(b, t, h, L, H, d_k);
                const double *at = a + tok_off(b, t, h, L, H, d_k);
                const double *vt = v + tok_off(b, t, h, L, H, d_v);
                const double *bt = bg ? bg + tok_off(b, t, h, L, H, d_v) : NULL;
                for (int c = 0; c < d_k; ++c) {
                    const double al = exp(at[c]);
                    for (int e = 0; e < d_v; ++e)
                        S[(size_t)c * d_v + e] = al * (bt ? exp(bt[e]) : 1.0) * S[(size_t)c * d_v + e] + kt[c] * vt[e];
                }
            }
            free(S);
        }
        for (long long s = nseg - 1; s >= 0; --s) {
            const long long p0 = s * SEG;
            const long long n = (L - p0 < SEG) ? (L - p0) : SEG;
            memcpy(seg, ckpt + SZ * (size_t)s, sizeof(double) * SZ);
            for (long long j = 0; j < n; ++j) {                     /* seg[j+1] = S_{p0+j} */
                const long long t = perm[p0 + j];
                const double *kt = k + tok_off(b, t, h, L, H, d_k);
                const double *at = a + tok_off(b, t, h, L, H, d_k);
                const double *vt = v + tok_off(b, t, h, L, H, d_v);
                const double *Sp = seg + SZ * (size_t)j;
                double *Sn = seg + SZ * (size_t)(j + 1);
                const double *bt = bg ? bg + tok_off(b, t, h, L, H, d_v) : NULL;
                for (int c = 0; c < d_k; ++c) {
                    const double al = exp(at[c]);
                    for (int e = 0; e < d_v; ++e)
                        Sn[(size_t)c * d_v + e] = al * (bt ? exp(bt[e]) : 1.0) * Sp[(size_t)c * d_v + e] + kt[c] * vt[e];
                }
            }
            for (long long j = n - 1; j >= 0; --j) {
                const long long t = perm[p0 + j];
                const double *qt = q + tok_off(b, t, h, L, H, d_k);
                const double *kt = k + tok_off(b, t, h, L, H, d_k);
                const double *at = a + tok_off(b, t, h, L, H, d_k);
                const double *vt = v + tok_off(b, t, h, L, H, d_v);
                const double *dot = dout + tok_off(b, t, h, L, H, d_v);
                double *dqt = dq + tok_off(b, t, h, L, H, d_k);
                double *dkt = dk + tok_off(b, t, h, L, H, d_k);
                double *dat = da + tok_off(b, t, h, L, H, d_k);
                double *dvt = dv + tok_off(b, t, h, L, H, d_v);
                const double *Sprev = seg + SZ * (size_t)j;         /* S_{t-1} */
                const double *Scur = seg + SZ * (size_t)(j + 1);    /* S_t     */
                for (int c = 0; c < d_k; ++c)
                    for (int e = 0; e < d_v; ++e) dS[(size_t)c * d_v + e] += qt[c] * dot[e];
                const double *bt = bg ? bg + tok_off(b, t, h, L, H, d_v) : NULL;
                double *dbt = db ? db + tok_off(b, t, h, L, H, d_v) : NULL;
                for (int e = 0; e < d_v; ++e) dvt[e] = 0.0;
                if (dbt) for (int e = 0; e < d_v; ++e) dbt[e] = 0.0;
                for (int c = 0; c < d_k; ++c) {
                    const double al = exp(at[c]);
                    double sq = 0.0, sk = 0.0, sa = 0.0;
                    for (int e = 0; e < d_v; ++e) {
                        const double g = dS[(size_t)c * d_v + e];
                        const double be = bt ? exp(bt[e]) : 1.0;
                        sq += Scur[(size_t)c * d_v + e] * dot[e];
                        sk += g * vt[e];
                        sa += g * be * Sprev[(size_t)c * d_v + e];            /* d/d(log alpha) of alpha*beta*S_{t-1} */
                        if (dbt) dbt[e] += g * al * be * Sprev[(size_t)c * d_v + e];   /* d/d(log beta) of the same */
                        dvt[e] += kt[c] * g;
                    }
                    dqt[c] = sq;
                    dkt[c] = sk;
                    dat[c] = al * sa;
                    for (int e = 0; e < d_v; ++e)                                       /* hand dS to step t-1 */
                        dS[(size_t)c * d_v + e] *= al * (bt ? exp(bt[e]) : 1.0);
                }
            }
        }
        if (ds_in) memcpy(ds_in + SZ * (size_t)bh, dS, sizeof(double) * SZ);
        free(ckpt); free(seg); free(dS);
    }
    free(perm);
    return err;
}

int dig_oracle_gla_bwd(const double *q, const double *k, const double *v, const double *a,
                       const double *dout, double *dq, double *dk, double *dv, double *da,
                       int B, int H, int grid_h, int grid_w, int d_k, int d_v,
                       int direction, int threads)
{
    return gla_bwd_impl(q, k, v, a, NULL, dout, NULL, NULL, dq, dk, dv, da, NULL, NULL, B, H, grid_h, grid_w, d_k, d_v,
                        direction, threads);
}

int dig_oracle_gla_bwd_state(const double *q, const double *k, const double *v, const double *a,
                             const double *dout, const double *s_in, const double *ds_out, double *dq,
                             double *dk, double *dv, double *da, double *ds_in, int B, int H, int grid_h,
                             int grid_w, int d_k, int d_v, int direction, int threads)
{
    return gla_bwd_impl(q, k, v, a, NULL, dout, s_in, ds_out, dq, dk, dv, da, NULL, ds_in, B, H, grid_h, grid_w, d_k, d_v,
                        direction, threads);
}

/* The paper's full gate G_t = alpha_t^T beta_t (Eq. gate_gla): the state decays along the key channels
 * by alpha and along the value channels by beta.  bg = log(beta) <= 0, [B][L][H][d_v]. */
int dig_oracle_gla_fwd_beta(const double *q, const double *k, const double *v, const double *a, const double *bg,
                            double *out, int B, int H, int grid_h, int grid_w, int d_k, int d_v, int direction,
                            int threads)
{
    return gla_fwd_impl(q, k, v, a, bg, out, NULL, NULL, B, H, grid_h, grid_w, d_k, d_v, direction, threads);
}

int dig_oracle_gla_bwd_beta(const double *q, const double *k, const double *v, const double *a, const double *bg,
                            const double *dout, double *dq, double *dk, double *dv, double *da, double *db, int B,
                            int H, int grid_h, int grid_w, int d_k, int d_v, int direction, int threads)
{
    return gla_bwd_impl(q, k, v, a, bg, dout, NULL, NULL, dq, dk, dv, da, db, NULL, B, H, grid_h, grid_w, d_k, d_v,
                        direction, threads);
}

/* SREM depthwise convolution (Algorithm 1: DWConv2d(reshape2d(z))).
 * x, y: [B][grid_h*grid_w][D] at canonical token positions.  w: [3][3][D].  bias: [D] or NULL.
 * The residual stream of a block that scans in `direction` is the sequence z[p] = x[perm[p]].
 * reshape2d views it as R x C with (R,C) = (grid_h,grid_w) for the row-major orders and
 * (grid_w,grid_h) for the column-major ones.  The convolution is a 3x3, stride-1,
 * zero-padded cross-correlation on that matrix: tap (u,v) multiplies z2d[i+u-1][j+v-1].
 * The result is scattered back to canonical positions. */
int dig_oracle_dwconv(const double *x, const double *w, const double *bias, double *y,
                      int B, int grid_h, int grid_w, int D, int direction)
{
    const long long L = (long long)grid_h * grid_w;
    long long *perm = (long long *)malloc(sizeof(long long) * (size_t)L);
    if (!perm) return 2;
    if (dig_oracle_perm(direction, grid_h, grid_w, perm)) { free(perm); return 1; }
    const int R = (direction >= 2) ? grid_w : grid_h;
    const int C = (direction >= 2) ? grid_h : grid_w;
    double *z = (double *)malloc(sizeof(double) * (size_t)L * D);
    double *zo = (double *)malloc(sizeof(double) * (size_t)L * D);
    if (!z || !zo) { free(perm); free(z); free(zo); return 2; }
    for (int b = 0; b < B; ++b) {
        const double *xb = x + (size_t)b * L * D;
        double *yb = y + (size_t)b * L * D;
        for (long long p = 0; p < L; ++p)                           /* gather into scan order */
            memcpy(z + (size_t)p * D, xb + (size_t)perm[p] * D, sizeof(double) * (size_t)D);
        for (int i = 0; i < R; ++i)
            for (int j = 0; j < C; ++j)
                for (int ch = 0; ch < D; ++ch) {
                    double acc = bias ? bias[ch] : 0.0;
                    for (int u = 0; u < 3; ++u)
                        for (int vv = 0; vv < 3; ++vv) {
                            const int ii = i + u - 1, jj = j + vv - 1;
                            if (ii < 0 || ii >= R || jj < 0 || jj >= C) continue;
                            acc += w[((size_t)u * 3 + vv) * D + ch] *
                                   z[((size_t)ii * C + jj) * D + ch];
                        }
                    zo[((size_t)i * C + j) * D + ch] = acc;
                }
        for (long long p = 0; p < L; ++p)                           /* scatter back */
            memcpy(yb + (size_t)perm[p] * D, zo + (size_t)p * D, sizeof(double) * (size_t)D);
    }
    free(perm); free(z); free(zo);
    return 0;
}

/* Reverse mode of the SREM depthwise convolution above (the paper trains through the module but
 * does not print its derivative): given dL/dy, returns dL/dx, dL/dw and dL/dbias of
 *     y = DWConv2d(reshape2d(z)) + bias
 * in the same re-oriented layout.  Written as the transpose of the forward loops: every product
 * w[u][v][ch] * z[i+u-1][j+v-1][ch] that contributed to y[i][j][ch] sends dy[i][j][ch] * w back to
 * that input pixel and dy * z to that tap.  dw: [3][3][D], dbias: [D] (may be NULL). */
int dig_oracle_dwconv_bwd(const double *x, const double *w, const double *dy, double *dx, double *dw,
                          double *dbias, int B, int grid_h, int grid_w, int D, int direction)
{
    const long long L = (long long)grid_h * grid_w;
    long long *perm = (long long *)malloc(sizeof(long long) * (size_t)L);
    if (!perm) return 2;
    if (dig_oracle_perm(direction, grid_h, grid_w, perm)) { free(perm); return 1; }
    const int R = (direction >= 2) ? grid_w : grid_h;
    const int C = (direction >= 2) ? grid_h : grid_w;
    double *z = (double *)malloc(sizeof(double) * (size_t)L * D);
    double *g = (double *)malloc(sizeof(double) * (size_t)L * D);
    double *dz = (double *)malloc(sizeof(double) * (size_t)L * D);
    if (!z || !g || !dz) { free(perm); free(z); free(g); free(dz); return 2; }
    memset(dw, 0, sizeof(double) * 9 * (size_t)D);
    if (dbias) memset(dbias, 0, sizeof(double) * (size_t)D);
    for (int b = 0; b < B; ++b) {
        const double *xb = x + (size_t)b * L * D, *gb = dy + (size_t)b * L * D;
        double *dxb = dx + (size_t)b * L * D;
        for (long long p = 0; p < L; ++p) {                         /* gather into scan order */
            memcpy(z + (size_t)p * D, xb + (size_t)perm[p] * D, sizeof(double) * (size_t)D);
            memcpy(g + (size_t)p * D, gb + (size_t)perm[p] * D, sizeof(double) * (size_t)D);
        }
        memset(dz, 0, sizeof(double) * (size_t)L * D);
        for (int i = 0; i < R; ++i)
            for (int j = 0; j < C; ++j)
                for (int ch = 0; ch < D; ++ch) {
                    const double gy = g[((size_t)i * C + j) * D + ch];
                    if (dbias) dbias[ch] += gy;
                    for (int u = 0; u < 3; ++u)
                        for (int vv = 0; vv < 3; ++vv) {
                            const int ii = i + u - 1, jj = j + vv - 1;
                            if (ii < 0 || ii >= R || jj < 0 || jj >= C) continue;
                            dz[((size_t)ii * C + jj) * D + ch] += gy * w[((size_t)u * 3 + vv) * D + ch];
                            dw[((size_t)u * 3 + vv) * D + ch] += gy * z[((size_t)ii * C + jj) * D + ch];
                        }
                }
        for (long long p = 0; p < L; ++p)                           /* scatter back */
            memcpy(dxb + (size_t)perm[p] * D, dz + (size_t)p * D, sizeof(double) * (size_t)D);
    }
    free(perm); free(z); free(g); free(dz);
    return 0;
}

int dig_oracle_has_openmp(void)
{
#ifdef _OPENMP
    return 1;
#else
    return 0;
#endif
}

/* ---- output gate of the GLA layer -------------------------------------------------------------------
 * Eq. attn_gla, the line that forms Y_t before the output projection: per (token, head) row o of
 * length d_v and gate pre-activation r = X_t W_r + b_r of the same length,
 *     z = Swish(r) (.) LN(o),    Swish(r) = r * sigmoid(r),
 *     LN(o)_e = (o_e - mean(o)) / sqrt(var(o) + eps) * ln_w[e] + ln_b[e],
 * mean and (biased) variance over the d_v entries of the row.  The paper does not say what LN
 * normalises over, nor whether it has an affine part or which eps: this reading takes one row per
 * head, an optional affine part shared by all heads (NULL = weight 1 / bias 0) and eps as an
 * argument.  rows = B * L * H. */
int dig_oracle_outgate_fwd(const double *o, const double *r, const double *ln_w, const double *ln_b,
                           double *z, long long rows, int d_v, double eps)
{
    if (rows < 0 || d_v <= 0) return 1;
    for (long long i = 0; i < rows; ++i) {
        const double *oi = o + (size_t)i * d_v, *ri = r + (size_t)i * d_v;
        double mean = 0.0, var = 0.0;
        for (int e = 0; e < d_v; ++e) mean += oi[e];
        mean /= d_v;
        for (int e = 0; e < d_v; ++e) var += (oi[e] - mean) * (oi[e] - mean);
        var /= d_v;
        const double rstd = 1.0 / sqrt(var + eps);
        for (int e = 0; e < d_v; ++e) {
            const double y = (oi[e] - mean) * rstd * (ln_w ? ln_w[e] : 1.0) + (ln_b ? ln_b[e] : 0.0);
            const double sg = 1.0 / (1.0 + exp(-ri[e]));
            z[(size_t)i * d_v + e] = ri[e] * sg * y;
        }
    }
    return 0;
}

/* Reverse mode of the above (not printed in the paper): given dz, the gradients with respect to o, r
 * and the affine part.  With n = (o - mean) * rstd, y = n * w + b, s = Swish(r):
 *   dr = dz * y * s'(r),  s'(r) = sg + r * sg * (1 - sg);   dy = dz * s;
 *   dln_w = sum over rows of dy * n;  dln_b = sum over rows of dy;   dn = dy * w;
 *   do = rstd * (dn - mean(dn) - n * mean(dn * n))   (the derivative of the normalisation). */
int dig_oracle_outgate_bwd(const double *o, const double *r, const double *ln_w, const double *ln_b,
                           const double *dz, double *d_o, double *d_r, double *dln_w, double *dln_b,
                           long long rows, int d_v, double eps)
{
    if (rows < 0 || d_v <= 0) return 1;
    double *n = (double *)malloc(sizeof(double) * (size_t)d_v);
    double *dn = (double *)malloc(sizeof(double) * (size_t)d_v);
    if (!n || !dn) { free(n); free(dn); return 2; }
    if (dln_w) memset(dln_w, 0, sizeof(double) * (size_t)d_v);
    if (dln_b) memset(dln_b, 0, sizeof(double) * (size_t)d_v);
    for (long long i = 0; i < rows; ++i) {
        const double *oi = o + (size_t)i * d_v, *ri = r + (size_t)i * d_v, *gi = dz + (size_t)i * d_v;
        double mean = 0.0, var = 0.0;
        for (int e = 0; e < d_v; ++e) mean += oi[e];
        mean /= d_v;
        for (int e = 0; e < d_v; ++e) var += (oi[e] - mean) * (oi[e] - mean);
        var /= d_v;
        const double rstd = 1.0 / sqrt(var + eps);
        double m1 = 0.0, m2 = 0.0;
        for (int e = 0; e < d_v; ++e) {
            const double w = ln_w ? ln_w[e] : 1.0, b = ln_b ? ln_b[e] : 0.0;
            n[e] = (oi[e] - mean) * rstd;
            const double y = n[e] * w + b;
            const double sg = 1.0 / (1.0 + exp(-ri[e]));
            const double s = ri[e] * sg;
            d_r[(size_t)i * d_v + e] = gi[e] * y * (sg + ri[e] * sg * (1.0 - sg));
            const double dy = gi[e] * s;
            if (dln_w) dln_w[e] += dy * n[e];
            if (dln_b) dln_b[e] += dy;
            dn[e] = dy * w;
            m1 += dn[e];
            m2 += dn[e] * n[e];
        }
        m1 /= d_v;
        m2 /= d_v;
        for (int e = 0; e < d_v; ++e) d_o[(size_t)i * d_v + e] = rstd * (dn[e] - m1 - n[e] * m2);
    }
    free(n);
    free(dn);
    return 0;
}
