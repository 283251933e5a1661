/*
 * CPU ORACLE for the DEER-GRU hot path -- TEST INFRASTRUCTURE, not product code.
 *
 * Plain, slow, sequential loops; no blocking, fusion or reordering beyond what
 * the definitions state.  This file is included twice by deer_oracle.c, once
 * with REAL = double (suffix _f64: ground truth) and once with REAL = float
 * (suffix _f32: "the sequential fp32 trajectory" of the acceptance criterion).
 * It shares no code with the CUDA library.
 *
 * Conventions (0-based): y[b][t] = f(y[b][t-1], x[b][t]), y[b][-1] = y0[b];
 * all arrays row-major; gate order (r, z, n) along the packed 3n axis.
 *
 * Every function below is pinned by the CPU test-suite against something
 * other than itself (closed forms, brute-force products, finite differences,
 * the fixed-point property): see each header.
 */

#define CAT2(a, b) a##b
#define CAT(a, b) CAT2(a, b)
#define FN(name) CAT(name, SFX)

/* ------------------------------------------------------------------------
 * GRU cell  (Sec. 3.4: y_i = f(y_{i-1}, x_i, theta); Sec. 4.1: f = GRU)
 *   r = sigma(W_ir x + b_ir + W_hr h + b_hr)
 *   z = sigma(W_iz x + b_iz + W_hz h + b_hz)
 *   q = W_hn h + b_hn
 *   c = tanh(W_in x + b_in + r * q)
 *   f = (1 - z) * c + z * h
 * gates (optional, may be NULL) receives r, z, q, c as 4 vectors of n.
 * Pinned by: hand-computed n=1 case; DEER fixed point; finite differences of
 * everything that is derived from it.
 * ------------------------------------------------------------------------ */
static void FN(gru_cell_)(int n, int m, const REAL *W_i, const REAL *W_h,
                          const REAL *b_i, const REAL *b_h, const REAL *h,
                          const REAL *x, REAL *f, REAL *gates)
{
    for (int i = 0; i < n; ++i) {
        REAL ur = b_i[i], uz = b_i[n + i], un = b_i[2 * n + i];
        for (int k = 0; k < m; ++k) {
            ur += W_i[(size_t)i * m + k] * x[k];
            uz += W_i[(size_t)(n + i) * m + k] * x[k];
            un += W_i[(size_t)(2 * n + i) * m + k] * x[k];
        }
        REAL gr = b_h[i], gz = b_h[n + i], gq = b_h[2 * n + i];
        for (int k = 0; k < n; ++k) {
            gr += W_h[(size_t)i * n + k] * h[k];
            gz += W_h[(size_t)(n + i) * n + k] * h[k];
            gq += W_h[(size_t)(2 * n + i) * n + k] * h[k];
        }
        REAL r = (REAL)1 / ((REAL)1 + R_EXP(-(ur + gr)));
        REAL z = (REAL)1 / ((REAL)1 + R_EXP(-(uz + gz)));
        REAL c = R_TANH(un + r * gq);
        f[i] = ((REAL)1 - z) * c + z * h[i];
        if (gates) {
            gates[i] = r; gates[n + i] = z; gates[2 * n + i] = gq; gates[3 * n + i] = c;
        }
    }
}

/* State Jacobian J[i][j] = d f_i / d h_j in closed form (replaces the
 * forward-mode autodiff of App. B.1; G = -J in Eq. 5):
 *   J = diag(z) + diag(a_z) W_hz + diag(a_n r) W_hn + diag(a_n q r (1-r)) W_hr
 *   a_z = (h - c) z (1 - z),  a_n = (1 - z)(1 - c^2)
 * Pinned by central finite differences of gru_cell. */
static void FN(gru_jac_)(int n, const REAL *W_h, const REAL *h, const REAL *gates, REAL *J)
{
    const REAL *r = gates, *z = gates + n, *q = gates + 2 * n, *c = gates + 3 * n;
    for (int i = 0; i < n; ++i) {
        REAL az = (h[i] - c[i]) * z[i] * ((REAL)1 - z[i]);
        REAL an = ((REAL)1 - z[i]) * ((REAL)1 - c[i] * c[i]);
        REAL kr = an * q[i] * r[i] * ((REAL)1 - r[i]);
        REAL kn = an * r[i];
        for (int j = 0; j < n; ++j) {
            REAL v = kr * W_h[(size_t)i * n + j] + az * W_h[(size_t)(n + i) * n + j]
                   + kn * W_h[(size_t)(2 * n + i) * n + j];
            if (i == j) v += z[i];
            J[(size_t)i * n + j] = v;
        }
    }
}

/* Affine test cell f(h, x) = M h + x  (m == n): Newton solves it in one
 * body (Sec. 3.1 / App. A.1).  params: W_h = M [n,n]; others unused. */
static void FN(affine_cell_)(int n, const REAL *M, const REAL *h, const REAL *x, REAL *f)
{
    for (int i = 0; i < n; ++i) {
        REAL s = x[i];
        for (int k = 0; k < n; ++k) s += M[(size_t)i * n + k] * h[k];
        f[i] = s;
    }
}

/* ------------------------------------------------------------------------
 * O-1  Sequential evaluation (the definition of the result, Sec. 3.4).
 * ------------------------------------------------------------------------ */
void FN(oracle_gru_seq_)(int n, int m, const REAL *W_i, const REAL *W_h, const REAL *b_i,
                         const REAL *b_h, const REAL *x, const REAL *y0, int B, int T, REAL *y)
{
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b) {
        const REAL *h = y0 + (size_t)b * n;
        for (int t = 0; t < T; ++t) {
            REAL *out = y + ((size_t)b * T + t) * n;
            FN(gru_cell_)(n, m, W_i, W_h, b_i, b_h, h, x + ((size_t)b * T + t) * m, out, NULL);
            h = out;
        }
    }
}

/* Cell value, gates and Jacobian at given (h_prev, x) for every row of a
 * flat list of N positions (used by tests to check the CUDA cell kernel). */
void FN(oracle_gru_cell_jac_)(int n, int m, const REAL *W_i, const REAL *W_h, const REAL *b_i,
                              const REAL *b_h, const REAL *hprev, const REAL *x, long N,
                              REAL *f, REAL *J)
{
    REAL *gates = (REAL *)malloc(sizeof(REAL) * 4 * (size_t)n);
    for (long e = 0; e < N; ++e) {
        FN(gru_cell_)(n, m, W_i, W_h, b_i, b_h, hprev + e * n, x + e * m, f + e * n, gates);
        if (J) FN(gru_jac_)(n, W_h, hprev + e * n, gates, J + e * n * n);
    }
    free(gates);
}

/* ------------------------------------------------------------------------
 * O-2  Sequential linear recurrence (Eq. 10 with J = -G):
 *   forward : y[t] = J[t] y[t-1] + b[t],            y[-1] = y0 (NULL -> 0)
 *   reverse : y[t] = b[t] + J[t+1]^T y[t+1],        y[T-1] = b[T-1] (+ y0)
 * The reverse form is the adjoint of the forward solve with respect to b
 * (the dual operator of Sec. 3.1.1).  Pinned by the closed form for J = a I,
 * brute-force products for T <= 8 and the adjoint identity.
 * ------------------------------------------------------------------------ */
void FN(oracle_linrec_)(const REAL *J, const REAL *b, const REAL *y0, int B, int T, int n,
                        int reverse, REAL *y)
{
    for (int s = 0; s < B; ++s) {
        const REAL *Js = J + (size_t)s * T * n * n;
        const REAL *bs = b + (size_t)s * T * n;
        REAL *ys = y + (size_t)s * T * n;
        if (!reverse) {
            for (int t = 0; t < T; ++t)
                for (int i = 0; i < n; ++i) {
                    REAL acc = bs[(size_t)t * n + i];
                    for (int k = 0; k < n; ++k) {
                        REAL prev = (t == 0) ? (y0 ? y0[(size_t)s * n + k] : (REAL)0)
                                             : ys[(size_t)(t - 1) * n + k];
                        acc += Js[((size_t)t * n + i) * n + k] * prev;
                    }
                    ys[(size_t)t * n + i] = acc;
                }
        } else {
            for (int t = T - 1; t >= 0; --t)
                for (int i = 0; i < n; ++i) {
                    REAL acc = bs[(size_t)t * n + i];
                    if (t == T - 1) {
                        if (y0) acc += y0[(size_t)s * n + i];
                    } else {
                        for (int k = 0; k < n; ++k)   /* (J[t+1]^T y[t+1])_i */
                            acc += Js[((size_t)(t + 1) * n + k) * n + i] * ys[(size_t)(t + 1) * n + k];
                    }
                    ys[(size_t)t * n + i] = acc;
                }
        }
    }
}

/* ------------------------------------------------------------------------
 * A second cell behind the same interface (Sec. 3.4: any y_i = f(y_{i-1}, x_i, theta)): LSTM with k units,
 * state s = [h; c] of 2k components, gates in the order (i, f, g, o):
 *   a = W_i x + b + W_h h   (4k rows),  i = sigma(a_i), f = sigma(a_f), g = tanh(a_g), o = sigma(a_o)
 *   c' = f * c + i * g,     h' = o * tanh(c'),     f(s, x) = [h'; c']
 * Closed-form state Jacobian (rows: h' then c'; columns: h then c):
 *   dc'/dc = diag(f),  dc'/dh = diag(c f(1-f)) W_hf + diag(g i(1-i)) W_hi + diag(i (1-g^2)) W_hg
 *   dh'/dc = diag(o (1 - tanh^2 c')) dc'/dc,  dh'/dh = diag(tanh(c') o(1-o)) W_ho + diag(o (1 - tanh^2 c')) dc'/dh
 * Pinned by: a library LSTM, central differences, the DEER fixed point.
 * ------------------------------------------------------------------------ */
static void FN(lstm_cell_)(int k, int m, const REAL *W_i, const REAL *W_h, const REAL *b, const REAL *s,
                           const REAL *x, REAL *out, REAL *J)
{
    const REAL *h = s, *c = s + k;
    for (int u = 0; u < k; ++u) {
        REAL a[4];
        for (int q = 0; q < 4; ++q) {
            REAL acc = b[q * k + u];
            for (int j = 0; j < m; ++j) acc += W_i[(size_t)(q * k + u) * m + j] * x[j];
            for (int j = 0; j < k; ++j) acc += W_h[(size_t)(q * k + u) * k + j] * h[j];
            a[q] = acc;
        }
        REAL gi = (REAL)1 / ((REAL)1 + R_EXP(-a[0])), gf = (REAL)1 / ((REAL)1 + R_EXP(-a[1]));
        REAL gg = R_TANH(a[2]), go = (REAL)1 / ((REAL)1 + R_EXP(-a[3]));
        REAL cn = gf * c[u] + gi * gg;
        REAL tc = R_TANH(cn);
        out[u] = go * tc;
        out[k + u] = cn;
        if (J) {
            const int n = 2 * k;
            REAL dti = gg * gi * ((REAL)1 - gi), dtf = c[u] * gf * ((REAL)1 - gf), dtg = gi * ((REAL)1 - gg * gg);
            REAL dho = tc * go * ((REAL)1 - go), dhc = go * ((REAL)1 - tc * tc);
            for (int j = 0; j < k; ++j) {
                REAL dcdh = dti * W_h[(size_t)(0 * k + u) * k + j] + dtf * W_h[(size_t)(1 * k + u) * k + j]
                          + dtg * W_h[(size_t)(2 * k + u) * k + j];
                J[(size_t)(k + u) * n + j] = dcdh;
                J[(size_t)u * n + j] = dho * W_h[(size_t)(3 * k + u) * k + j] + dhc * dcdh;
                J[(size_t)(k + u) * n + k + j] = (j == u) ? gf : (REAL)0;
                J[(size_t)u * n + k + j] = (j == u) ? dhc * gf : (REAL)0;
            }
        }
    }
}

void FN(oracle_lstm_seq_)(int k, int m, const REAL *W_i, const REAL *W_h, const REAL *b, const REAL *x,
                          const REAL *s0, int B, int T, REAL *y)
{
#pragma omp parallel for schedule(static)
    for (int bb = 0; bb < B; ++bb) {
        const REAL *s = s0 + (size_t)bb * 2 * k;
        for (int t = 0; t < T; ++t) {
            REAL *out = y + ((size_t)bb * T + t) * 2 * k;
            FN(lstm_cell_)(k, m, W_i, W_h, b, s, x + ((size_t)bb * T + t) * m, out, NULL);
            s = out;
        }
    }
}

void FN(oracle_lstm_cell_jac_)(int k, int m, const REAL *W_i, const REAL *W_h, const REAL *b, const REAL *sprev,
                               const REAL *x, long N, REAL *f, REAL *J)
{
    for (long e = 0; e < N; ++e)
        FN(lstm_cell_)(k, m, W_i, W_h, b, sprev + e * 2 * k, x + e * m, f + e * 2 * k, J ? J + e * 4 * k * k : NULL);
}

/* ------------------------------------------------------------------------
 * O-3  DEER / Newton iteration, in the order of the paper's iteration body
 * (Eq. 3 with Eq. 5; App. B.1): shift, Jacobian, f, rhs = f - J y_prev,
 * linear solve, err = max|y_new - y|, k += 1; repeat while err > tol and
 * k < max_iter.  One global err over the whole batch.
 *   cell   : 0 = GRU, 1 = affine test cell (W_h = M, x added), 2 = LSTM (n = 2k state components,
 *            W_i [4k,m], W_h [4k,k], b_i [4k] the bias; b_h unused)
 *   form   : 0 = paper's form above; 1 = Newton-update (residual) form of
 *            App. A.1: delta = L_J^{-1}[f - y], y += delta
 *   y      : in = initial guess, out = last iterate
 *   trace  : optional [max_iter] err after each body
 *   yhist  : optional [max_iter][B*T*n] iterates after each body
 * Returns the number of executed bodies.
 * Pinned by: equals the sequential trajectory; affine cell exact after one
 * body; prefix-exactness after k bodies; quadratic error decay.
 * ------------------------------------------------------------------------ */
int FN(oracle_deer_)(int cell, int form, int n, int m, const REAL *W_i, const REAL *W_h,
                     const REAL *b_i, const REAL *b_h, const REAL *x, const REAL *y0, int B,
                     int T, REAL tol, int max_iter, REAL *y, REAL *err_out, REAL *trace,
                     REAL *yhist)
{
    size_t N = (size_t)B * T;
    REAL *J = (REAL *)malloc(sizeof(REAL) * N * n * n);
    REAL *rhs = (REAL *)malloc(sizeof(REAL) * N * n);
    REAL *ynew = (REAL *)malloc(sizeof(REAL) * N * n);
    REAL *gates = (REAL *)malloc(sizeof(REAL) * 4 * (size_t)n);
    REAL *fv = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL err = (REAL)1e10;
    int k = 0;
    while (err > tol && k < max_iter) {
        for (int s = 0; s < B; ++s)
            for (int t = 0; t < T; ++t) {
                size_t e = (size_t)s * T + t;
                const REAL *hp = (t == 0) ? y0 + (size_t)s * n : y + (e - 1) * n;   /* shifter */
                REAL *Je = J + e * n * n;
                if (cell == 0) {
                    FN(gru_cell_)(n, m, W_i, W_h, b_i, b_h, hp, x + e * m, fv, gates);
                    FN(gru_jac_)(n, W_h, hp, gates, Je);
                } else if (cell == 2) {
                    FN(lstm_cell_)(n / 2, m, W_i, W_h, b_i, hp, x + e * m, fv, Je);
                } else {
                    FN(affine_cell_)(n, W_h, hp, x + e * m, fv);
                    for (int i = 0; i < n * n; ++i) Je[i] = W_h[i];
                }
                for (int i = 0; i < n; ++i) {
                    if (form == 0) {             /* rhs = f + G y_prev, G = -J */
                        REAL acc = fv[i];
                        for (int j = 0; j < n; ++j) acc -= Je[(size_t)i * n + j] * hp[j];
                        rhs[e * n + i] = acc;
                    } else {                     /* residual f - y */
                        rhs[e * n + i] = fv[i] - y[e * n + i];
                    }
                }
            }
        if (form == 0) {
            FN(oracle_linrec_)(J, rhs, y0, B, T, n, 0, ynew);
        } else {
            FN(oracle_linrec_)(J, rhs, NULL, B, T, n, 0, ynew);   /* delta, zero start */
            for (size_t i = 0; i < N * n; ++i) ynew[i] += y[i];
        }
        err = (REAL)0;
        for (size_t i = 0; i < N * n; ++i) {
            REAL d = R_ABS(ynew[i] - y[i]);
            if (d > err || d != d) err = d;      /* a NaN sticks, like a plain max */
            y[i] = ynew[i];
        }
        if (trace) trace[k] = err;
        if (yhist) memcpy(yhist + (size_t)k * N * n, y, sizeof(REAL) * N * n);
        ++k;
    }
    if (err_out) *err_out = err;
    free(J); free(rhs); free(ynew); free(gates); free(fv);
    return k;
}

/* ------------------------------------------------------------------------
 * O-4  Back-propagation through time (textbook reverse loop) for
 * L with dL/dy = gy [B,T,n].  Outputs are overwritten.  y is the forward
 * trajectory (so that a gradient can be taken at any given trajectory).
 * Pinned by central finite differences of the sequential loss.
 * ------------------------------------------------------------------------ */
static void FN(gru_cell_vjp_)(int n, int m, const REAL *W_i, const REAL *W_h, const REAL *b_i,
                              const REAL *b_h, const REAL *h, const REAL *x, const REAL *lam,
                              REAL *dW_i, REAL *dW_h, REAL *db_i, REAL *db_h, REAL *dx,
                              REAL *dh, REAL *scratch /* 4n gates + n f + 6n dG */)
{
    REAL *gates = scratch, *fv = scratch + 4 * n, *dGi = scratch + 5 * n, *dGh = scratch + 8 * n;
    FN(gru_cell_)(n, m, W_i, W_h, b_i, b_h, h, x, fv, gates);
    const REAL *r = gates, *z = gates + n, *q = gates + 2 * n, *c = gates + 3 * n;
    for (int i = 0; i < n; ++i) {
        REAL dc = lam[i] * ((REAL)1 - z[i]);             /* f = (1-z) c + z h */
        REAL dz = lam[i] * (h[i] - c[i]);
        REAL dan = dc * ((REAL)1 - c[i] * c[i]);          /* c = tanh(a_n), a_n = u_n + r q */
        REAL dr = dan * q[i];
        REAL dq = dan * r[i];
        REAL dar = dr * r[i] * ((REAL)1 - r[i]);
        REAL daz = dz * z[i] * ((REAL)1 - z[i]);
        dGi[i] = dar; dGi[n + i] = daz; dGi[2 * n + i] = dan;
        dGh[i] = dar; dGh[n + i] = daz; dGh[2 * n + i] = dq;
        dh[i] = lam[i] * z[i];
    }
    for (int g = 0; g < 3 * n; ++g) {
        db_i[g] += dGi[g];
        db_h[g] += dGh[g];
        for (int k = 0; k < m; ++k) dW_i[(size_t)g * m + k] += dGi[g] * x[k];
        for (int k = 0; k < n; ++k) dW_h[(size_t)g * n + k] += dGh[g] * h[k];
    }
    if (dx)
        for (int k = 0; k < m; ++k) {
            REAL s = 0;
            for (int g = 0; g < 3 * n; ++g) s += W_i[(size_t)g * m + k] * dGi[g];
            dx[k] = s;
        }
    for (int k = 0; k < n; ++k) {
        REAL s = 0;
        for (int g = 0; g < 3 * n; ++g) s += W_h[(size_t)g * n + k] * dGh[g];
        dh[k] += s;
    }
}

void FN(oracle_gru_bptt_)(int n, int m, const REAL *W_i, const REAL *W_h, const REAL *b_i,
                          const REAL *b_h, const REAL *x, const REAL *y0, const REAL *y,
                          const REAL *gy, int B, int T, REAL *dW_i, REAL *dW_h, REAL *db_i,
                          REAL *db_h, REAL *dx, REAL *dy0)
{
    memset(dW_i, 0, sizeof(REAL) * 3 * (size_t)n * m);
    memset(dW_h, 0, sizeof(REAL) * 3 * (size_t)n * n);
    memset(db_i, 0, sizeof(REAL) * 3 * (size_t)n);
    memset(db_h, 0, sizeof(REAL) * 3 * (size_t)n);
    REAL *lam = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *dh = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *scratch = (REAL *)malloc(sizeof(REAL) * 11 * (size_t)n);
    for (int s = 0; s < B; ++s) {
        for (int i = 0; i < n; ++i) lam[i] = 0;
        for (int t = T - 1; t >= 0; --t) {
            size_t e = (size_t)s * T + t;
            for (int i = 0; i < n; ++i) lam[i] += gy[e * n + i];
            const REAL *hp = (t == 0) ? y0 + (size_t)s * n : y + (e - 1) * n;
            FN(gru_cell_vjp_)(n, m, W_i, W_h, b_i, b_h, hp, x + e * m, lam, dW_i, dW_h, db_i,
                              db_h, dx ? dx + e * m : NULL, dh, scratch);
            for (int i = 0; i < n; ++i) lam[i] = dh[i];
        }
        if (dy0) for (int i = 0; i < n; ++i) dy0[(size_t)s * n + i] = lam[i];
    }
    free(lam); free(dh); free(scratch);
}

/* DEER gradient (Eq. 7): lambda = gy L_G^{-1} through ONE reverse linear
 * solve with the Jacobians at the given trajectory, then the cell's
 * vector-Jacobian product at every position, summed over positions.
 * Must equal BPTT (tests assert it). */
void FN(oracle_deer_grad_)(int n, int m, const REAL *W_i, const REAL *W_h, const REAL *b_i,
                           const REAL *b_h, const REAL *x, const REAL *y0, const REAL *y,
                           const REAL *gy, int B, int T, REAL *dW_i, REAL *dW_h, REAL *db_i,
                           REAL *db_h, REAL *dx, REAL *dy0, REAL *lam_out)
{
    size_t N = (size_t)B * T;
    REAL *J = (REAL *)malloc(sizeof(REAL) * N * n * n);
    REAL *lam = lam_out ? lam_out : (REAL *)malloc(sizeof(REAL) * N * n);
    REAL *gates = (REAL *)malloc(sizeof(REAL) * 4 * (size_t)n);
    REAL *fv = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *dh = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *scratch = (REAL *)malloc(sizeof(REAL) * 11 * (size_t)n);
    for (int s = 0; s < B; ++s)
        for (int t = 0; t < T; ++t) {
            size_t e = (size_t)s * T + t;
            const REAL *hp = (t == 0) ? y0 + (size_t)s * n : y + (e - 1) * n;
            FN(gru_cell_)(n, m, W_i, W_h, b_i, b_h, hp, x + e * m, fv, gates);
            FN(gru_jac_)(n, W_h, hp, gates, J + e * n * n);
        }
    FN(oracle_linrec_)(J, gy, NULL, B, T, n, 1, lam);
    memset(dW_i, 0, sizeof(REAL) * 3 * (size_t)n * m);
    memset(dW_h, 0, sizeof(REAL) * 3 * (size_t)n * n);
    memset(db_i, 0, sizeof(REAL) * 3 * (size_t)n);
    memset(db_h, 0, sizeof(REAL) * 3 * (size_t)n);
    for (int s = 0; s < B; ++s)
        for (int t = 0; t < T; ++t) {
            size_t e = (size_t)s * T + t;
            const REAL *hp = (t == 0) ? y0 + (size_t)s * n : y + (e - 1) * n;
            FN(gru_cell_vjp_)(n, m, W_i, W_h, b_i, b_h, hp, x + e * m, lam + e * n, dW_i, dW_h,
                              db_i, db_h, dx ? dx + e * m : NULL, dh, scratch);
            if (t == 0 && dy0) for (int i = 0; i < n; ++i) dy0[(size_t)s * n + i] = dh[i];
        }
    free(J); if (!lam_out) free(lam); free(gates); free(fv); free(dh); free(scratch);
}

/* ------------------------------------------------------------------------
 * O-5  Long-series classifier: two stacked GRU layers (layer 2 reads layer
 * 1's output), mean over t of the layer-2 states, linear head, softmax
 * cross-entropy averaged over the batch; sequential forward and BPTT.
 * (App. B.3: mean over the sequence, then a decoder to 5 classes.)
 * Gradient arrays are overwritten.  Pinned by finite differences.
 * ------------------------------------------------------------------------ */
REAL FN(oracle_classifier_)(int n, int m, int ncls, const REAL *W_i1, const REAL *W_h1,
                            const REAL *b_i1, const REAL *b_h1, const REAL *W_i2,
                            const REAL *W_h2, const REAL *b_i2, const REAL *b_h2,
                            const REAL *W_o, const REAL *b_o, const REAL *x, const int *labels,
                            int B, int T, int want_grad, REAL *dW_i1, REAL *dW_h1, REAL *db_i1,
                            REAL *db_h1, REAL *dW_i2, REAL *dW_h2, REAL *db_i2, REAL *db_h2,
                            REAL *dW_o, REAL *db_o, REAL *y1_out, REAL *y2_out)
{
    size_t N = (size_t)B * T;
    REAL *y0 = (REAL *)calloc((size_t)B * n, sizeof(REAL));
    REAL *y1 = y1_out ? y1_out : (REAL *)malloc(sizeof(REAL) * N * n);
    REAL *y2 = y2_out ? y2_out : (REAL *)malloc(sizeof(REAL) * N * n);
    FN(oracle_gru_seq_)(n, m, W_i1, W_h1, b_i1, b_h1, x, y0, B, T, y1);
    FN(oracle_gru_seq_)(n, n, W_i2, W_h2, b_i2, b_h2, y1, y0, B, T, y2);
    REAL *pool = (REAL *)calloc((size_t)B * n, sizeof(REAL));
    REAL *dlog = (REAL *)malloc(sizeof(REAL) * (size_t)B * ncls);
    REAL loss = 0;
    for (int s = 0; s < B; ++s) {
        for (int t = 0; t < T; ++t)
            for (int i = 0; i < n; ++i) pool[(size_t)s * n + i] += y2[((size_t)s * T + t) * n + i];
        for (int i = 0; i < n; ++i) pool[(size_t)s * n + i] /= (REAL)T;
        REAL mx = 0;
        for (int c = 0; c < ncls; ++c) {
            REAL l = b_o[c];
            for (int i = 0; i < n; ++i) l += W_o[(size_t)c * n + i] * pool[(size_t)s * n + i];
            dlog[(size_t)s * ncls + c] = l;
            if (c == 0 || l > mx) mx = l;
        }
        REAL se = 0;
        for (int c = 0; c < ncls; ++c) se += R_EXP(dlog[(size_t)s * ncls + c] - mx);
        REAL lse = mx + R_LOG(se);
        loss += lse - dlog[(size_t)s * ncls + labels[s]];
        for (int c = 0; c < ncls; ++c) {
            REAL p = R_EXP(dlog[(size_t)s * ncls + c] - lse);
            dlog[(size_t)s * ncls + c] = (p - (c == labels[s] ? (REAL)1 : (REAL)0)) / (REAL)B;
        }
    }
    loss /= (REAL)B;
    if (want_grad) {
        memset(dW_o, 0, sizeof(REAL) * (size_t)ncls * n);
        memset(db_o, 0, sizeof(REAL) * (size_t)ncls);
        REAL *gy2 = (REAL *)malloc(sizeof(REAL) * N * n);
        REAL *gy1 = (REAL *)malloc(sizeof(REAL) * N * n);
        for (int s = 0; s < B; ++s) {
            for (int c = 0; c < ncls; ++c) {
                db_o[c] += dlog[(size_t)s * ncls + c];
                for (int i = 0; i < n; ++i)
                    dW_o[(size_t)c * n + i] += dlog[(size_t)s * ncls + c] * pool[(size_t)s * n + i];
            }
            for (int i = 0; i < n; ++i) {
                REAL g = 0;
                for (int c = 0; c < ncls; ++c) g += W_o[(size_t)c * n + i] * dlog[(size_t)s * ncls + c];
                g /= (REAL)T;
                for (int t = 0; t < T; ++t) gy2[((size_t)s * T + t) * n + i] = g;
            }
        }
        FN(oracle_gru_bptt_)(n, n, W_i2, W_h2, b_i2, b_h2, y1, y0, y2, gy2, B, T, dW_i2, dW_h2,
                             db_i2, db_h2, gy1, NULL);
        FN(oracle_gru_bptt_)(n, m, W_i1, W_h1, b_i1, b_h1, x, y0, y1, gy1, B, T, dW_i1, dW_h1,
                             db_i1, db_h1, NULL, NULL);
        free(gy2); free(gy1);
    }
    free(y0); if (!y1_out) free(y1); if (!y2_out) free(y2); free(pool); free(dlog);
    return loss;
}

/* ------------------------------------------------------------------------
 * O-7  Forward-mode derivative (Sec. 3.1.1, the forward derivative equation:
 * dy = L_G^{-1}[ (df/dtheta) dtheta ], likewise for x): the first-order
 * change of the trajectory under a change (dW_i, dW_h, db_i, db_h) of the
 * parameters, dx [B,T,m] of the inputs and dy0 [B,n] of the initial state,
 * written out as the sequential tangent recurrence
 *     dy[t] = J[t] dy[t-1] + df[t],   dy[-1] = dy0,
 * with df[t] the cell's first-order change at fixed y[t-1]:
 *     da_r = dW_ir x + W_ir dx + db_ir + dW_hr h + db_hr      (same for z)
 *     dq   = dW_hn h + db_hn,       du_n = dW_in x + W_in dx + db_in
 *     dr = r (1-r) da_r,  dz = z (1-z) da_z,  dc = (1-c^2)(du_n + dr q + r dq)
 *     df = (1-z) dc + (h - c) dz
 * Any of the tangent arrays may be NULL (= zero).  y is the trajectory.
 * Pinned by central finite differences of oracle_gru_seq along the direction.
 * ------------------------------------------------------------------------ */
void FN(oracle_gru_jvp_)(int n, int m, const REAL *W_i, const REAL *W_h, const REAL *b_i,
                         const REAL *b_h, const REAL *dW_i, const REAL *dW_h, const REAL *db_i,
                         const REAL *db_h, const REAL *x, const REAL *dx, const REAL *y0,
                         const REAL *dy0, const REAL *y, int B, int T, REAL *dy)
{
    REAL *gates = (REAL *)malloc(sizeof(REAL) * 4 * (size_t)n);
    REAL *fv = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *J = (REAL *)malloc(sizeof(REAL) * (size_t)n * n);
    for (int s = 0; s < B; ++s)
        for (int t = 0; t < T; ++t) {
            size_t e = (size_t)s * T + t;
            const REAL *h = (t == 0) ? y0 + (size_t)s * n : y + (e - 1) * n;
            const REAL *xe = x + e * m;
            FN(gru_cell_)(n, m, W_i, W_h, b_i, b_h, h, xe, fv, gates);
            FN(gru_jac_)(n, W_h, h, gates, J);
            const REAL *r = gates, *z = gates + n, *q = gates + 2 * n, *c = gates + 3 * n;
            for (int i = 0; i < n; ++i) {
                REAL dar = 0, daz = 0, dun = 0, dq = 0;
                for (int k = 0; k < m; ++k) {
                    if (dW_i) {
                        dar += dW_i[(size_t)i * m + k] * xe[k];
                        daz += dW_i[(size_t)(n + i) * m + k] * xe[k];
                        dun += dW_i[(size_t)(2 * n + i) * m + k] * xe[k];
                    }
                    if (dx) {
                        dar += W_i[(size_t)i * m + k] * dx[e * m + k];
                        daz += W_i[(size_t)(n + i) * m + k] * dx[e * m + k];
                        dun += W_i[(size_t)(2 * n + i) * m + k] * dx[e * m + k];
                    }
                }
                if (db_i) { dar += db_i[i]; daz += db_i[n + i]; dun += db_i[2 * n + i]; }
                if (dW_h)
                    for (int k = 0; k < n; ++k) {
                        dar += dW_h[(size_t)i * n + k] * h[k];
                        daz += dW_h[(size_t)(n + i) * n + k] * h[k];
                        dq += dW_h[(size_t)(2 * n + i) * n + k] * h[k];
                    }
                if (db_h) { dar += db_h[i]; daz += db_h[n + i]; dq += db_h[2 * n + i]; }
                REAL dr = r[i] * ((REAL)1 - r[i]) * dar;
                REAL dz = z[i] * ((REAL)1 - z[i]) * daz;
                REAL dc = ((REAL)1 - c[i] * c[i]) * (dun + dr * q[i] + r[i] * dq);
                REAL acc = ((REAL)1 - z[i]) * dc + (h[i] - c[i]) * dz;            /* df */
                for (int k = 0; k < n; ++k) {
                    REAL dprev = (t == 0) ? (dy0 ? dy0[(size_t)s * n + k] : (REAL)0) : dy[(e - 1) * n + k];
                    acc += J[(size_t)i * n + k] * dprev;
                }
                dy[e * n + i] = acc;
            }
        }
    free(gates); free(fv); free(J);
}

/* ------------------------------------------------------------------------
 * O-8  The linear operator L_G^{-1} of an ODE (Sec. 3.3): dy/dt + G(t) y = z(t),
 * y(t_0) = y0, with G and z given at the time points t_0 < ... < t_{T-1} and
 * taken constant at their MID-POINT values on every interval,
 *     G_i = (G(t_i) + G(t_{i+1})) / 2,   z_i likewise,   D_i = t_{i+1} - t_i,
 *     y_{i+1} = Gbar_i y_i + zbar_i,  Gbar_i = exp(-G_i D_i),  zbar_i = G_i^{-1}(I - Gbar_i) z_i.
 * Both come from ONE matrix exponential of the augmented matrix
 *     exp( [ -G_i D_i   z_i D_i ] )  =  [ Gbar_i  zbar_i ]
 *        ( [     0         0    ] )     [   0       1    ]
 * (an identity of the matrix exponential: it needs no inverse, so singular G is
 * fine), evaluated by scaling and squaring with a Taylor polynomial.
 * y [B,T,n] with y[b][0] = y0[b].  Optionally returns Gbar [B,T-1,n,n], zbar [B,T-1,n].
 * Pinned by: scalar closed form, a library matrix exponential, the exact
 * solution for constant coefficients, second-order convergence for varying
 * ones (App. A.5), G = 0.
 * ------------------------------------------------------------------------ */
static void FN(expm_aug_)(int n, const REAL *G, const REAL *z, REAL D, REAL *Gbar, REAL *zbar, REAL *work /* 3 (n+1)^2 */)
{
    const int m = n + 1;
    REAL *A = work, *P = work + m * m, *Q = work + 2 * m * m;
    REAL norm = 0;
    for (int i = 0; i < m; ++i) {
        REAL rs = 0;
        for (int j = 0; j < m; ++j) {
            REAL v = 0;
            if (i < n) v = (j < n) ? -G[(size_t)i * n + j] * D : z[i] * D;
            A[i * m + j] = v;
            rs += R_ABS(v);
        }
        if (rs > norm) norm = rs;
    }
    int s = 0;
    while (norm > (REAL)0.25 && s < 60) { norm *= (REAL)0.5; ++s; }
    REAL scale = (REAL)1;
    for (int k = 0; k < s; ++k) scale *= (REAL)0.5;
    for (int i = 0; i < m * m; ++i) A[i] *= scale;
    /* Horner: P = I + A (I + A/2 (I + A/3 ( ... (I + A/K)))) */
    const int K = 18;
    for (int i = 0; i < m * m; ++i) P[i] = (i / m == i % m) ? (REAL)1 : (REAL)0;
    for (int k = K; k >= 1; --k) {
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < m; ++j) {
                REAL acc = 0;
                for (int l = 0; l < m; ++l) acc += A[i * m + l] * P[l * m + j];
                Q[i * m + j] = acc / (REAL)k + ((i == j) ? (REAL)1 : (REAL)0);
            }
        for (int i = 0; i < m * m; ++i) P[i] = Q[i];
    }
    for (int k = 0; k < s; ++k) {
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < m; ++j) {
                REAL acc = 0;
                for (int l = 0; l < m; ++l) acc += P[i * m + l] * P[l * m + j];
                Q[i * m + j] = acc;
            }
        for (int i = 0; i < m * m; ++i) P[i] = Q[i];
    }
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j < n; ++j) Gbar[(size_t)i * n + j] = P[i * m + j];
        zbar[i] = P[i * m + n];
    }
}

void FN(oracle_ode_linear_)(const REAL *G, const REAL *z, const REAL *t, const REAL *y0, int B, int T, int n,
                            REAL *y, REAL *Gbar_out, REAL *zbar_out)
{
    REAL *Gm = (REAL *)malloc(sizeof(REAL) * (size_t)n * n);
    REAL *zm = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *Gb = (REAL *)malloc(sizeof(REAL) * (size_t)n * n);
    REAL *zb = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *work = (REAL *)malloc(sizeof(REAL) * 3 * (size_t)(n + 1) * (n + 1));
    for (int b = 0; b < B; ++b) {
        for (int i = 0; i < n; ++i) y[((size_t)b * T) * n + i] = y0[(size_t)b * n + i];
        for (int k = 0; k + 1 < T; ++k) {
            const size_t e = (size_t)b * T + k;
            for (int i = 0; i < n * n; ++i) Gm[i] = (REAL)0.5 * (G[e * n * n + i] + G[(e + 1) * n * n + i]);
            for (int i = 0; i < n; ++i) zm[i] = (REAL)0.5 * (z[e * n + i] + z[(e + 1) * n + i]);
            FN(expm_aug_)(n, Gm, zm, t[k + 1] - t[k], Gb, zb, work);
            for (int i = 0; i < n; ++i) {
                REAL acc = zb[i];
                for (int j = 0; j < n; ++j) acc += Gb[(size_t)i * n + j] * y[e * n + j];
                y[(e + 1) * n + i] = acc;
            }
            if (Gbar_out) memcpy(Gbar_out + ((size_t)b * (T - 1) + k) * n * n, Gb, sizeof(REAL) * (size_t)n * n);
            if (zbar_out) memcpy(zbar_out + ((size_t)b * (T - 1) + k) * n, zb, sizeof(REAL) * (size_t)n);
        }
    }
    free(Gm); free(zm); free(Gb); free(zb); free(work);
}

/* ------------------------------------------------------------------------
 * O-6  Multi-head GRU (Sec. 4.4; App. B.4): H independent GRU heads of hidden
 * size n read the same input x[b][t] (m channels); head h has its own
 * parameters and a stride s_h and advances
 *     y[b][t][h] = f_h(y[b][t - s_h][h], x[b][t]),   y[b][t'][h] = y0[b][h] for t' < 0
 * (a head of stride s is s interleaved sequences).  The unit's output is the
 * heads' states side by side: y [B,T,H,n].  Parameters are stacked per head:
 * W_i [H,3n,m], W_h [H,3n,n], b_i, b_h [H,3n].
 * Pinned by: H = 1, stride 1 equals oracle_gru_seq; a stride-s head equals s
 * interleaved runs of oracle_gru_seq; finite differences for the gradient.
 * ------------------------------------------------------------------------ */
void FN(oracle_multihead_seq_)(int H, int n, int m, const REAL *W_i, const REAL *W_h,
                               const REAL *b_i, const REAL *b_h, const int *stride, const REAL *x,
                               const REAL *y0, int B, int T, REAL *y)
{
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < T; ++t)
            for (int h = 0; h < H; ++h) {
                const int tp = t - stride[h];
                const REAL *hp = tp >= 0 ? y + (((size_t)b * T + tp) * H + h) * n
                                         : y0 + ((size_t)b * H + h) * n;
                FN(gru_cell_)(n, m, W_i + (size_t)h * 3 * n * m, W_h + (size_t)h * 3 * n * n,
                              b_i + (size_t)h * 3 * n, b_h + (size_t)h * 3 * n, hp,
                              x + ((size_t)b * T + t) * m, y + (((size_t)b * T + t) * H + h) * n, NULL);
            }
}

/* Back-propagation through the multi-head unit for dL/dy = gy [B,T,H,n] at the
 * trajectory y: the adjoint of head h flows from t to t - s_h.  Outputs are
 * overwritten; dx [B,T,m] sums the heads' contributions; dy0 [B,H,n]. */
void FN(oracle_multihead_bptt_)(int H, int n, int m, const REAL *W_i, const REAL *W_h,
                                const REAL *b_i, const REAL *b_h, const int *stride, const REAL *x,
                                const REAL *y0, const REAL *y, const REAL *gy, int B, int T,
                                REAL *dW_i, REAL *dW_h, REAL *db_i, REAL *db_h, REAL *dx, REAL *dy0)
{
    size_t N = (size_t)B * T;
    memset(dW_i, 0, sizeof(REAL) * (size_t)H * 3 * n * m);
    memset(dW_h, 0, sizeof(REAL) * (size_t)H * 3 * n * n);
    memset(db_i, 0, sizeof(REAL) * (size_t)H * 3 * n);
    memset(db_h, 0, sizeof(REAL) * (size_t)H * 3 * n);
    memset(dx, 0, sizeof(REAL) * N * m);
    memset(dy0, 0, sizeof(REAL) * (size_t)B * H * n);
    REAL *lam = (REAL *)malloc(sizeof(REAL) * N * H * n);
    memcpy(lam, gy, sizeof(REAL) * N * H * n);
    REAL *dh = (REAL *)malloc(sizeof(REAL) * (size_t)n);
    REAL *dxe = (REAL *)malloc(sizeof(REAL) * (size_t)m);
    REAL *scratch = (REAL *)malloc(sizeof(REAL) * 11 * (size_t)n);
    for (int b = 0; b < B; ++b)
        for (int t = T - 1; t >= 0; --t)
            for (int h = 0; h < H; ++h) {
                const size_t e = (size_t)b * T + t;
                const int tp = t - stride[h];
                const REAL *hp = tp >= 0 ? y + (((size_t)b * T + tp) * H + h) * n
                                         : y0 + ((size_t)b * H + h) * n;
                FN(gru_cell_vjp_)(n, m, W_i + (size_t)h * 3 * n * m, W_h + (size_t)h * 3 * n * n,
                                  b_i + (size_t)h * 3 * n, b_h + (size_t)h * 3 * n, hp, x + e * m,
                                  lam + (e * H + h) * n, dW_i + (size_t)h * 3 * n * m,
                                  dW_h + (size_t)h * 3 * n * n, db_i + (size_t)h * 3 * n,
                                  db_h + (size_t)h * 3 * n, dxe, dh, scratch);
                for (int k = 0; k < m; ++k) dx[e * m + k] += dxe[k];
                REAL *dst = tp >= 0 ? lam + (((size_t)b * T + tp) * H + h) * n
                                    : dy0 + ((size_t)b * H + h) * n;
                for (int i = 0; i < n; ++i) dst[i] += dh[i];
            }
    free(lam); free(dh); free(dxe); free(scratch);
}

#undef FN
#undef CAT
#undef CAT2
