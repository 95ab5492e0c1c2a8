/*
 * Float64 CPU oracle for causal Local Linear Attention (LLA).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  Only the tests, the smoke check and the
 * bench's CPU-baseline leg may build or call it; the product library neither
 * links nor imports it and the two share no code.
 *
 * What is computed, per (batch b, head h, query row i), follows the paper's
 * Section 2.3 literally (Eq. "query_specific" and Eq. "lla"):
 *
 *   L      = causal ? i+1 : n            visible keys j = 0..L-1 (the diagonal
 *                                        is included: D_i = {(k_j,v_j)}_{j<=i})
 *   w_j    = exp(scale * <q_i, k_j>)     kernel weight (Section 3.2, W=exp(QK^T/h),
 *                                        scale = 1/h)
 *   z_j    = k_j - q_i
 *   omega  = sum_j w_j                   (also written s0)
 *   mu     = sum_j w_j z_j               (s1)
 *   Sigma  = sum_j w_j z_j z_j^T + lambda I   (S2)
 *   rho    = Sigma^{-1} mu               (dense Cholesky, no iteration)
 *   o_i    = sum_j w_j (1 - z_j^T rho) v_j / (omega - mu^T rho)
 *
 * The denominator omega - mu^T rho equals sum_j w_j (1 - z_j^T rho); the oracle
 * evaluates it in that second form, from the same coefficients as the
 * numerator, so numerator and denominator are consistent term by term.
 *
 * Overflow guard.  The weights are evaluated as exp(s_j - m) with m = max_j s_j
 * and the ridge as lambda * exp(-m).  Scaling every weight AND the ridge by the
 * same positive constant scales mu and Sigma alike, so rho = Sigma^{-1} mu and
 * the output are unchanged: this is the raw definition evaluated without
 * overflow.  (Scaling the weights alone would change the effective ridge; the
 * paper's remark that the computation is homogeneous in w holds only for
 * lambda = 0.)
 *
 * Nothing here is blocked, fused, re-centred or iterated: sums run in ascending
 * j in double precision, z_j is formed explicitly and Sigma is materialised.
 * "parity pinned": tests/test_oracle_pins.py checks this file against brute-force
 * weighted least squares, closed forms and limits (softmax limit, affine
 * reproduction, shift equivariance, first row, uniform-weight ridge regression,
 * joint scaling, permutation invariance, dual form).
 *
 * Inputs may be float32 or float64 arrays (in_f32 flag); float32 holds every
 * bf16 value exactly, so the bf16 test inputs are passed as float32.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_RIDGE_DEFINITION 0
#define ORACLE_RIDGE_PRINTED 1
#define ORACLE_NOT_SPD 1 /* Cholesky met a non-positive pivot (only possible at lambda = 0) */

static inline double ld(const void *p, size_t idx, int in_f32)
{
    return in_f32 ? (double)((const float *)p)[idx] : ((const double *)p)[idx];
}

/* In-place lower Cholesky of the d x d row-major matrix a; returns 0 on success. */
static int cholesky_lower(double *a, int d)
{
    for (int c = 0; c < d; ++c) {
        double diag = a[(size_t)c * d + c];
        for (int t = 0; t < c; ++t)
            diag -= a[(size_t)c * d + t] * a[(size_t)c * d + t];
        if (!(diag > 0.0))
            return 1;
        diag = sqrt(diag);
        a[(size_t)c * d + c] = diag;
        for (int r = c + 1; r < d; ++r) {
            double s = a[(size_t)r * d + c];
            for (int t = 0; t < c; ++t)
                s -= a[(size_t)r * d + t] * a[(size_t)c * d + t];
            a[(size_t)r * d + c] = s / diag;
        }
    }
    return 0;
}

/* Solve (L L^T) x = b with L the lower Cholesky factor; x overwrites b. */
static void cholesky_solve(const double *l, int d, double *b)
{
    for (int r = 0; r < d; ++r) {
        double s = b[r];
        for (int t = 0; t < r; ++t)
            s -= l[(size_t)r * d + t] * b[t];
        b[r] = s / l[(size_t)r * d + r];
    }
    for (int r = d - 1; r >= 0; --r) {
        double s = b[r];
        for (int t = r + 1; t < d; ++t)
            s -= l[(size_t)t * d + r] * b[t];
        b[r] = s / l[(size_t)r * d + r];
    }
}

/*
 * One query against L keys/values (Eq. "query_specific", Eq. "lla").
 *   q       : d values at offset q_off
 *   k, v    : L rows of d / dv values starting at offsets k_off / v_off (row stride d / dv)
 *   out     : dv doubles
 *   rho_out : optional d doubles (Sigma^{-1} mu)
 *   aux_out : optional 3 doubles: m (max score), omega and delta = omega - mu^T rho,
 *             the last two in the max-subtracted frame (weights exp(s - m))
 * work must hold L + L*d + d*d + 2*d doubles.
 */
static int oracle_row(const void *q, size_t q_off, const void *k, size_t k_off, const void *v,
                      size_t v_off, int L, int d, int dv, double scale, double lambda,
                      int ridge_mode, int in_f32, double *out, double *rho_out, double *aux_out,
                      double *work)
{
    double *w = work;                /* L   */
    double *z = w + L;               /* L*d */
    double *sigma = z + (size_t)L * d; /* d*d */
    double *mu = sigma + (size_t)d * d; /* d   */
    double *qi = mu + d;             /* d   */

    for (int c = 0; c < d; ++c)
        qi[c] = ld(q, q_off + c, in_f32);

    /* scores and their maximum */
    double m = -INFINITY;
    for (int j = 0; j < L; ++j) {
        double s = 0.0;
        for (int c = 0; c < d; ++c)
            s += qi[c] * ld(k, k_off + (size_t)j * d + c, in_f32);
        s *= scale;
        w[j] = s;
        if (s > m)
            m = s;
    }
    /* Ridge in the max-subtracted frame.  Mode 0: the definition, raw weights exp(s) with
     * ridge lambda, i.e. lambda * exp(-m) here.  Mode 1: Algorithm 1/2 as printed, which add
     * lambda to the moments of the weights exp(s - m) unchanged (an effective ridge
     * lambda * exp(m_i) in the raw frame). */
    const double lambda_m = ridge_mode == ORACLE_RIDGE_PRINTED ? lambda : lambda * exp(-m);

    /* weights, centred keys, moments */
    double omega = 0.0;
    memset(mu, 0, sizeof(double) * d);
    memset(sigma, 0, sizeof(double) * d * d);
    for (int j = 0; j < L; ++j) {
        const double wj = exp(w[j] - m);
        w[j] = wj;
        double *zj = z + (size_t)j * d;
        for (int c = 0; c < d; ++c)
            zj[c] = ld(k, k_off + (size_t)j * d + c, in_f32) - qi[c];
        omega += wj;
        for (int c = 0; c < d; ++c)
            mu[c] += wj * zj[c];
        for (int r = 0; r < d; ++r) {
            const double wz = wj * zj[r];
            double *srow = sigma + (size_t)r * d;
            for (int c = 0; c <= r; ++c)
                srow[c] += wz * zj[c];
        }
    }
    for (int r = 0; r < d; ++r) {
        sigma[(size_t)r * d + r] += lambda_m;
        for (int c = r + 1; c < d; ++c)
            sigma[(size_t)r * d + c] = sigma[(size_t)c * d + r];
    }

    /* rho = Sigma^{-1} mu */
    if (cholesky_lower(sigma, d) != 0) {
        for (int c = 0; c < dv; ++c)
            out[c] = NAN;
        if (rho_out)
            for (int c = 0; c < d; ++c)
                rho_out[c] = NAN;
        if (aux_out) {
            aux_out[0] = m;
            aux_out[1] = omega;
            aux_out[2] = NAN;
        }
        return ORACLE_NOT_SPD;
    }
    double *rho = mu; /* solved in place */
    cholesky_solve(sigma, d, rho);

    /* intercept: sum_j c_j v_j / sum_j c_j with c_j = w_j (1 - z_j^T rho) */
    for (int c = 0; c < dv; ++c)
        out[c] = 0.0;
    double denom = 0.0;
    for (int j = 0; j < L; ++j) {
        const double *zj = z + (size_t)j * d;
        double t = 0.0;
        for (int c = 0; c < d; ++c)
            t += zj[c] * rho[c];
        const double cj = w[j] * (1.0 - t);
        denom += cj;
        for (int c = 0; c < dv; ++c)
            out[c] += cj * ld(v, v_off + (size_t)j * dv + c, in_f32);
    }
    for (int c = 0; c < dv; ++c)
        out[c] /= denom;
    if (rho_out)
        for (int c = 0; c < d; ++c)
            rho_out[c] = rho[c];
    if (aux_out) {
        aux_out[0] = m;
        aux_out[1] = omega;
        aux_out[2] = denom;
    }
    return ORACLE_OK;
}

static size_t work_doubles(int L, int d)
{
    return (size_t)L + (size_t)L * d + (size_t)d * d + 2 * (size_t)d;
}

/*
 * Selected rows of the forward pass.
 *   q [B,H,n,d], k [B,H,n,d], v [B,H,n,dv]   contiguous, float32 or float64 (in_f32)
 *   rows[r] = flat index (b*H + h)*n + i     for r < n_rows
 *   out [n_rows, dv] float64; rho [n_rows, d] (may be NULL); aux [n_rows, 3] (may be NULL)
 *   status [n_rows] int (may be NULL): ORACLE_OK or ORACLE_NOT_SPD
 * Returns the number of rows whose Cholesky failed, or -1 on allocation failure.
 */
/*
 * As above with the ridge variants: lambda_rows (may be NULL) holds one ridge per query row,
 * [B*H*n] in the flat row order, and replaces the scalar (per-token regularisation, the
 * appendix on learnable lambda); ridge_mode is ORACLE_RIDGE_DEFINITION or ORACLE_RIDGE_PRINTED.
 */
int lla_oracle_forward_rows_ex(const void *q, const void *k, const void *v, int in_f32, int B,
                               int H, int n, int d, int dv, double scale, double lambda,
                               const double *lambda_rows, int ridge_mode, int causal,
                               const long long *rows, long long n_rows, double *out, double *rho,
                               double *aux, int *status);

int lla_oracle_forward_rows(const void *q, const void *k, const void *v, int in_f32, int B, int H,
                            int n, int d, int dv, double scale, double lambda, int causal,
                            const long long *rows, long long n_rows, double *out, double *rho,
                            double *aux, int *status)
{
    return lla_oracle_forward_rows_ex(q, k, v, in_f32, B, H, n, d, dv, scale, lambda, NULL,
                                      ORACLE_RIDGE_DEFINITION, causal, rows, n_rows, out, rho, aux,
                                      status);
}

int lla_oracle_forward_rows_ex(const void *q, const void *k, const void *v, int in_f32, int B,
                               int H, int n, int d, int dv, double scale, double lambda,
                               const double *lambda_rows, int ridge_mode, int causal,
                               const long long *rows, long long n_rows, double *out, double *rho,
                               double *aux, int *status)
{
    (void)B;
    (void)H;
    long long failures = 0;
    int alloc_failed = 0;
#pragma omp parallel reduction(+ : failures)
    {
        double *work = (double *)malloc(sizeof(double) * work_doubles(n, d));
        if (!work) {
#pragma omp atomic write
            alloc_failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long long r = 0; r < n_rows; ++r) {
            if (!work)
                continue;
            const long long flat = rows[r];
            const long long bh = flat / n;
            const int i = (int)(flat % n);
            const int L = causal ? i + 1 : n;
            const int st = oracle_row(q, (size_t)flat * d, k, (size_t)bh * n * d, v,
                                      (size_t)bh * n * dv, L, d, dv, scale,
                                      lambda_rows ? lambda_rows[flat] : lambda, ridge_mode, in_f32,
                                      out + (size_t)r * dv, rho ? rho + (size_t)r * d : NULL,
                                      aux ? aux + (size_t)r * 3 : NULL, work);
            if (status)
                status[r] = st;
            failures += (st != ORACLE_OK);
        }
        free(work);
    }
    return alloc_failed ? -1 : (int)failures;
}

/*
 * Single-query decode over a KV cache: the same formula with L = lens[b] keys.
 *   q [B,H,d]; kcache [B,H,Lmax,d]; vcache [B,H,Lmax,dv]; lens [B] (each in 1..Lmax; the
 *   current token's key and value are already in the cache, matching j <= i)
 *   out [B,H,dv] float64
 */
int lla_oracle_decode_ex(const void *q, const void *kcache, const void *vcache, int in_f32,
                         const int *lens, int B, int H, int Lmax, int d, int dv, double scale,
                         double lambda, const double *lambda_units, int ridge_mode, double *out,
                         int *status);

int lla_oracle_decode(const void *q, const void *kcache, const void *vcache, int in_f32,
                      const int *lens, int B, int H, int Lmax, int d, int dv, double scale,
                      double lambda, double *out, int *status)
{
    return lla_oracle_decode_ex(q, kcache, vcache, in_f32, lens, B, H, Lmax, d, dv, scale, lambda,
                                NULL, ORACLE_RIDGE_DEFINITION, out, status);
}

/* Decode with the ridge variants: lambda_units (may be NULL) is one ridge per (sequence, head). */
int lla_oracle_decode_ex(const void *q, const void *kcache, const void *vcache, int in_f32,
                         const int *lens, int B, int H, int Lmax, int d, int dv, double scale,
                         double lambda, const double *lambda_units, int ridge_mode, double *out,
                         int *status)
{
    long long failures = 0;
    int alloc_failed = 0;
#pragma omp parallel reduction(+ : failures)
    {
        double *work = (double *)malloc(sizeof(double) * work_doubles(Lmax, d));
        if (!work) {
#pragma omp atomic write
            alloc_failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long long bh = 0; bh < (long long)B * H; ++bh) {
            if (!work)
                continue;
            const int b = (int)(bh / H);
            const int st = oracle_row(q, (size_t)bh * d, kcache, (size_t)bh * Lmax * d, vcache,
                                      (size_t)bh * Lmax * dv, lens[b], d, dv, scale,
                                      lambda_units ? lambda_units[bh] : lambda, ridge_mode,
                                      in_f32, out + (size_t)bh * dv, NULL, NULL, work);
            if (status)
                status[bh] = st;
            failures += (st != ORACLE_OK);
        }
        free(work);
    }
    return alloc_failed ? -1 : (int)failures;
}

/* Threads the parallel loops above will use (1 when built without OpenMP). */
int lla_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
