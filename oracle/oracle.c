/*
 * ORACLE -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain, slow, double-precision CPU statement of what the filter-gradient path
 * computes: the exact filter gradient of a convolution layer and the three
 * approximation methods of the paper's Section 2 (zero gradient 2.1, random
 * gradient 2.2, max-gradient approximation 2.3 / Algorithm 1).
 *
 * Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call this file.  It shares no code, header, table or constant with the CUDA
 * library; the product never routes through it.
 *
 * Conventions (all arrays dense, row-major, double precision):
 *   x  [N][C][H][W]   input activations          (paper: I,  N x C_i x H x W)
 *   dy [N][K][P][Q]   output gradient            (paper: dO, N x C_o x H x W)
 *   dw [K][C][R][S]   filter gradient            (paper: df)
 *   P = (H + 2*pad_h - R)/stride_h + 1, Q likewise.
 * Padding is zero padding: x is read as 0 outside [0,H) x [0,W).
 * The operation is a cross-correlation (no filter flip), i.e. the derivative of
 *   y[n,k,p,q] = sum_{c,r,s} x[n,c,p*stride+r-pad,q*stride+s-pad] * w[k,c,r,s]
 * with respect to w, contracted with dy.
 *
 * Pins (tests/test_oracle_*.py): finite differences of a tiny convolution's loss,
 * a seven-deep brute-force loop in Python, delta inputs with a closed-form answer,
 * the 1x1 and full-window special cases that reduce to a matrix product, torch's
 * CPU float64 weight gradient, the identities "top-1 == exact on the sparsified
 * dY" and "full selection == exact", spatially constant X (where Algorithm 1 is
 * exact), published known-answer vectors of the Philox-4x32-10 generator, and
 * the paper's stated counts of approximated layers for its first schedule.
 * Top-k beyond k = 1 follows a reading the paper does not fix (each retained entry
 * gets sum/k): pinned only by k = 1 == Algorithm 1, by the sparse-list identity and
 * by the constant-X case -- "parity unpinned" for the choice of scale itself.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int n, c, h, w;      /* input activations */
    int k, r, s;         /* filters */
    int stride_h, stride_w, pad_h, pad_w;
    int p, q;            /* output map size (derived by the caller, checked here) */
} oracle_shape_t;

static int shape_ok(const oracle_shape_t *g)
{
    if (g->n < 1 || g->c < 1 || g->h < 1 || g->w < 1 || g->k < 1 || g->r < 1 || g->s < 1) return 0;
    if (g->stride_h < 1 || g->stride_w < 1 || g->pad_h < 0 || g->pad_w < 0) return 0;
    if (g->h + 2 * g->pad_h < g->r || g->w + 2 * g->pad_w < g->s) return 0;
    if (g->p != (g->h + 2 * g->pad_h - g->r) / g->stride_h + 1) return 0;
    if (g->q != (g->w + 2 * g->pad_w - g->s) / g->stride_w + 1) return 0;
    return 1;
}

/* x read with zero padding */
static double xz(const double *x, const oracle_shape_t *g, int n, int c, int hh, int ww)
{
    if (hh < 0 || hh >= g->h || ww < 0 || ww >= g->w) return 0.0;
    return x[(((size_t)n * g->c + c) * g->h + hh) * g->w + ww];
}

/* ---------------------------------------------------------------------------
 * Exact filter gradient (the operation in the red box of the paper's Figure 1;
 * Section 2.4, which states the filter gradient as the convolution of the input with the output gradient):
 *
 *   dw[k,c,r,s] = alpha * sum_{n,p,q} xz[n,c,p*st_h+r-pad_h,q*st_w+s-pad_w] * dy[n,k,p,q]
 *
 * dnorm (may be NULL) receives |alpha| * sum |xz * dy|, the normaliser of the
 * parity metric.  One output element.
 * ------------------------------------------------------------------------- */
void oracle_dw_exact_at(const double *x, const double *dy, const oracle_shape_t *g, double alpha,
                        int k, int c, int r, int s, double *value, double *norm)
{
    double acc = 0.0, nrm = 0.0;
    for (int n = 0; n < g->n; ++n)
        for (int p = 0; p < g->p; ++p)
            for (int q = 0; q < g->q; ++q) {
                double a = xz(x, g, n, c, p * g->stride_h + r - g->pad_h, q * g->stride_w + s - g->pad_w);
                double b = dy[(((size_t)n * g->k + k) * g->p + p) * g->q + q];
                acc += a * b;
                nrm += fabs(a * b);
            }
    *value = alpha * acc;
    if (norm) *norm = fabs(alpha) * nrm;
}

int oracle_dw_exact(const double *x, const double *dy, double *dw, double *dnorm,
                    const oracle_shape_t *g, double alpha)
{
    if (!shape_ok(g)) return 1;
#pragma omp parallel for schedule(static)
    for (int k = 0; k < g->k; ++k)
        for (int c = 0; c < g->c; ++c)
            for (int r = 0; r < g->r; ++r)
                for (int s = 0; s < g->s; ++s) {
                    size_t o = (((size_t)k * g->c + c) * g->r + r) * g->s + s;
                    double v, nrm;
                    oracle_dw_exact_at(x, dy, g, alpha, k, c, r, s, &v, &nrm);
                    dw[o] = v;
                    if (dnorm) dnorm[o] = nrm;
                }
    return 0;
}

/* ---------------------------------------------------------------------------
 * Order of magnitudes used by every selection below: the bit pattern of |v| read as
 * an unsigned integer.  For finite values this is the order of |v| itself; it also
 * gives -0 = +0, infinity above every finite value and NaNs above infinity (ordered
 * by payload), so the selected position is defined for any input.  Widening a bf16
 * or fp32 value to double keeps this order, so the key of the double equals the
 * order of the keys in the input type.
 * ------------------------------------------------------------------------- */
static uint64_t mag_key(double v)
{
    uint64_t b;
    memcpy(&b, &v, sizeof b);
    return b & 0x7fffffffffffffffull;
}

/* ---------------------------------------------------------------------------
 * Selection step of Algorithm 1 for every (n, k) pair:
 *   idx[n,k]    = position j = p*Q+q of the largest-magnitude element of dy[n,k,:,:];
 *                 among equal magnitudes the lowest j
 *   sum[n,k]    = signed sum of dy[n,k,:,:]
 *   abssum[n,k] = sum of |dy[n,k,:,:]|   (normaliser only; may be NULL)
 * ------------------------------------------------------------------------- */
void oracle_top1_select(const double *dy, int n_, int k_, int pq, int32_t *idx, double *sum, double *abssum)
{
    for (int n = 0; n < n_; ++n)
        for (int k = 0; k < k_; ++k) {
            const double *m = dy + ((size_t)n * k_ + k) * pq;
            int best = 0;
            uint64_t bestkey = mag_key(m[0]);
            double t = 0.0, ta = 0.0;
            for (int j = 0; j < pq; ++j) {
                if (mag_key(m[j]) > bestkey) { bestkey = mag_key(m[j]); best = j; }
                t += m[j];
                ta += fabs(m[j]);
            }
            idx[(size_t)n * k_ + k] = best;
            sum[(size_t)n * k_ + k] = t;
            if (abssum) abssum[(size_t)n * k_ + k] = ta;
        }
}

/* ---------------------------------------------------------------------------
 * Max-gradient approximation (Section 2.3, Algorithm 1).  What it computes: the
 * exact filter gradient of a tensor that keeps, for every image n and output channel
 * k, a single entry of dy[n,k,:,:] -- at the position of the largest magnitude -- and
 * gives that entry the signed sum of the whole map.  Hence, per (k, n): find the
 * position, take the sum, and add sum * (the input patch that the exact formula
 * pairs with that output position) to the gradient of filter k.
 * The patch comes from the zero-padded input: element (r,s) of it is
 * xz[n, c, row*st_h + r - pad_h, col*st_w + s - pad_w].
 * alpha scales the result (the paper scales by 1/128 = 1/batch, Section 2.3).
 * dnorm (may be NULL) receives |alpha| * sum_n abssum[n,k] * |patch element|.
 * ------------------------------------------------------------------------- */
int oracle_dw_top1(const double *x, const double *dy, double *dw, double *dnorm,
                   const oracle_shape_t *g, double alpha)
{
    if (!shape_ok(g)) return 1;
    size_t total = (size_t)g->k * g->c * g->r * g->s;
    memset(dw, 0, total * sizeof(double));
    if (dnorm) memset(dnorm, 0, total * sizeof(double));
    int pq = g->p * g->q;
    for (int k = 0; k < g->k; ++k)
        for (int n = 0; n < g->n; ++n) {
            const double *m = dy + ((size_t)n * g->k + k) * pq;
            int best = 0;
            for (int j = 1; j < pq; ++j)
                if (mag_key(m[j]) > mag_key(m[best])) best = j;
            double sum = 0.0, asum = 0.0;
            for (int j = 0; j < pq; ++j) { sum += m[j]; asum += fabs(m[j]); }
            int row = best / g->q, col = best % g->q;
            for (int c = 0; c < g->c; ++c)
                for (int r = 0; r < g->r; ++r)
                    for (int s = 0; s < g->s; ++s) {
                        double v = xz(x, g, n, c, row * g->stride_h + r - g->pad_h, col * g->stride_w + s - g->pad_w);
                        size_t o = (((size_t)k * g->c + c) * g->r + r) * g->s + s;
                        dw[o] += alpha * (v * sum);
                        if (dnorm) dnorm[o] += fabs(alpha) * fabs(v) * asum;
                    }
        }
    return 0;
}

/* ---------------------------------------------------------------------------
 * Top-k variant (Section 2.3 says the method extends to the k largest magnitudes
 * with an adjusted scale; the scale is not given).  Reading taken here: the `topk`
 * largest-magnitude entries of a map are retained (equal magnitudes: lower position
 * first) and each receives sum/topk, so that the retained entries still add up to the
 * signed sum of the map.  topk = 1 is Algorithm 1.
 *   idx[(n*K+k)*topk + t] = position of the t-th retained entry, in order of selection.
 * ------------------------------------------------------------------------- */
void oracle_topk_select(const double *dy, int n_, int k_, int pq, int topk, int32_t *idx, double *sum, double *abssum)
{
    if (topk > pq) topk = pq;
    for (size_t mi = 0; mi < (size_t)n_ * k_; ++mi) {
        const double *m = dy + mi * pq;
        double t = 0.0, ta = 0.0;
        for (int j = 0; j < pq; ++j) { t += m[j]; ta += fabs(m[j]); }
        sum[mi] = t;
        if (abssum) abssum[mi] = ta;
        for (int sel = 0; sel < topk; ++sel) {
            int best = -1;
            for (int j = 0; j < pq; ++j) {
                int taken = 0;
                for (int u = 0; u < sel; ++u) if (idx[mi * topk + u] == j) taken = 1;
                if (taken) continue;
                if (best < 0 || mag_key(m[j]) > mag_key(m[best])) best = j;
            }
            idx[mi * topk + sel] = best;
        }
    }
}

int oracle_dw_topk(const double *x, const double *dy, double *dw, double *dnorm,
                   const oracle_shape_t *g, double alpha, int topk)
{
    if (!shape_ok(g) || topk < 1) return 1;
    size_t total = (size_t)g->k * g->c * g->r * g->s;
    memset(dw, 0, total * sizeof(double));
    if (dnorm) memset(dnorm, 0, total * sizeof(double));
    int pq = g->p * g->q;
    if (topk > pq) topk = pq;
    size_t maps = (size_t)g->n * g->k;
    int32_t *idx = (int32_t *)malloc(maps * topk * sizeof(int32_t));
    double *sum = (double *)malloc(maps * sizeof(double)), *asum = (double *)malloc(maps * sizeof(double));
    if (!idx || !sum || !asum) { free(idx); free(sum); free(asum); return 3; }
    oracle_topk_select(dy, g->n, g->k, pq, topk, idx, sum, asum);
    for (int k = 0; k < g->k; ++k)
        for (int n = 0; n < g->n; ++n) {
            size_t mi = (size_t)n * g->k + k;
            double share = sum[mi] / topk, ashare = asum[mi] / topk;
            for (int t = 0; t < topk; ++t) {
                int row = idx[mi * topk + t] / g->q, col = idx[mi * topk + t] % g->q;
                for (int c = 0; c < g->c; ++c)
                    for (int r = 0; r < g->r; ++r)
                        for (int s = 0; s < g->s; ++s) {
                            double v = xz(x, g, n, c, row * g->stride_h + r - g->pad_h, col * g->stride_w + s - g->pad_w);
                            size_t o = (((size_t)k * g->c + c) * g->r + r) * g->s + s;
                            dw[o] += alpha * (v * share);
                            if (dnorm) dnorm[o] += fabs(alpha) * fabs(v) * ashare;
                        }
            }
        }
    free(idx); free(sum); free(asum);
    return 0;
}

/* ---------------------------------------------------------------------------
 * Sparse accumulate: the filter gradient of an arbitrary list of retained
 * output-gradient entries (n, k, p, q, value).  Section 2.3: the filter gradient
 * is the one computed from the sparse version of the output-gradient tensor.
 * With the top-1 list it must equal oracle_dw_top1; with every entry of dy listed
 * it must equal oracle_dw_exact.
 * ------------------------------------------------------------------------- */
int oracle_dw_sparse(const double *x, const int32_t *en, const int32_t *ek, const int32_t *ep,
                     const int32_t *eq, const double *ev, size_t count, double *dw,
                     const oracle_shape_t *g, double alpha)
{
    if (!shape_ok(g)) return 1;
    size_t total = (size_t)g->k * g->c * g->r * g->s;
    memset(dw, 0, total * sizeof(double));
    for (size_t e = 0; e < count; ++e) {
        int n = en[e], k = ek[e], p = ep[e], q = eq[e];
        if (n < 0 || n >= g->n || k < 0 || k >= g->k || p < 0 || p >= g->p || q < 0 || q >= g->q) return 2;
        for (int c = 0; c < g->c; ++c)
            for (int r = 0; r < g->r; ++r)
                for (int s = 0; s < g->s; ++s) {
                    double v = xz(x, g, n, c, p * g->stride_h + r - g->pad_h, q * g->stride_w + s - g->pad_w);
                    dw[(((size_t)k * g->c + c) * g->r + r) * g->s + s] += alpha * (v * ev[e]);
                }
    }
    return 0;
}

/* The sparse version of the output gradient, stored densely (Section 2.3): sum at idx, 0 elsewhere. */
void oracle_sparsify(const int32_t *idx, const double *sum, int n_, int k_, int pq, double *dy_sparse)
{
    memset(dy_sparse, 0, (size_t)n_ * k_ * pq * sizeof(double));
    for (size_t i = 0; i < (size_t)n_ * k_; ++i) dy_sparse[i * pq + idx[i]] = sum[i];
}

/* ---------------------------------------------------------------------------
 * Zero gradient (Section 2.1).
 * ------------------------------------------------------------------------- */
void oracle_dw_zero(double *dw, size_t count)
{
    for (size_t i = 0; i < count; ++i) dw[i] = 0.0;
}

/* ---------------------------------------------------------------------------
 * Random gradient (Section 2.2): independent N(0, std^2) values, regenerated for
 * every (seed).  The paper drew them from a host generator that cannot be
 * reproduced, so both sides follow a written recipe instead:
 *
 *   Philox-4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with
 *     key     = (seed low 32 bits, seed high 32 bits)
 *     counter = (j, 0, 0, 0)                       j = 0, 1, 2, ...
 *   gives words w0..w3, which become elements 4j .. 4j+3:
 *     u1 = (w_a + 1) * 2^-32  in (0,1],  u2 = w_b * 2^-32 in [0,1)
 *     rho = sqrt(-2 ln u1)
 *     z[4j]   = rho(w0,w1) cos(2 pi u2(w1)),  z[4j+1] = rho(w0,w1) sin(2 pi u2(w1))
 *     z[4j+2] = rho(w2,w3) cos(2 pi u2(w3)),  z[4j+3] = rho(w2,w3) sin(2 pi u2(w3))
 *   dw[i] = std * z[i], i indexing the logical [K][C][R][S] order.
 * ------------------------------------------------------------------------- */
static void mulhilo(uint32_t a, uint32_t b, uint32_t *hi, uint32_t *lo)
{
    uint64_t prod = (uint64_t)a * (uint64_t)b;
    *hi = (uint32_t)(prod >> 32);
    *lo = (uint32_t)prod;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u; /* round multipliers */
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u; /* key schedule (Weyl) increments */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo(M0, c0, &hi0, &lo0);
        mulhilo(M1, c2, &hi1, &lo1);
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

void oracle_random_words(uint64_t seed, size_t count, uint32_t *words)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (size_t j = 0; 4 * j < count; ++j) {
        uint32_t ctr[4] = { (uint32_t)j, 0u, 0u, 0u }, w[4];
        oracle_philox4x32_10(ctr, key, w);
        for (int t = 0; t < 4 && 4 * j + t < count; ++t) words[4 * j + t] = w[t];
    }
}

void oracle_dw_random(double *dw, size_t count, uint64_t seed, double std)
{
    const double two_pi = 6.283185307179586476925286766559;
    const double inv32 = 1.0 / 4294967296.0;
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (size_t j = 0; 4 * j < count; ++j) {
        uint32_t ctr[4] = { (uint32_t)j, 0u, 0u, 0u }, w[4];
        oracle_philox4x32_10(ctr, key, w);
        double z[4];
        for (int h = 0; h < 2; ++h) {
            double u1 = ((double)w[2 * h] + 1.0) * inv32;
            double u2 = (double)w[2 * h + 1] * inv32;
            double rho = sqrt(-2.0 * log(u1));
            z[2 * h] = rho * cos(two_pi * u2);
            z[2 * h + 1] = rho * sin(two_pi * u2);
        }
        for (int t = 0; t < 4 && 4 * j + t < count; ++t) dw[4 * j + t] = std * z[t];
    }
}

/* Number of OpenMP threads the exact path uses (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int oracle_num_threads(void) { return 1; }
#endif
