/*
 * CPU oracle for feature-map transform coding (Section 3 and 3.1 of the paper).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, scalar, fp64, bit-serial statement of
 * what the codec computes, written to be checked against the paper by eye.  Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it; the CUDA library never
 * does, and the two share no code, tables or helpers.
 *
 * Chain (Section 3): y = T (x - mu)  ->  Q_Delta  ->  VLC  ->  memory  ->  VLD  ->
 * Q_Delta^-1  ->  T^-1 = T^T  ->  x_hat.  Blocks are 1 x 1 x C (Section 3.1, "Linear
 * transform"): every pixel's C-vector is one block.
 *
 * Parity pins (see tests/test_oracle_*.py): every function below is pinned to something other
 * than itself -- hand-worked examples, closed forms, invariants, numpy's eigensolver, brute
 * force over all feasible code-length vectors.  Not pinned, because it needs ImageNet and
 * trained weights: the absolute bits/value the paper reports on real networks ("parity
 * unpinned" for those figures only).
 *
 * Tensors are dense NCHW, passed as float (both fp32 and bf16 inputs are exactly representable
 * in float); all arithmetic is double.  P = N*H*W pixels, pixel p = n*HW + s.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------
 * Rounding helpers
 * ---------------------------------------------------------------------------------------- */

/* Round a double to the nearest bfloat16 value (8 significant bits, fp32 exponent range),
 * ties to even.  Scaling by a power of two is exact, so rint() takes the one rounding. */
double orc_round_bf16(double v)
{
    if (v == 0.0 || isnan(v) || isinf(v)) return v;
    int e;
    frexp(v, &e);            /* |v| = f * 2^e, f in [0.5, 1)  ->  floor(log2|v|) = e - 1 */
    int ex = e - 1;
    if (ex < -126) ex = -126; /* subnormal range shares one spacing */
    double ulp = ldexp(1.0, ex - 7);
    double r = rint(v / ulp) * ulp;
    if (fabs(r) >= ldexp(1.0, 128)) r = copysign(INFINITY, v);
    return r;
}

/* ------------------------------------------------------------------------------------------
 * O1. Fit (Section 3: x ~ N(mu, Sigma), T diagonalises Sigma, T^-1 = T^T; Section 3.1:
 * covariance estimated on a small calibration batch; quantiser range from the channel with
 * the highest variance).
 * ---------------------------------------------------------------------------------------- */

/* mean[c] and the unbiased sample covariance cov[c][c] over all M = n*hw pixel vectors.
 * Two passes: mean first, then centred outer products. */
void orc_mean_cov(const float *x, int64_t n, int c, int64_t hw, double *mean, double *cov)
{
    const int64_t m = n * hw;
    for (int a = 0; a < c; ++a) mean[a] = 0.0;
    for (int64_t i = 0; i < n; ++i)
        for (int a = 0; a < c; ++a) {
            const float *row = x + (i * c + a) * hw;
            double s = 0.0;
            for (int64_t t = 0; t < hw; ++t) s += (double)row[t];
            mean[a] += s;
        }
    for (int a = 0; a < c; ++a) mean[a] /= (double)m;

    for (int64_t k = 0; k < (int64_t)c * c; ++k) cov[k] = 0.0;
    double *d = (double *)malloc(sizeof(double) * (size_t)c);
    for (int64_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < hw; ++t) {
            for (int a = 0; a < c; ++a) d[a] = (double)x[(i * c + a) * hw + t] - mean[a];
            for (int a = 0; a < c; ++a)
                for (int b = a; b < c; ++b) cov[(int64_t)a * c + b] += d[a] * d[b];
        }
    free(d);
    const double denom = (m > 1) ? (double)(m - 1) : 1.0;
    for (int a = 0; a < c; ++a)
        for (int b = a; b < c; ++b) {
            cov[(int64_t)a * c + b] /= denom;
            cov[(int64_t)b * c + a] = cov[(int64_t)a * c + b];
        }
}

/* Symmetric eigendecomposition by cyclic Jacobi rotations.  `a` (n x n, symmetric) is
 * destroyed; on return evals[i] is the i-th diagonal entry and row i of `vt` its unit
 * eigenvector (unsorted).  Returns the number of sweeps used, or -1 if not converged. */
int orc_eigh_jacobi(double *a, int n, double *evals, double *vt)
{
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) vt[(int64_t)i * n + j] = (i == j) ? 1.0 : 0.0;
    double total = 0.0;
    for (int64_t k = 0; k < (int64_t)n * n; ++k) total += a[k] * a[k];
    if (total == 0.0) { for (int i = 0; i < n; ++i) evals[i] = 0.0; return 0; }
    const double tol = 1e-24 * total;   /* on the squared off-diagonal norm: |off| <= 1e-12 |A|_F */
    int sweep;
    for (sweep = 0; sweep < 100; ++sweep) {
        double off = 0.0;
        for (int p = 0; p < n; ++p)
            for (int q = p + 1; q < n; ++q) off += 2.0 * a[(int64_t)p * n + q] * a[(int64_t)p * n + q];
        if (off <= tol) break;
        for (int p = 0; p < n - 1; ++p)
            for (int q = p + 1; q < n; ++q) {
                const double apq = a[(int64_t)p * n + q];
                if (apq == 0.0) continue;
                const double app = a[(int64_t)p * n + p], aqq = a[(int64_t)q * n + q];
                const double theta = (aqq - app) / (2.0 * apq);
                const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                const double cs = 1.0 / sqrt(t * t + 1.0), sn = t * cs;
                double *rp = a + (int64_t)p * n, *rq = a + (int64_t)q * n;
                for (int k = 0; k < n; ++k) {
                    if (k == p || k == q) continue;
                    const double akp = rp[k], akq = rq[k];
                    rp[k] = cs * akp - sn * akq;
                    rq[k] = sn * akp + cs * akq;
                    a[(int64_t)k * n + p] = rp[k];
                    a[(int64_t)k * n + q] = rq[k];
                }
                rp[p] = app - t * apq;
                rq[q] = aqq + t * apq;
                rp[q] = 0.0;
                rq[p] = 0.0;
                double *vp = vt + (int64_t)p * n, *vq = vt + (int64_t)q * n;
                for (int k = 0; k < n; ++k) {
                    const double vkp = vp[k], vkq = vq[k];
                    vp[k] = cs * vkp - sn * vkq;
                    vq[k] = sn * vkp + cs * vkq;
                }
            }
    }
    for (int i = 0; i < n; ++i) evals[i] = a[(int64_t)i * n + i];
    return sweep < 100 ? sweep : -1;
}

/* Full fit.  Outputs: mean[c]; basis[c][c], row j = j-th principal direction (descending
 * eigenvalue; equal eigenvalues keep their original order; each row signed so that its
 * entry of largest magnitude -- the first such on ties -- is positive); eig[c]; and the
 * quantiser range [lo, hi] = min/max over the calibration pixels of coefficient 0, the
 * highest-variance channel, with step = (hi - lo) / (2^bits - 1).
 * basis_round: 0 keeps fp64; 1 rounds every entry of the basis to bfloat16, 2 to fp32 (ties to
 * even) before the range pass, and that rounded matrix is the transform from then on.
 * 3 quantises the matrix to 8 bits (Section 3.1 says the PCA matrix is stored in 8 bits; the
 * quantiser is this reading: one scale s = max|T| / 127 for the whole matrix, every entry
 * becomes s * rint(T / s), an integer in [-127, 127] times s); *basis_scale receives s (1.0 in
 * the other modes).  The decoder uses the transpose of the same quantised matrix.
 * The eigendecomposition is the in-file Jacobi solver, unless the caller passes one it
 * obtained from a library routine (pre_evals[c], pre_vt[c][c] with unit eigenvectors as rows,
 * any order): Jacobi takes minutes beyond a few hundred channels.
 * Returns 0, or -1 if the eigensolver did not converge. */
static int fit_from_mean_cov(const float *x, int64_t n, int c, int64_t hw, int bits, int basis_round,
                             const double *pre_evals, const double *pre_vt, const double *mean, double *cov,
                             double *basis, double *eig, double *lo, double *step, double *basis_scale)
{
    double *ev = (double *)malloc(sizeof(double) * (size_t)c);
    double *vt = (double *)malloc(sizeof(double) * (size_t)c * c);
    int *order = (int *)malloc(sizeof(int) * (size_t)c);
    int rc = 0;
    if (pre_evals && pre_vt) {
        memcpy(ev, pre_evals, sizeof(double) * (size_t)c);
        memcpy(vt, pre_vt, sizeof(double) * (size_t)c * c);
    } else {
        rc = orc_eigh_jacobi(cov, c, ev, vt);
    }
    /* stable insertion sort of indices by descending eigenvalue */
    for (int i = 0; i < c; ++i) order[i] = i;
    for (int i = 1; i < c; ++i) {
        int o = order[i], j = i - 1;
        while (j >= 0 && ev[order[j]] < ev[o]) { order[j + 1] = order[j]; --j; }
        order[j + 1] = o;
    }
    for (int j = 0; j < c; ++j) {
        const double *src = vt + (int64_t)order[j] * c;
        int big = 0;
        for (int k = 1; k < c; ++k) if (fabs(src[k]) > fabs(src[big])) big = k;
        const double sgn = (src[big] < 0.0) ? -1.0 : 1.0;
        for (int k = 0; k < c; ++k) {
            double v = sgn * src[k];
            if (basis_round == 1) v = orc_round_bf16(v);
            else if (basis_round == 2) v = (double)(float)v;
            basis[(int64_t)j * c + k] = v;
        }
        eig[j] = ev[order[j]];
    }
    double scale = 1.0;
    if (basis_round == 3) {
        double biggest = 0.0;
        for (int64_t i = 0; i < (int64_t)c * c; ++i) if (fabs(basis[i]) > biggest) biggest = fabs(basis[i]);
        scale = biggest / 127.0;
        for (int64_t i = 0; i < (int64_t)c * c; ++i) basis[i] = scale * rint(basis[i] / scale);
    }
    if (basis_scale) *basis_scale = scale;
    double mn = INFINITY, mx = -INFINITY;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < hw; ++t) {
            double y0 = 0.0;
            for (int a = 0; a < c; ++a) y0 += basis[a] * ((double)x[(i * c + a) * hw + t] - mean[a]);
            if (y0 < mn) mn = y0;
            if (y0 > mx) mx = y0;
        }
    *lo = mn;
    *step = (mx - mn) / (double)((1 << bits) - 1);
    free(ev); free(vt); free(order);
    return rc < 0 ? -1 : 0;
}

int orc_fit_pca(const float *x, int64_t n, int c, int64_t hw, int bits, int basis_round,
                const double *pre_evals, const double *pre_vt,
                double *mean, double *basis, double *eig, double *lo, double *step, double *basis_scale)
{
    double *cov = (double *)malloc(sizeof(double) * (size_t)c * c);
    orc_mean_cov(x, n, c, hw, mean, cov);
    const int rc = fit_from_mean_cov(x, n, c, hw, bits, basis_round, pre_evals, pre_vt, mean, cov, basis, eig, lo, step,
                                     basis_scale);
    free(cov);
    return rc;
}

/* Online estimate (Section 3.1: the covariance "can be updated online").  The running state is
 * the sample count M, the sum of the pixel vectors s[c] and the sum of their outer products
 * S[c][c]; a further batch only adds to the three, so states of disjoint batches (later
 * batches, other devices, an earlier run) merge by addition.  orc_moments_update adds the n*hw
 * pixel vectors of x. */
void orc_moments_update(const float *x, int64_t n, int c, int64_t hw, int64_t *count, double *sum, double *outer)
{
    double *v = (double *)malloc(sizeof(double) * (size_t)c);
    for (int64_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < hw; ++t) {
            for (int a = 0; a < c; ++a) v[a] = (double)x[(i * c + a) * hw + t];
            for (int a = 0; a < c; ++a) {
                sum[a] += v[a];
                for (int b = 0; b < c; ++b) outer[(int64_t)a * c + b] += v[a] * v[b];
            }
        }
    free(v);
    *count += n * hw;
}

/* mean = s / M and the unbiased covariance (S - s s^T / M) / (M - 1) of the running state. */
void orc_moments_mean_cov(int64_t count, const double *sum, const double *outer, int c, double *mean, double *cov)
{
    const double m = (double)count;
    for (int a = 0; a < c; ++a) mean[a] = sum[a] / m;
    const double denom = (count > 1) ? m - 1.0 : 1.0;
    for (int a = 0; a < c; ++a)
        for (int b = 0; b < c; ++b)
            cov[(int64_t)a * c + b] = (outer[(int64_t)a * c + b] - sum[a] * sum[b] / m) / denom;
}

/* The fit of orc_fit_pca with mean and covariance taken from a running state; the quantiser
 * range (coefficient 0) is measured on the maps x, which the caller chooses (for instance the
 * last calibration batch): the basis is not known while the state is being accumulated. */
int orc_fit_pca_moments(int64_t count, const double *sum, const double *outer,
                        const float *x, int64_t n, int c, int64_t hw, int bits, int basis_round,
                        const double *pre_evals, const double *pre_vt,
                        double *mean, double *basis, double *eig, double *lo, double *step, double *basis_scale)
{
    double *cov = (double *)malloc(sizeof(double) * (size_t)c * c);
    orc_moments_mean_cov(count, sum, outer, c, mean, cov);
    const int rc = fit_from_mean_cov(x, n, c, hw, bits, basis_round, pre_evals, pre_vt, mean, cov, basis, eig, lo, step,
                                     basis_scale);
    free(cov);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * O2. Projection  y_p = T (x_p - mu)   (Section 3, first equation).  y is [P][K].
 * ---------------------------------------------------------------------------------------- */
void orc_project(const float *x, int64_t n, int c, int64_t hw, const double *mean,
                 const double *basis, int k, double *y)
{
    for (int64_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < hw; ++t) {
            double *yp = y + (i * hw + t) * k;
            for (int j = 0; j < k; ++j) {
                double s = 0.0;
                for (int a = 0; a < c; ++a)
                    s += basis[(int64_t)j * c + a] * ((double)x[(i * c + a) * hw + t] - mean[a]);
                yp[j] = s;
            }
        }
}

/* ------------------------------------------------------------------------------------------
 * O3. Uniform scalar quantiser Q_Delta with one step for all coefficient channels (Section
 * 3.1 "Quantization", Fig. 1c).  Levels are lo + q*step, q = 0 .. 2^bits - 1; values outside
 * the range clamp; halves round to even.  `units` (optional) receives (y - lo)/step, the
 * position in step units, which the parity tests use to recognise rounding ties.
 * ---------------------------------------------------------------------------------------- */
void orc_quantize(const double *y, int64_t count, double lo, double step, int bits,
                  uint8_t *q, double *units)
{
    const double top = (double)((1 << bits) - 1);
    for (int64_t i = 0; i < count; ++i) {
        const double u = (y[i] - lo) / step;
        double r = rint(u);
        if (r < 0.0) r = 0.0;
        if (r > top) r = top;
        q[i] = (uint8_t)r;
        if (units) units[i] = u;
    }
}

/* O4. Histogram of symbols per group: group = coefficient index j when groups == k,
 * else 0 (one table per layer).  hist is [groups][2^bits]. */
void orc_histogram(const uint8_t *q, int64_t pixels, int k, int groups, int bits, uint64_t *hist)
{
    const int nsym = 1 << bits;
    memset(hist, 0, sizeof(uint64_t) * (size_t)groups * nsym);
    for (int64_t p = 0; p < pixels; ++p)
        for (int j = 0; j < k; ++j) {
            const int g = (groups == 1) ? 0 : j;
            hist[(int64_t)g * nsym + q[p * k + j]] += 1;
        }
}

/* ------------------------------------------------------------------------------------------
 * O5. Huffman code lengths (Section 3.1 "Variable length coding"), canonical codes.
 * ---------------------------------------------------------------------------------------- */

/* Plain Huffman by the two-queue construction.  Leaves sorted by (weight, symbol); when a
 * leaf and an internal node weigh the same, the leaf is taken first.  All weights > 0. */
static void huffman_unlimited(const uint64_t *w, int nsym, uint8_t *len)
{
    int *leaf = (int *)malloc(sizeof(int) * (size_t)nsym);
    for (int i = 0; i < nsym; ++i) leaf[i] = i;
    for (int i = 1; i < nsym; ++i) {           /* stable insertion sort by weight */
        int s = leaf[i], j = i - 1;
        while (j >= 0 && w[leaf[j]] > w[s]) { leaf[j + 1] = leaf[j]; --j; }
        leaf[j + 1] = s;
    }
    const int total = 2 * nsym - 1;
    uint64_t *nw = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)total);
    int *parent = (int *)malloc(sizeof(int) * (size_t)total);
    for (int i = 0; i < nsym; ++i) nw[i] = w[leaf[i]];   /* nodes 0..nsym-1: sorted leaves */
    for (int i = 0; i < total; ++i) parent[i] = -1;
    int h1 = 0, h2 = nsym, made = nsym;                   /* queue heads, next internal id */
    while (made < total) {
        int pick[2];
        for (int r = 0; r < 2; ++r) {
            const int have1 = h1 < nsym, have2 = h2 < made;
            if (have1 && (!have2 || nw[h1] <= nw[h2])) pick[r] = h1++;
            else pick[r] = h2++;
        }
        nw[made] = nw[pick[0]] + nw[pick[1]];
        parent[pick[0]] = parent[pick[1]] = made;
        ++made;
    }
    for (int i = 0; i < nsym; ++i) {
        int d = 0;
        for (int v = i; parent[v] >= 0; v = parent[v]) ++d;
        len[leaf[i]] = (uint8_t)d;
    }
    free(leaf); free(nw); free(parent);
}

/* Length-limited optimal prefix code by package-merge: lmax rounds of "pair up the current
 * list into packages, merge with the leaves (leaves first on equal weight)"; the cheapest
 * 2n - 2 items of the final list are selected, and a symbol's length is the number of
 * selected items that contain it. */
static void huffman_limited(const uint64_t *w, int nsym, int lmax, uint8_t *len)
{
    typedef struct { uint64_t w; uint8_t *cnt; } item;
    int *leaf = (int *)malloc(sizeof(int) * (size_t)nsym);
    for (int i = 0; i < nsym; ++i) leaf[i] = i;
    for (int i = 1; i < nsym; ++i) {
        int s = leaf[i], j = i - 1;
        while (j >= 0 && w[leaf[j]] > w[s]) { leaf[j + 1] = leaf[j]; --j; }
        leaf[j + 1] = s;
    }
    const int cap = 2 * nsym;
    item *cur = (item *)malloc(sizeof(item) * (size_t)cap);
    item *nxt = (item *)malloc(sizeof(item) * (size_t)cap);
    uint8_t *pool_a = (uint8_t *)calloc((size_t)cap * nsym, 1);
    uint8_t *pool_b = (uint8_t *)calloc((size_t)cap * nsym, 1);
    for (int i = 0; i < cap; ++i) { cur[i].cnt = pool_a + (size_t)i * nsym; nxt[i].cnt = pool_b + (size_t)i * nsym; }
    int ncur = nsym;
    for (int i = 0; i < nsym; ++i) { cur[i].w = w[leaf[i]]; memset(cur[i].cnt, 0, (size_t)nsym); cur[i].cnt[leaf[i]] = 1; }
    for (int round = 1; round < lmax; ++round) {
        const int npk = ncur / 2;
        int il = 0, ip = 0, o = 0;
        while (il < nsym || ip < npk) {
            uint64_t pw = 0;
            if (ip < npk) pw = cur[2 * ip].w + cur[2 * ip + 1].w;
            if (il < nsym && (ip >= npk || w[leaf[il]] <= pw)) {
                nxt[o].w = w[leaf[il]];
                memset(nxt[o].cnt, 0, (size_t)nsym);
                nxt[o].cnt[leaf[il]] = 1;
                ++il;
            } else {
                nxt[o].w = pw;
                for (int s = 0; s < nsym; ++s) nxt[o].cnt[s] = (uint8_t)(cur[2 * ip].cnt[s] + cur[2 * ip + 1].cnt[s]);
                ++ip;
            }
            ++o;
        }
        item *tmp = cur; cur = nxt; nxt = tmp;
        ncur = o;
    }
    for (int s = 0; s < nsym; ++s) len[s] = 0;
    for (int i = 0; i < 2 * nsym - 2; ++i)
        for (int s = 0; s < nsym; ++s) len[s] = (uint8_t)(len[s] + cur[i].cnt[s]);
    free(leaf); free(cur); free(nxt); free(pool_a); free(pool_b);
}

/* Code lengths for one alphabet of nsym = 2^bits symbols from its counts.  Every symbol gets
 * a code: weights are count + 1.  Plain Huffman, unless its longest code exceeds lmax, in
 * which case the length-limited optimum is used.  Returns 0, or -1 on bad arguments. */
int orc_huffman_lengths(const uint64_t *counts, int nsym, int lmax, uint8_t *len)
{
    if (nsym < 2 || lmax < 1 || lmax > 31 || ((int64_t)1 << lmax) < nsym) return -1;
    uint64_t *w = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)nsym);
    for (int i = 0; i < nsym; ++i) w[i] = counts[i] + 1;
    huffman_unlimited(w, nsym, len);
    int mx = 0;
    for (int i = 0; i < nsym; ++i) if (len[i] > mx) mx = len[i];
    if (mx > lmax) huffman_limited(w, nsym, lmax, len);
    free(w);
    return 0;
}

/* Same, with the weights given directly (no +1): used by the brute-force pins. */
int orc_huffman_lengths_raw(const uint64_t *w, int nsym, int lmax, int force_limited, uint8_t *len)
{
    if (nsym < 2 || lmax < 1 || lmax > 31 || ((int64_t)1 << lmax) < nsym) return -1;
    huffman_unlimited(w, nsym, len);
    int mx = 0;
    for (int i = 0; i < nsym; ++i) if (len[i] > mx) mx = len[i];
    if (mx > lmax || force_limited) huffman_limited(w, nsym, lmax, len);
    return 0;
}

/* Canonical code assignment: symbols ordered by (length, symbol); the first code is 0; each
 * next code is the previous plus one, shifted left by the growth in length. */
void orc_canonical_codes(const uint8_t *len, int nsym, uint32_t *code)
{
    uint32_t next = 0;
    int prev = 0;
    for (int l = 1; l <= 32; ++l)
        for (int s = 0; s < nsym; ++s)
            if (len[s] == l) {
                if (prev) next = (next + 1) << (l - prev);
                code[s] = next;
                prev = l;
            }
}

/* ------------------------------------------------------------------------------------------
 * O6 / O7. Bit stream.  Symbols are emitted pixel by pixel (p ascending), coefficient j
 * ascending inside a pixel, each with the code of its group's table, most significant code
 * bit first.  Stream bit i lives in 32-bit word i/32 at bit position 31 - (i mod 32).
 * A tile is tile_pixels consecutive pixels; a chunk is chunk_symbols consecutive symbols of
 * that order (several pixels, one pixel, or a fraction of a pixel's coefficients), with
 * tile_pixels * K a multiple of chunk_symbols, so that every tile starts a chunk.
 * Tile t starts at absolute bit tile_off[t], always a multiple of 128 (zero padding before
 * it); tile_off[n_tiles] is the padded end of the stream.  chunk_len[i] is the length of
 * chunk i in bits (16 bits each); inside a tile the chunks follow one another without gaps,
 * so a chunk starts at its tile's start plus the lengths of the tile's earlier chunks.
 * (The paper leaves the layout open: Section 3.1 only says the bit stream is accumulated in
 * external memory.)
 * ---------------------------------------------------------------------------------------- */
static void put_bit(uint32_t *stream, uint64_t pos, int bit)
{
    if (bit) stream[pos >> 5] |= (uint32_t)1 << (31 - (pos & 31));
}
static int get_bit(const uint32_t *stream, uint64_t pos)
{
    return (int)((stream[pos >> 5] >> (31 - (pos & 31))) & 1u);
}

/* Encode.  len is [groups][2^bits].  Returns the total padded length in bits, -1 if
 * cap_words is too small, -2 if a chunk is longer than 65535 bits.  stream[0 .. cap_words) is
 * zeroed first. */
int64_t orc_encode(const uint8_t *q, int64_t pixels, int k, int groups, int bits,
                   const uint8_t *len, int64_t chunk_symbols, int64_t tile_pixels,
                   uint32_t *stream, int64_t cap_words, uint16_t *chunk_len, uint64_t *tile_off)
{
    const int nsym = 1 << bits;
    uint32_t *code = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)groups * nsym);
    for (int g = 0; g < groups; ++g) orc_canonical_codes(len + (int64_t)g * nsym, nsym, code + (int64_t)g * nsym);
    memset(stream, 0, sizeof(uint32_t) * (size_t)cap_words);
    const uint64_t cap_bits = (uint64_t)cap_words * 32u;
    uint64_t pos = 0, chunk_start = 0;
    int64_t tile = 0, chunk = -1, rc = 0;
    for (int64_t p = 0; p < pixels && rc == 0; ++p) {
        if (p % tile_pixels == 0) {
            if (chunk >= 0) {
                if (pos - chunk_start > 65535u) { rc = -2; break; }
                chunk_len[chunk] = (uint16_t)(pos - chunk_start);   /* last chunk of the tile before */
            }
            pos = (pos + 127u) & ~(uint64_t)127u;
            tile_off[tile++] = pos;
            chunk_start = pos;
            ++chunk;
        }
        for (int j = 0; j < k; ++j) {
            const int64_t in_tile = (p % tile_pixels) * k + j;       /* symbol index inside the tile */
            if (in_tile > 0 && in_tile % chunk_symbols == 0) {
                if (pos - chunk_start > 65535u) { rc = -2; break; }
                chunk_len[chunk++] = (uint16_t)(pos - chunk_start);
                chunk_start = pos;
            }
            const int g = (groups == 1) ? 0 : j;
            const int s = q[p * k + j];
            const int l = len[(int64_t)g * nsym + s];
            const uint32_t cw = code[(int64_t)g * nsym + s];
            if (pos + (uint64_t)l > cap_bits) { rc = -1; break; }
            for (int b = l - 1; b >= 0; --b) put_bit(stream, pos++, (int)((cw >> b) & 1u));
        }
    }
    if (rc == 0 && chunk >= 0) {
        if (pos - chunk_start > 65535u) rc = -2;
        else chunk_len[chunk] = (uint16_t)(pos - chunk_start);
    }
    pos = (pos + 127u) & ~(uint64_t)127u;
    tile_off[tile] = pos;
    free(code);
    if (rc != 0) return rc;
    return (pos <= cap_bits) ? (int64_t)pos : -1;
}

/* Decode symbols by walking the canonical code one bit at a time: at length l the codes are
 * first[l] .. first[l] + count[l] - 1 and map to the symbols of that length in symbol
 * order.  Every chunk is decoded from its own start (tile start plus the lengths before it)
 * and must end exactly after chunk_len bits.  Returns 0, or -1 for a corrupt stream. */
int orc_decode_symbols(const uint32_t *stream, int64_t stream_words, const uint16_t *chunk_len,
                       const uint64_t *tile_off, int64_t pixels, int k, int groups, int bits,
                       const uint8_t *len, int64_t chunk_symbols, int64_t tile_pixels, uint8_t *q)
{
    const int nsym = 1 << bits;
    const uint64_t total_bits = (uint64_t)stream_words * 32u;
    int rc = 0;
    /* per group: first code, count and symbol list per length */
    uint32_t *first = (uint32_t *)calloc((size_t)groups * 33, sizeof(uint32_t));
    int *count = (int *)calloc((size_t)groups * 33, sizeof(int));
    int *start = (int *)calloc((size_t)groups * 33, sizeof(int));
    int *sorted = (int *)malloc(sizeof(int) * (size_t)groups * nsym);
    uint32_t *code = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)nsym);
    for (int g = 0; g < groups; ++g) {
        const uint8_t *lg = len + (int64_t)g * nsym;
        orc_canonical_codes(lg, nsym, code);
        int o = 0;
        for (int l = 1; l <= 32; ++l) {
            start[g * 33 + l] = o;
            int seen = 0;
            for (int s = 0; s < nsym; ++s)
                if (lg[s] == l) {
                    if (!seen) { first[g * 33 + l] = code[s]; seen = 1; }
                    sorted[(int64_t)g * nsym + o++] = s;
                    count[g * 33 + l] += 1;
                }
        }
    }
    const int64_t tile_symbols = tile_pixels * k;
    const int64_t chunks_per_tile = tile_symbols / chunk_symbols;
    const int64_t total_symbols = pixels * k;
    const int64_t n_tiles = (pixels + tile_pixels - 1) / tile_pixels;
    for (int64_t t = 0; t < n_tiles && rc == 0; ++t) {
        uint64_t chunk_start = tile_off[t];
        for (int64_t c = 0; c < chunks_per_tile && rc == 0; ++c) {
            const int64_t n0 = t * tile_symbols + c * chunk_symbols;       /* first symbol of the chunk */
            if (n0 >= total_symbols) break;
            const int64_t n1 = (n0 + chunk_symbols < total_symbols) ? n0 + chunk_symbols : total_symbols;
            const int64_t ch = t * chunks_per_tile + c;
            uint64_t pos = chunk_start;
            for (int64_t n = n0; n < n1 && rc == 0; ++n) {
                const int j = (int)(n % k);
                const int g = (groups == 1) ? 0 : j;
                uint32_t cw = 0;
                int l = 0, found = 0;
                while (l < 32 && pos < total_bits) {
                    cw = (cw << 1) | (uint32_t)get_bit(stream, pos++);
                    ++l;
                    if (count[g * 33 + l] > 0 && cw >= first[g * 33 + l] &&
                        cw - first[g * 33 + l] < (uint32_t)count[g * 33 + l]) {
                        q[n] = (uint8_t)sorted[(int64_t)g * nsym + start[g * 33 + l] + (int)(cw - first[g * 33 + l])];
                        found = 1;
                        break;
                    }
                }
                if (!found) rc = -1;
            }
            if (rc == 0 && pos - chunk_start != (uint64_t)chunk_len[ch]) rc = -1;
            chunk_start += chunk_len[ch];
        }
    }
    free(first); free(count); free(start); free(sorted); free(code);
    return rc;
}

/* O7 (second half). Inverse quantiser and inverse transform: y_hat = lo + q*step (levels
 * "scaled back to the transform domain"), x_hat = T^T y_hat + mu (T orthonormal, Section 3),
 * rounded to the tensor's type (out_bf16 != 0: bfloat16, else fp32), ties to even.  With
 * relu != 0 the layer's non-linearity follows the decoder (Section 3.1: the inverse PCA is
 * applied "before applying the non-linearity"): x_hat = max(T^T y_hat + mu, 0), then rounded. */
void orc_reconstruct(const uint8_t *q, int64_t n, int c, int64_t hw, int k, const double *mean,
                     const double *basis, double lo, double step, int out_bf16, int relu, float *xhat)
{
    double *yh = (double *)malloc(sizeof(double) * (size_t)k);
    for (int64_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < hw; ++t) {
            const uint8_t *qp = q + (i * hw + t) * k;
            for (int j = 0; j < k; ++j) yh[j] = lo + (double)qp[j] * step;
            for (int a = 0; a < c; ++a) {
                double s = 0.0;
                for (int j = 0; j < k; ++j) s += basis[(int64_t)j * c + a] * yh[j];
                s += mean[a];
                if (relu && s < 0.0) s = 0.0;
                xhat[(i * c + a) * hw + t] = out_bf16 ? (float)orc_round_bf16(s) : (float)s;
            }
        }
    free(yh);
}

/* ------------------------------------------------------------------------------------------
 * Folding (Section 3.1, "Linear transform": with 1 x 1 x C blocks the PCA is a 1 x 1
 * convolution and, like the batch normalisation, folds into the convolution that produces the
 * feature map; the inverse transform folds into the convolution that consumes it).
 * ---------------------------------------------------------------------------------------- */

/* Producer side.  The layer computes z_c = scale_c * (sum_f W[c][f] u_f + bias_c) + shift_c
 * (f runs over input channel x kernel position, `fan` of them; scale/shift are the batch
 * normalisation written as an affine map) and the encoder y_j = sum_c T[j][c] (z_c - mu_c).
 * Folded: y_j = sum_f Wf[j][f] u_f + bf[j] with
 *   Wf[j][f] = sum_c T[j][c] scale_c W[c][f],   bf[j] = sum_c T[j][c] (scale_c bias_c + shift_c - mu_c). */
void orc_fold_forward(const double *basis, const double *mean, int c, int k, const double *w, const double *bias,
                      const double *scale, const double *shift, int64_t fan, double *wf, double *bf)
{
    for (int j = 0; j < k; ++j) {
        for (int64_t f = 0; f < fan; ++f) {
            double s = 0.0;
            for (int a = 0; a < c; ++a) s += basis[(int64_t)j * c + a] * (scale[a] * w[(int64_t)a * fan + f]);
            wf[(int64_t)j * fan + f] = s;
        }
        double b = 0.0;
        for (int a = 0; a < c; ++a) b += basis[(int64_t)j * c + a] * (scale[a] * bias[a] + shift[a] - mean[a]);
        bf[j] = b;
    }
}

/* Consumer side, for a next layer that takes x_hat = T^T y_hat + mu with no non-linearity in
 * between: v_o = sum_{c,s} Wn[o][c][s] x_hat_c(s) + bias_o (s runs over the `taps` kernel
 * positions).  Folded: v_o = sum_{j,s} Wi[o][j][s] y_hat_j(s) + bi[o] with
 *   Wi[o][j][s] = sum_c Wn[o][c][s] T[j][c],   bi[o] = bias_o + sum_{c,s} Wn[o][c][s] mu_c
 * (the constant holds where every tap lies inside the map; zero padding breaks it at the border). */
void orc_fold_inverse(const double *basis, const double *mean, int c, int k, const double *wn, const double *bias,
                      int cout, int taps, double *wi, double *bi)
{
    for (int o = 0; o < cout; ++o) {
        for (int j = 0; j < k; ++j)
            for (int s = 0; s < taps; ++s) {
                double acc = 0.0;
                for (int a = 0; a < c; ++a) acc += wn[((int64_t)o * c + a) * taps + s] * basis[(int64_t)j * c + a];
                wi[((int64_t)o * k + j) * taps + s] = acc;
            }
        double b = bias[o];
        for (int a = 0; a < c; ++a)
            for (int s = 0; s < taps; ++s) b += wn[((int64_t)o * c + a) * taps + s] * mean[a];
        bi[o] = b;
    }
}

/* ------------------------------------------------------------------------------------------
 * O8. Statistics: entropy H = -sum p log2 p (Section 3.1), mean code length, and the MSE
 * distortion D = |x - x_hat|^2 / n (Section 3).
 * ---------------------------------------------------------------------------------------- */
double orc_entropy(const uint64_t *hist, int nsym)
{
    double total = 0.0, h = 0.0;
    for (int s = 0; s < nsym; ++s) total += (double)hist[s];
    if (total == 0.0) return 0.0;
    for (int s = 0; s < nsym; ++s)
        if (hist[s]) { const double p = (double)hist[s] / total; h -= p * log2(p); }
    return h;
}

double orc_mean_length(const uint64_t *hist, const uint8_t *len, int nsym)
{
    double total = 0.0, acc = 0.0;
    for (int s = 0; s < nsym; ++s) { total += (double)hist[s]; acc += (double)hist[s] * (double)len[s]; }
    return total > 0.0 ? acc / total : 0.0;
}

double orc_mse(const float *x, const float *xhat, int64_t count)
{
    double acc = 0.0;
    for (int64_t i = 0; i < count; ++i) { const double d = (double)x[i] - (double)xhat[i]; acc += d * d; }
    return count > 0 ? acc / (double)count : 0.0;
}
