// Second half of the fit on the device (Section 3.1, "Linear transform": the PCA matrix is
// pre-computed from the covariance of calibration data, which "can be updated online"): from the
// running moments to the covariance, its eigendecomposition, the rounded basis and the constants
// the codec kernels read -- without moving a C x C matrix to the host.
//
// Eigensolver: one-sided Jacobi (Hestenes).  With G = A and V = I, plane rotations applied to
// the same pair of columns of G and V make the columns of G mutually orthogonal; then G = A V,
// the columns of V are eigenvectors and, for a symmetric A, v_i . (A v_i) the eigenvalues.  The
// n / 2 column pairs of a round of a round-robin tournament are disjoint, so one launch rotates
// them all, one block per pair; n - 1 rounds visit every pair once (a sweep).  Columns are stored
// as rows (A is symmetric), so a block reads and writes contiguous memory.
#include "tc_internal.h"

#include <cuda_bf16.h>
#include <cfloat>

#define TC_CUDA(call)                                   \
    do {                                                \
        if ((call) != cudaSuccess) { cudaGetLastError(); return TC_ERR_CUDA; } \
    } while (0)

namespace {

constexpr int kPairThreads = 128;
// A covariance with a steeply graded spectrum takes 20 to 40 sweeps (the method works on the
// squared spectrum); an ordinary matrix under 10.
constexpr int kMaxSweeps = 150;

__device__ __forceinline__ double block_sum(double v, double *s_red)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    __syncthreads();                                   // s_red may still be read from the previous call
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < n_warps; ++w) t += s_red[w];   // same order in every thread
    return t;
}

// mean = s / M and covariance = (S - s s^T / M) / (M - 1) from the running moments (S holds the
// upper triangle), written as a full symmetric matrix
__global__ void moments_to_cov_kernel(const double *sum, const double *outer, double m, int c, double *mean, double *cov)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)c * c) return;
    const int a = (int)(i / c), b = (int)(i % c);
    const int lo = min(a, b), hi = max(a, b);
    const double prod = __dmul_rn(sum[lo], sum[hi]);
    cov[i] = __ddiv_rn(__dsub_rn(outer[(size_t)lo * c + hi], __ddiv_rn(prod, m)), __dsub_rn(m, 1.0));
    if (b == 0) mean[a] = __ddiv_rn(sum[a], m);
}

// centred sums (upper triangle) -> covariance, full symmetric
__global__ void scale_mirror_kernel(double *cov, int c, double denom)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)c * c) return;
    const int a = (int)(i / c), b = (int)(i % c);
    if (a > b) return;
    const double v = __ddiv_rn(cov[i], denom);
    cov[i] = v;
    cov[(size_t)b * c + a] = v;
}

__global__ void jacobi_init_kernel(const double *a, int c, double *g, double *vt, double *frob2)
{
    __shared__ double s_red[kPairThreads / 32];
    const int r = blockIdx.x;
    double acc = 0.0;
    for (int j = threadIdx.x; j < c; j += blockDim.x) {
        const double v = a[(size_t)r * c + j];
        g[(size_t)r * c + j] = v;
        vt[(size_t)r * c + j] = (j == r) ? 1.0 : 0.0;
        acc += v * v;
    }
    acc = block_sum(acc, s_red);
    if (threadIdx.x == 0) atomicAdd(frob2, acc);
}

// The pair of round `round` played at table `t` (n even): player n - 1 stays, the others rotate.
__device__ __forceinline__ void round_robin_pair(int n, int round, int t, int &p, int &q)
{
    const int m = n - 1;
    if (t == 0) { p = m; q = round % m; }
    else { p = (round + t) % m; q = (round - t + m) % m; }
    if (p > q) { const int x = p; p = q; q = x; }
}

__global__ void jacobi_round_kernel(double *g, double *vt, int c, int n_even, int round, double tol, const double *frob2,
                                    unsigned int *rotations)
{
    __shared__ double s_red[kPairThreads / 32];
    int p, q;
    round_robin_pair(n_even, round, blockIdx.x, p, q);
    if (q >= c) return;                                 // the bye of an odd n
    double *gp = g + (size_t)p * c, *gq = g + (size_t)q * c;
    double alpha = 0.0, beta = 0.0, gamma = 0.0;
    for (int j = threadIdx.x; j < c; j += blockDim.x) {
        const double x = gp[j], y = gq[j];
        alpha += x * x; beta += y * y; gamma += x * y;
    }
    alpha = block_sum(alpha, s_red);
    beta = block_sum(beta, s_red);
    gamma = block_sum(gamma, s_red);
    // The columns carry an absolute error of about eps |A| (every rotation with a large column
    // leaves that much in a small one), so their inner product is known to eps |A| times the
    // larger norm, whatever the smaller one: below that a rotation would only chase noise.  (The
    // eigenvectors of A are not determined any better than that by A itself.)
    const double bigger = sqrt(fmax(alpha, beta));
    if (fabs(gamma) <= tol * sqrt(*frob2) * bigger) return;
    const double zeta = (beta - alpha) / (2.0 * gamma);
    const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
    const double cs = 1.0 / sqrt(1.0 + t * t), sn = cs * t;
    double *vp = vt + (size_t)p * c, *vq = vt + (size_t)q * c;
    for (int j = threadIdx.x; j < c; j += blockDim.x) {
        const double x = gp[j], y = gq[j];
        gp[j] = cs * x - sn * y;
        gq[j] = sn * x + cs * y;
        const double u = vp[j], w = vq[j];
        vp[j] = cs * u - sn * w;
        vq[j] = sn * u + cs * w;
    }
    if (threadIdx.x == 0) atomicAdd(rotations, 1u);
}

// eigenvalue of row i of vt against the untouched matrix: v^T A v
__global__ void rayleigh_kernel(const double *a, const double *vt, int c, double *lambda)
{
    __shared__ double s_red[kPairThreads / 32];
    const double *v = vt + (size_t)blockIdx.x * c;
    double acc = 0.0;
    for (int r = threadIdx.x; r < c; r += blockDim.x) {
        const double *row = a + (size_t)r * c;
        double w = 0.0;
        for (int j = 0; j < c; ++j) w += row[j] * v[j];
        acc += v[r] * w;
    }
    acc = block_sum(acc, s_red);
    if (threadIdx.x == 0) lambda[blockIdx.x] = acc;
}

// Descending eigenvalues (equal ones in their original order); each vector signed so that its
// largest-magnitude entry (the first of equal ones) is positive.
__global__ void order_sign_kernel(const double *vt, const double *lambda, int c, double *evals, double *evecs)
{
    __shared__ int s_rank, s_big;
    const int i = blockIdx.x;
    if (threadIdx.x == 0) {
        const double li = lambda[i];
        int rank = 0;
        for (int j = 0; j < c; ++j) rank += (lambda[j] > li || (lambda[j] == li && j < i)) ? 1 : 0;
        const double *v = vt + (size_t)i * c;
        int big = 0;
        for (int j = 1; j < c; ++j)
            if (fabs(v[j]) > fabs(v[big])) big = j;
        s_rank = rank;
        s_big = big;
        evals[rank] = li;
    }
    __syncthreads();
    const double *v = vt + (size_t)i * c;
    const double sgn = v[s_big] < 0.0 ? -1.0 : 1.0;
    for (int j = threadIdx.x; j < c; j += blockDim.x) evecs[(size_t)s_rank * c + j] = sgn * v[j];
}

__global__ void abs_max_kernel(const double *x, long long n, double *out)
{
    __shared__ double s_red[32];
    double m = 0.0;
    for (long long i = threadIdx.x; i < n; i += blockDim.x) m = fmax(m, fabs(x[i]));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, d));
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) m = fmax(m, s_red[w]);
        *out = m;
    }
}

// nearest bfloat16 (ties to even) of a double, as a double: eight significant bits, fewer in
// the subnormal range
__device__ __forceinline__ double round_bf16(double v)
{
    if (v == 0.0 || !isfinite(v)) return v;
    int e;
    const double f = frexp(v, &e);
    int shift = 8;
    if (e - 8 < -133) shift = e + 133;
    return ldexp(rint(ldexp(f, shift)), e - shift);
}

// dtype: TC_F32 / TC_BF16 round every entry; TC_INT8: scale = *abs_max / 127, entries become
// scale * rint(v / scale), and *abs_max is replaced by the scale
__global__ void round_basis_kernel(double *basis, long long n, int dtype, double *abs_max)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    double scale = 1.0;
    if (dtype == TC_INT8) scale = __ddiv_rn(*abs_max, 127.0);
    if (i < n) {
        const double v = basis[i];
        basis[i] = dtype == TC_F32 ? (double)(float)v : dtype == TC_BF16 ? round_bf16(v) : __dmul_rn(scale, rint(__ddiv_rn(v, scale)));
    }
}
__global__ void store_scale_kernel(double *abs_max) { *abs_max = __ddiv_rn(*abs_max, 127.0); }

// The constants of a model from its basis and mean, in the summation order of a plain loop
// (one thread per output, separate multiply and add):
//   tmu[j] = sum_a T[j][a] mu[a], enc_bias[j] = -(tmu[j] + lo) / step,
//   dec_bias[a] = mu[a] + (lo + center step) sum_{j<k} T[j][a]
__global__ void model_consts_kernel(const double *basis, const double *mean, int c, int k, double lo, double step, double center,
                                    float *enc_bias, float *tmu32, float *dec_bias)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < k) {
        double s = 0.0;
        for (int a = 0; a < c; ++a) s = __dadd_rn(s, __dmul_rn(basis[(size_t)i * c + a], mean[a]));
        enc_bias[i] = (float)__ddiv_rn(-__dadd_rn(s, lo), step);
        tmu32[i] = (float)s;
    }
    if (i < c) {
        double s = 0.0;
        for (int j = 0; j < k; ++j) s = __dadd_rn(s, basis[(size_t)j * c + i]);
        dec_bias[i] = (float)__dadd_rn(mean[i], __dmul_rn(__dadd_rn(lo, __dmul_rn(center, step)), s));
    }
}

// bf16 operand copies: b[j][a] and its transpose bt[a][j] (an 8-bit basis as its integers)
__global__ void basis_bf16_kernel(const double *basis, int c, int k, double scale_or_zero, __nv_bfloat16 *b, __nv_bfloat16 *bt)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)k * c) return;
    const int j = (int)(i / c), a = (int)(i % c);
    const double v = basis[i];
    const float f = scale_or_zero != 0.0 ? (float)rint(__ddiv_rn(v, scale_or_zero)) : (float)v;
    const __nv_bfloat16 h = __float2bfloat16(f);
    b[i] = h;
    bt[(size_t)a * k + j] = h;
}

}  // namespace

tc_status tc_launch_moments_to_cov(const double *sum, const double *outer, long long count, int c, double *mean, double *cov,
                                   cudaStream_t s)
{
    const long long n = (long long)c * c;
    moments_to_cov_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(sum, outer, (double)count, c, mean, cov);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_scale_mirror(double *cov, int c, double denom, cudaStream_t s)
{
    const long long n = (long long)c * c;
    scale_mirror_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(cov, c, denom);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

size_t tc_eigh_device_workspace_bytes(int c) { return (2 * (size_t)c * c + (size_t)c + 2) * sizeof(double); }

// a: [c][c] symmetric, DEVICE, left untouched.  evals [c], evecs [c][c] (row j = eigenvector of
// evals[j]), DEVICE.  `work`: tc_eigh_device_workspace_bytes(c) bytes, DEVICE.  Synchronises the
// stream once per sweep (a 4-byte read of the rotation count).
tc_status tc_eigh_device(const double *a, int c, double *evals, double *evecs, void *work, int *sweeps_out, cudaStream_t s)
{
    if (c < 1) return TC_ERR_INVALID_ARG;
    double *g = static_cast<double *>(work), *vt = g + (size_t)c * c, *lambda = vt + (size_t)c * c, *frob2 = lambda + c;
    unsigned int *rotations = reinterpret_cast<unsigned int *>(frob2 + 1);
    TC_CUDA(cudaMemsetAsync(frob2, 0, 2 * sizeof(double), s));
    jacobi_init_kernel<<<c, kPairThreads, 0, s>>>(a, c, g, vt, frob2);
    const int n_even = (c + 1) & ~1;
    const double tol = (double)(c < 16 ? 16 : c) * DBL_EPSILON;
    int sweeps = 0;
    bool converged = c == 1;
    for (; sweeps < kMaxSweeps && !converged; ++sweeps) {
        TC_CUDA(cudaMemsetAsync(rotations, 0, sizeof(unsigned int), s));
        for (int round = 0; round < n_even - 1; ++round)
            jacobi_round_kernel<<<n_even / 2, kPairThreads, 0, s>>>(g, vt, c, n_even, round, tol, frob2, rotations);
        unsigned int n_rot = 0;
        TC_CUDA(cudaMemcpyAsync(&n_rot, rotations, sizeof(n_rot), cudaMemcpyDeviceToHost, s));
        TC_CUDA(cudaStreamSynchronize(s));
        converged = n_rot == 0;
    }
    if (sweeps_out) *sweeps_out = sweeps;
    if (!converged) return TC_ERR_NOT_CONVERGED;
    rayleigh_kernel<<<c, kPairThreads, 0, s>>>(a, vt, c, lambda);
    order_sign_kernel<<<c, kPairThreads, 0, s>>>(vt, lambda, c, evals, evecs);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

// Rounds the basis in place to `dtype`.  scale_slot (DEVICE, one double) receives the scale of an
// 8-bit basis (untouched otherwise).
tc_status tc_launch_round_basis(double *basis, int c, int dtype, double *scale_slot, cudaStream_t s)
{
    const long long n = (long long)c * c;
    if (dtype == TC_INT8) abs_max_kernel<<<1, 1024, 0, s>>>(basis, n, scale_slot);
    round_basis_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(basis, n, dtype, scale_slot);
    if (dtype == TC_INT8) store_scale_kernel<<<1, 1, 0, s>>>(scale_slot);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_model_consts(const double *basis, const double *mean, int c, int k, double lo, double step, double center,
                                 float *enc_bias, float *tmu32, float *dec_bias, cudaStream_t s)
{
    model_consts_kernel<<<(c + 127) / 128, 128, 0, s>>>(basis, mean, c, k, lo, step, center, enc_bias, tmu32, dec_bias);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_basis_bf16(const double *basis, int c, int k, double basis_scale, bool int8, void *b, void *bt, cudaStream_t s)
{
    const long long n = (long long)k * c;
    basis_bf16_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(basis, c, k, int8 ? basis_scale : 0.0,
                                                                 static_cast<__nv_bfloat16 *>(b), static_cast<__nv_bfloat16 *>(bt));
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
