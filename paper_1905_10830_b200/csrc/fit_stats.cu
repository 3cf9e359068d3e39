// Calibration and statistics kernels (off the timed path): channel sums, centred covariance
// and the range of coefficient 0 for the fit (Section 3; Section 3.1 "Linear transform" and
// "Quantization"), symbol histograms for the entropy and the codebook (Section 3.1 "Variable
// length coding"), and the squared error of a round trip (Section 3, MSE distortion).
#include "device_utils.cuh"

namespace {

using namespace tcdev;

// sums[c] += sum over pixels of x[n][c][:]  -- one block per (image, channel) row.
template <typename TIn>
__global__ void channel_sums_kernel(const TIn *x, int c, int hw, double *sums)
{
    const long long row = blockIdx.x;                  // n * c + channel
    const TIn *src = x + row * hw;
    double s = 0.0;
    for (int i = threadIdx.x; i < hw; i += blockDim.x) s += load_as_double(src + i);
    __shared__ double red[32];
    for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int i = 0; i < (int)(blockDim.x + 31) / 32; ++i) tot += red[i];
        atomicAdd(sums + (row % c), tot);
    }
}

// cov[a][b] += sum over a slab of pixels of (x_a - mu_a)(x_b - mu_b) for a 16 x 16 block of
// channel pairs; grid = (pixel slabs, channel-block pairs with b-block >= a-block).
constexpr int kCovTile = 16;
constexpr int kCovSlab = 128;

template <typename TIn>
__global__ void __launch_bounds__(256) covariance_kernel(const TIn *x, int n, int c, int hw, const double *mean,
                                                         double *cov, int blocks_per_dim)
{
    __shared__ double sa[kCovTile][kCovSlab + 1];
    __shared__ double sb[kCovTile][kCovSlab + 1];
    // decode the (ablk <= bblk) pair from blockIdx.y
    int pair = blockIdx.y, ablk = 0;
    while (pair >= blocks_per_dim - ablk) { pair -= blocks_per_dim - ablk; ++ablk; }
    const int bblk = ablk + pair;
    const long long pixels = (long long)n * hw;
    const int ti = threadIdx.x / kCovTile, tj = threadIdx.x % kCovTile;
    double acc = 0.0;
    for (long long p0 = (long long)blockIdx.x * kCovSlab; p0 < pixels; p0 += (long long)gridDim.x * kCovSlab) {
        __syncthreads();
        for (int i = threadIdx.x; i < kCovTile * kCovSlab; i += blockDim.x) {
            const int ch = i / kCovSlab, pp = i % kCovSlab;
            const long long p = p0 + pp;
            double va = 0.0, vb = 0.0;
            if (p < pixels) {
                const long long img = p / hw, s = p - img * hw;
                const int ca = ablk * kCovTile + ch, cb = bblk * kCovTile + ch;
                if (ca < c) va = load_as_double(x + (img * c + ca) * hw + s) - mean[ca];
                if (cb < c) vb = load_as_double(x + (img * c + cb) * hw + s) - mean[cb];
            }
            sa[ch][pp] = va;
            sb[ch][pp] = vb;
        }
        __syncthreads();
#pragma unroll 8
        for (int pp = 0; pp < kCovSlab; ++pp) acc += sa[ti][pp] * sb[tj][pp];
    }
    const int ca = ablk * kCovTile + ti, cb = bblk * kCovTile + tj;
    if (ca < c && cb < c) atomicAdd(cov + (long long)ca * c + cb, acc);
}

// Per-block min and max of coefficient 0: y0 = sum_c T[0][c] (x_c - mu_c), summed in channel
// order without contraction.
constexpr int kRangeThreads = 256;

template <typename TIn>
__global__ void __launch_bounds__(kRangeThreads) range0_kernel(const TIn *x, int n, int c, int hw, const double *mean,
                                                               const double *row0, double *block_minmax)
{
    extern __shared__ double s_rm[];      // [2][c]: row0, mean
    for (int i = threadIdx.x; i < c; i += blockDim.x) { s_rm[i] = row0[i]; s_rm[c + i] = mean[i]; }
    __syncthreads();
    const long long pixels = (long long)n * hw;
    double mn = INFINITY, mx = -INFINITY;
    for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < pixels; p += (long long)gridDim.x * blockDim.x) {
        const long long img = p / hw, s = p - img * hw;
        const TIn *src = x + img * c * (long long)hw + s;
        double y = 0.0;
        for (int cc = 0; cc < c; ++cc)
            y = __dadd_rn(y, __dmul_rn(s_rm[cc], __dsub_rn(load_as_double(src + (long long)cc * hw), s_rm[c + cc])));
        mn = fmin(mn, y);
        mx = fmax(mx, y);
    }
    __shared__ double rmin[kRangeThreads / 32], rmax[kRangeThreads / 32];
    for (int d = 16; d > 0; d >>= 1) {
        mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, d));
        mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    }
    if ((threadIdx.x & 31) == 0) { rmin[threadIdx.x >> 5] = mn; rmax[threadIdx.x >> 5] = mx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < kRangeThreads / 32; ++i) { mn = fmin(mn, rmin[i]); mx = fmax(mx, rmax[i]); }
        block_minmax[2 * blockIdx.x] = mn;
        block_minmax[2 * blockIdx.x + 1] = mx;
    }
}

// hist[g][s] += 1 for every symbol; g = coefficient index (groups == k) or 0.
__global__ void __launch_bounds__(256) histogram_kernel(const uint8_t *sym, long long pixels, int k, int groups,
                                                        int bits, unsigned long long *hist)
{
    __shared__ unsigned int local[256];
    const int nsym = 1 << bits;
    const long long total = pixels * k;
    if (groups == 1) {
        for (int i = threadIdx.x; i < nsym; i += blockDim.x) local[i] = 0;
        __syncthreads();
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
            atomicAdd(local + sym[i], 1u);
        __syncthreads();
        for (int i = threadIdx.x; i < nsym; i += blockDim.x)
            if (local[i]) atomicAdd(hist + i, (unsigned long long)local[i]);
    } else {
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
            atomicAdd(hist + (i % k) * nsym + sym[i], 1ull);
    }
}

template <typename TIn>
__global__ void __launch_bounds__(256) sqerr_kernel(const TIn *x, const TIn *xhat, long long count, double *sum_sq,
                                                    unsigned long long *zeros)
{
    double acc = 0.0;
    unsigned int z = 0;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        const double a = load_as_double(x + i), d = a - load_as_double(xhat + i);
        acc += d * d;
        z += (a == 0.0);
    }
    for (int d = 16; d > 0; d >>= 1) {
        acc += __shfl_xor_sync(0xffffffffu, acc, d);
        z += __shfl_xor_sync(0xffffffffu, z, d);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(sum_sq, acc);
        atomicAdd(zeros, (unsigned long long)z);
    }
}

inline bool launched() { return cudaGetLastError() == cudaSuccess; }

}  // namespace

tc_status tc_launch_channel_sums(const void *x, int dtype, int n, int c, int hw, double *sums, cudaStream_t s)
{
    const unsigned int rows = (unsigned int)((long long)n * c);
    if (rows == 0) return TC_OK;
    if (dtype == TC_F32) channel_sums_kernel<float><<<rows, 128, 0, s>>>((const float *)x, c, hw, sums);
    else channel_sums_kernel<__nv_bfloat16><<<rows, 128, 0, s>>>((const __nv_bfloat16 *)x, c, hw, sums);
    return launched() ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_covariance(const void *x, int dtype, int n, int c, int hw, const double *mean, double *cov,
                               cudaStream_t s)
{
    const int bpd = (c + kCovTile - 1) / kCovTile;
    const int pairs = bpd * (bpd + 1) / 2;
    const long long pixels = (long long)n * hw;
    long long slabs = (pixels + kCovSlab - 1) / kCovSlab;
    const long long want = (4096 + pairs - 1) / pairs;       // enough blocks to fill the device
    if (slabs > want) slabs = want;
    if (slabs < 1) slabs = 1;
    dim3 grid((unsigned int)slabs, (unsigned int)pairs);
    if (dtype == TC_F32) covariance_kernel<float><<<grid, 256, 0, s>>>((const float *)x, n, c, hw, mean, cov, bpd);
    else covariance_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)x, n, c, hw, mean, cov, bpd);
    return launched() ? TC_OK : TC_ERR_CUDA;
}

int tc_range0_max_blocks(long long pixels)
{
    long long b = (pixels + kRangeThreads - 1) / kRangeThreads;
    if (b > 1024) b = 1024;
    if (b < 1) b = 1;
    return (int)b;
}

tc_status tc_launch_range0(const void *x, int dtype, int n, int c, int hw, const double *mean, const double *row0,
                           double *block_minmax, int *n_blocks_out, cudaStream_t s)
{
    const int blocks = tc_range0_max_blocks((long long)n * hw);
    *n_blocks_out = blocks;
    const size_t smem = sizeof(double) * 2 * (size_t)c;
    if (dtype == TC_F32)
        range0_kernel<float><<<blocks, kRangeThreads, smem, s>>>((const float *)x, n, c, hw, mean, row0, block_minmax);
    else
        range0_kernel<__nv_bfloat16><<<blocks, kRangeThreads, smem, s>>>((const __nv_bfloat16 *)x, n, c, hw, mean, row0,
                                                                         block_minmax);
    return launched() ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_histogram(const uint8_t *sym, long long pixels, int k, int groups, int bits,
                              unsigned long long *hist, cudaStream_t s)
{
    long long blocks = (pixels * k + 256 * 64 - 1) / (256 * 64);
    if (blocks > 2048) blocks = 2048;
    if (blocks < 1) blocks = 1;
    histogram_kernel<<<(unsigned int)blocks, 256, 0, s>>>(sym, pixels, k, groups, bits, hist);
    return launched() ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_sqerr(const void *x, const void *xhat, int dtype, long long count, double *sum_sq,
                          unsigned long long *zeros, cudaStream_t s)
{
    long long blocks = (count + 256 * 32 - 1) / (256 * 32);
    if (blocks > 4096) blocks = 4096;
    if (blocks < 1) blocks = 1;
    if (dtype == TC_F32)
        sqerr_kernel<float><<<(unsigned int)blocks, 256, 0, s>>>((const float *)x, (const float *)xhat, count, sum_sq, zeros);
    else
        sqerr_kernel<__nv_bfloat16><<<(unsigned int)blocks, 256, 0, s>>>((const __nv_bfloat16 *)x, (const __nv_bfloat16 *)xhat,
                                                                         count, sum_sq, zeros);
    return launched() ? TC_OK : TC_ERR_CUDA;
}
