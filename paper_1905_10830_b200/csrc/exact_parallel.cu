// Exact (fp64) projection and reconstruction with one thread per output value, for tensors of
// few pixels (the fp32 maps of one image: Section 4's ResNet-18 layers at batch 1).
//
// The exact encode / decode kernels give a pixel to a thread, which then walks C x K products
// alone: a 512 x 7 x 7 map keeps 49 threads busy for milliseconds.  Here every (pixel,
// coefficient) pair of the projection y_j = sum_c T[j][c] (x_c - mu_c) (Section 3, first
// equation) and every (pixel, channel) pair of the inverse x_hat_c = sum_j T[j][c] y_hat_j + mu_c
// is a thread of its own.  Each thread adds its products in the same order and with the same
// unfused double operations as the per-pixel kernels, so the results are bit-identical to theirs
// (and to the definition evaluated in fp64); the entropy coder then runs in the per-pixel kernels
// on the symbols these kernels leave in memory.
#include "device_utils.cuh"

namespace {

using namespace tcdev;

constexpr int kPx = 32;        // pixels per block (one warp row: loads along the pixels coalesce)
constexpr int kOut = 16;       // coefficients (encode) or channels (decode) per block

template <typename TIn>
__global__ void __launch_bounds__(kPx * kOut) project_quantise_kernel(EncodeArgs a, uint8_t *sym)
{
    __shared__ uint8_t s_q[kPx][kOut];
    __shared__ float s_y[kPx][kOut + 1];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const long long p = (long long)blockIdx.x * kPx + tx;
    const int j = blockIdx.y * kOut + ty;
    const bool valid = p < a.pixels && j < a.k;
    const int nsym = 1 << a.bits;
    const double top = (double)(nsym - 1);
    unsigned int clamped = 0;
    if (valid) {
        const TIn *xin = reinterpret_cast<const TIn *>(a.x);
        const long long img = p / a.hw;
        const TIn *xp = xin + img * a.c * (long long)a.hw + (p - img * a.hw);
        const double *row = a.basis64 + (long long)j * a.c;
        double acc = 0.0;
#pragma unroll 4
        for (int cc = 0; cc < a.c; ++cc) {
            const double d = __dsub_rn(load_as_double(xp + (long long)cc * a.hw), __ldg(a.mean64 + cc));
            acc = __dadd_rn(acc, __dmul_rn(__ldg(row + cc), d));
        }
        const double u = __ddiv_rn(__dsub_rn(acc, a.lo), a.step);
        double r = rint(u);
        if (u < 0.0 || u > top) clamped = 1;
        r = fmin(fmax(r, 0.0), top);
        s_q[tx][ty] = (uint8_t)(unsigned int)r;
        s_y[tx][ty] = (float)acc;
    }
    if (a.clamped) {
        const unsigned int n = __popc(__ballot_sync(0xffffffffu, clamped != 0));
        if (tx == 0 && n) atomicAdd(a.clamped, (unsigned long long)n);
    }
    __syncthreads();
    // a pixel's kOut symbols are contiguous in [P][K]: rows of the block leave in 16-byte pieces
    const int t = ty * kPx + tx;
    const int j0 = blockIdx.y * kOut;
    for (int i = t; i < kPx * kOut; i += kPx * kOut) {
        const int px = i / kOut, jj = i - px * kOut;
        const long long pp = (long long)blockIdx.x * kPx + px;
        if (pp < a.pixels && j0 + jj < a.k) {
            const uint8_t q = s_q[px][jj];
            sym[pp * a.k + j0 + jj] = q;
            if (a.dbg_sym) a.dbg_sym[pp * a.k + j0 + jj] = q;
            if (a.dbg_coef) a.dbg_coef[pp * a.k + j0 + jj] = s_y[px][jj];
        }
    }
}

template <typename TOut>
__global__ void __launch_bounds__(kPx * kOut) reconstruct_kernel(DecodeArgs a, const uint8_t *sym)
{
    extern __shared__ __align__(16) unsigned char s_sym[];          // [kPx][K] symbols of the block's pixels
    const int tx = threadIdx.x, ty = threadIdx.y;
    const long long p0 = (long long)blockIdx.x * kPx;
    const int n_px = (int)min((long long)kPx, a.pixels - p0);
    for (int i = ty * kPx + tx; i < n_px * a.k; i += kPx * kOut) s_sym[i] = sym[p0 * a.k + i];
    __syncthreads();
    const long long p = p0 + tx;
    const int c = blockIdx.y * kOut + ty;
    if (tx >= n_px || c >= a.c) return;
    double acc = 0.0;
#pragma unroll 4
    for (int j = 0; j < a.k; ++j) {
        const double yh = __dadd_rn(a.lo, __dmul_rn((double)s_sym[tx * a.k + j], a.step));
        acc = __dadd_rn(acc, __dmul_rn(__ldg(a.basis64 + (long long)j * a.c + c), yh));
    }
    double v = __dadd_rn(acc, __ldg(a.mean64 + c));
    if (a.relu && v < 0.0) v = 0.0;
    const long long img = p / a.hw;
    TOut *out = reinterpret_cast<TOut *>(a.xhat);
    store_rounded(out + img * a.c * (long long)a.hw + (long long)c * a.hw + (p - img * a.hw), v);
}

}  // namespace

tc_status tc_launch_project_quantise(const EncodeArgs &a, int dtype, uint8_t *sym, cudaStream_t s)
{
    if (a.pixels <= 0) return TC_OK;
    const dim3 block(kPx, kOut), grid((unsigned int)((a.pixels + kPx - 1) / kPx), (unsigned int)((a.k + kOut - 1) / kOut));
    if (dtype == TC_F32) project_quantise_kernel<float><<<grid, block, 0, s>>>(a, sym);
    else project_quantise_kernel<__nv_bfloat16><<<grid, block, 0, s>>>(a, sym);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_reconstruct(const DecodeArgs &a, int dtype, const uint8_t *sym, cudaStream_t s)
{
    if (a.pixels <= 0) return TC_OK;
    const dim3 block(kPx, kOut), grid((unsigned int)((a.pixels + kPx - 1) / kPx), (unsigned int)((a.c + kOut - 1) / kOut));
    const size_t smem = (size_t)kPx * a.k;
    if (dtype == TC_F32) reconstruct_kernel<float><<<grid, block, smem, s>>>(a, sym);
    else reconstruct_kernel<__nv_bfloat16><<<grid, block, smem, s>>>(a, sym);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
