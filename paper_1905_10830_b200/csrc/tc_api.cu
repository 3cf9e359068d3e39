// Host side of the C ABI declared in include/tc.h: handles, argument checks, table building
// and kernel launches.  No step of the coding path runs on the host.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "tc_internal.h"

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link the
// driver library (it must load, for the host-side entry points, on machines without a driver).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return (EncodeTiledFn)p;
    }();
    return fn;
}


#define TC_CUDA(call)                                   \
    do {                                                \
        if ((call) != cudaSuccess) { cudaGetLastError(); return TC_ERR_CUDA; } \
    } while (0)

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

double round_to_dtype(double v, int dtype)
{
    if (dtype == TC_F32) return (double)(float)v;
    if (v == 0.0 || !std::isfinite(v)) return v;
    int e;
    const double f = std::frexp(v, &e);                 // |f| in [0.5, 1)
    int shift = 8;                                      // 8 significant bits
    if (e - 8 < -133) shift = e + 133;                  // bfloat16 subnormals
    return std::ldexp(std::nearbyint(std::ldexp(f, shift)), e - shift);
}

template <typename T>
tc_status upload(T **dst, const std::vector<T> &src)
{
    *dst = nullptr;
    if (src.empty()) return TC_OK;
    TC_CUDA(cudaMalloc((void **)dst, src.size() * sizeof(T)));
    TC_CUDA(cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice));
    return TC_OK;
}

bool valid_tensor(const tc_tensor *t)
{
    return t && t->n >= 0 && t->c > 0 && t->h > 0 && t->w > 0 && (t->dtype == TC_F32 || t->dtype == TC_BF16) &&
           (t->data != nullptr || t->n == 0);
}

// Chunk shape: `cp` pixels per chunk, or `splits` chunks per pixel when cp == 1.  Defaults
// keep the side information at 16 bits per 96 to 255 symbols (0.06 to 0.17 bit per value): a chunk is
// one decoder thread's work, and a tile of 128 pixels wants as many of them as the rate allows.
struct ChunkShape {
    int cp, splits;
    long long chunks(long long pixels) const { return splits > 1 ? pixels * splits : (pixels + cp - 1) / cp; }
};

bool resolve_chunks(const tc_encode_params *p, int k, int max_len, ChunkShape *out)
{
    int cp = 1;
    if (p && p->chunk_pixels) cp = p->chunk_pixels;
    else while (cp < TC_TILE_PIXELS && cp * k < 96) cp <<= 1;       // at least 96 symbols per chunk: 16 bits of side information per 96 .. 255 symbols
    if (cp < 1 || cp > TC_TILE_PIXELS || (cp & (cp - 1)) != 0) return false;
    // default: a chunk of 128 .. 255 symbols where the shape allows it -- two chunks per pixel
    // from 256 coefficients, four from 512
    int splits = (p && p->pixel_splits) ? p->pixel_splits
                 : (cp == 1 && k >= 512 && k % 64 == 0) ? 4 : ((cp == 1 && k >= 256 && k % 32 == 0) ? 2 : 1);
    if (splits != 1 && splits != 2 && splits != 4) return false;
    if (splits > 1 && (cp != 1 || k % (8 * splits) != 0)) return false;
    if ((long long)cp * k / splits * max_len > 65535) return false;     // a chunk length has 16 bits
    out->cp = cp;
    out->splits = splits;
    return true;
}

tc_status ensure_scratch(tc_ctx *ctx, size_t bytes)
{
    if (bytes <= ctx->scratch_bytes) return TC_OK;
    if (ctx->scratch) { TC_CUDA(cudaDeviceSynchronize()); cudaFree(ctx->scratch); ctx->scratch = nullptr; ctx->scratch_bytes = 0; }
    size_t want = std::max<size_t>(bytes, 1 << 20);
    TC_CUDA(cudaMalloc(&ctx->scratch, want));
    ctx->scratch_bytes = want;
    return TC_OK;
}

// The host copy of a model's basis, fetched from the device at first use.
const std::vector<double> *host_basis(const tc_model *m)
{
    if (m->basis.empty() && m->d_basis64) {
        DeviceGuard guard(m->device);
        m->basis.resize((size_t)m->c * m->c);
        if (cudaMemcpy(m->basis.data(), m->d_basis64, m->basis.size() * sizeof(double), cudaMemcpyDeviceToHost) != cudaSuccess) {
            cudaGetLastError();
            m->basis.clear();
            return nullptr;
        }
    }
    return &m->basis;
}

// Completes a model whose basis and mean are on the device (d_basis64, d_mean64) and whose
// scalars are set: the constants and operand copies the codec kernels read are computed there.
tc_status finish_model(tc_model *m)
{
    const int c = m->c, k = m->k;
    // The inverse projection runs on symbols centred on the level nearest to y = 0, so that the
    // accumulators stay small and no large terms cancel in fp32:
    // x_hat = step * sum_j T[j][c] (q_j - center) + mu_c + (lo + center*step) * sum_j T[j][c]
    const double top = (double)((1 << m->bits) - 1);
    m->center = (int)std::min(top, std::max(0.0, std::nearbyint(-m->lo / m->step)));
    tc_status st;
    if (!m->d_basis64 && (st = upload(&m->d_basis64, m->basis)) != TC_OK) return st;
    if (!m->d_mean64 && (st = upload(&m->d_mean64, m->mean)) != TC_OK) return st;
    TC_CUDA(cudaMalloc((void **)&m->d_enc_bias, sizeof(float) * k));
    TC_CUDA(cudaMalloc((void **)&m->d_tmu32, sizeof(float) * k));
    TC_CUDA(cudaMalloc((void **)&m->d_dec_bias, sizeof(float) * c));
    if ((st = tc_launch_model_consts(m->d_basis64, m->d_mean64, c, k, m->lo, m->step, (double)m->center, m->d_enc_bias,
                                     m->d_tmu32, m->d_dec_bias, nullptr)) != TC_OK) return st;
    if (m->basis_dtype == TC_BF16 || m->basis_dtype == TC_INT8) {
        // an 8-bit basis goes to the bf16 kernels as its integers (exact in bf16); the scale is
        // folded into their quantiser and dequantiser constants
        TC_CUDA(cudaMalloc((void **)&m->d_basis_bf16, sizeof(__nv_bfloat16) * (size_t)k * c));
        TC_CUDA(cudaMalloc((void **)&m->d_basis_t_bf16, sizeof(__nv_bfloat16) * (size_t)k * c));
        if ((st = tc_launch_basis_bf16(m->d_basis64, c, k, m->basis_scale, m->basis_dtype == TC_INT8, m->d_basis_bf16,
                                       m->d_basis_t_bf16, nullptr)) != TC_OK) return st;
        // Tensor map for the kernels that stream the basis: boxes of 256 coefficient rows x 32
        // channels (64 bytes), written with the 64-byte swizzle the MMA descriptor names.  Needs
        // rows of a multiple of 16 bytes; without a map those kernels copy the basis with cp.async.
        m->has_basis_map = false;
        const EncodeTiledFn encode_tiled = encode_tiled_fn();
        if (encode_tiled && c % 16 == 0) {
            const cuuint64_t dims[2] = {(cuuint64_t)c, (cuuint64_t)k};
            const cuuint64_t strides[1] = {(cuuint64_t)c * 2};
            const cuuint32_t box[2] = {32u, 256u};
            const cuuint32_t elem[2] = {1u, 1u};
            const CUresult rc = encode_tiled(&m->basis_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, m->d_basis_bf16, dims,
                                                       strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            m->has_basis_map = rc == CUDA_SUCCESS;
        }
        // and for the decoder: the transposed basis in boxes of 128 channel rows x 64 coefficients
        m->has_basis_t_map = false;
        if (encode_tiled && k % 16 == 0) {
            const cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)c};
            const cuuint64_t strides[1] = {(cuuint64_t)k * 2};
            const cuuint32_t box[2] = {64u, 128u};
            const cuuint32_t elem[2] = {1u, 1u};
            const CUresult rc = encode_tiled(&m->basis_t_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, m->d_basis_t_bf16, dims,
                                                       strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            m->has_basis_t_map = rc == CUDA_SUCCESS;
        }
    }
    TC_CUDA(cudaStreamSynchronize(nullptr));
    return TC_OK;
}

tc_status finish_codebook(tc_codebook *cb)
{
    const int nsym = 1 << cb->bits;
    int mx = 0;
    for (uint8_t l : cb->lengths) mx = std::max<int>(mx, l);
    cb->max_len = mx;
    cb->lut_bits = mx;
    // canonical codes give the first symbol of the shortest length the all-zero code: with a
    // one-bit code that is the single bit 0, and a run of that symbol is a run of zero bits
    cb->modal = -1;
    if (cb->groups == 1)
        for (int s = 0; s < nsym && cb->modal < 0; ++s)
            if (cb->lengths[s] == 1) cb->modal = s;
    std::vector<uint32_t> enc((size_t)cb->groups * nsym);
    std::vector<uint16_t> lut((size_t)cb->groups << cb->lut_bits);
    std::vector<uint32_t> lut32((size_t)cb->groups << cb->lut_bits);
    std::vector<uint32_t> code(nsym);
    for (int g = 0; g < cb->groups; ++g) {
        const uint8_t *len = cb->lengths.data() + (size_t)g * nsym;
        tc_canonical_codes_host(len, nsym, code.data());
        for (int s = 0; s < nsym; ++s) {
            enc[(size_t)g * nsym + s] = (code[s] << 8) | len[s];
            // every table index whose leading bits equal the code decodes to this symbol
            const uint32_t first = code[s] << (cb->lut_bits - len[s]);
            const uint32_t span = 1u << (cb->lut_bits - len[s]);
            const float as_float = (float)s;
            uint32_t fbits;
            std::memcpy(&fbits, &as_float, 4);               // small integers are exact in bf16
            for (uint32_t i = 0; i < span; ++i) {
                lut[((size_t)g << cb->lut_bits) + first + i] = (uint16_t)((s << 8) | len[s]);
                lut32[((size_t)g << cb->lut_bits) + first + i] = (fbits & 0xffff0000u) | ((uint32_t)s << 8) | len[s];
            }
        }
    }
    tc_status st;
    if ((st = upload(&cb->d_enc, enc)) != TC_OK) return st;
    if ((st = upload(&cb->d_lut32, lut32)) != TC_OK) return st;
    return upload(&cb->d_lut, lut);
}

bool kraft_complete(const uint8_t *len, int nsym, int lmax)
{
    unsigned long long sum = 0;
    for (int s = 0; s < nsym; ++s) {
        if (len[s] < 1 || len[s] > lmax) return false;
        sum += 1ull << (lmax - len[s]);
    }
    return sum == (1ull << lmax);
}

}  // namespace

extern "C" {

const char *tc_status_string(tc_status s)
{
    switch (s) {
        case TC_OK: return "ok";
        case TC_ERR_INVALID_ARG: return "invalid argument";
        case TC_ERR_UNSUPPORTED: return "unsupported configuration";
        case TC_ERR_BUFFER_TOO_SMALL: return "output buffer too small";
        case TC_ERR_CUDA: return "CUDA error";
        case TC_ERR_CORRUPT_STREAM: return "corrupt stream";
        case TC_ERR_TIMEOUT: return "device-side wait timed out";
        case TC_ERR_NOT_CONVERGED: return "eigensolver did not converge";
    }
    return "unknown status";
}

tc_status tc_create(tc_ctx **out, int device)
{
    if (!out) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return TC_ERR_CUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return TC_ERR_CUDA;
    tc_ctx *ctx = new (std::nothrow) tc_ctx();
    if (!ctx) return TC_ERR_CUDA;
    ctx->device = device;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return TC_ERR_CUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    if (cudaMalloc((void **)&ctx->d_status, 64) != cudaSuccess || cudaMemset(ctx->d_status, 0, 64) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return TC_ERR_CUDA;
    }
    *out = ctx;
    return TC_OK;
}

void tc_destroy(tc_ctx *ctx)
{
    if (!ctx) return;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->scratch) cudaFree(ctx->scratch);
    if (ctx->host_arena) cudaFree(ctx->host_arena);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    for (int i = 0; i < 2; ++i) {
        if (ctx->ev_in[i]) cudaEventDestroy(ctx->ev_in[i]);
        if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
        if (ctx->ev_out[i]) cudaEventDestroy(ctx->ev_out[i]);
    }
    if (ctx->chunk_bits) cudaFreeHost(ctx->chunk_bits);
    for (int i = 0; i < 4; ++i) {
        if (ctx->many_streams[i]) cudaStreamDestroy(ctx->many_streams[i]);
        if (ctx->many_join[i]) cudaEventDestroy(ctx->many_join[i]);
    }
    if (ctx->many_fork) cudaEventDestroy(ctx->many_fork);
    for (tc_codebook *cb : ctx->stats_cb) tc_codebook_free(cb);
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
}

void tc_force_exact_path(tc_ctx *ctx, int on)
{
    if (ctx) ctx->force_exact = (on == 2 || on == 3) ? on : (on ? 1 : 0);
}

int tc_last_path(const tc_ctx *ctx, int decode)
{
    if (!ctx) return -1;
    return decode ? ctx->last_decode_path : ctx->last_encode_path;
}

tc_status tc_get_status(tc_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    unsigned int word = 0;
    TC_CUDA(cudaMemcpyAsync(&word, ctx->d_status, sizeof(word), cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaStreamSynchronize(s));
    if (word != 0) {
        TC_CUDA(cudaMemsetAsync(ctx->d_status, 0, sizeof(word), s));
        TC_CUDA(cudaStreamSynchronize(s));
    }
    return (tc_status)word;
}

// ---- model ------------------------------------------------------------------------------

tc_status tc_model_import(tc_ctx *ctx, const tc_model_desc *d, tc_model **out)
{
    if (!ctx || !d || !out || !d->basis || !d->mean) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    if (d->c < 1 || d->k < 1 || d->k > d->c || !(d->step > 0.0) || !std::isfinite(d->lo)) return TC_ERR_INVALID_ARG;
    if (d->bits < 1 || d->bits > 8 || d->c > TC_MAX_C) return TC_ERR_UNSUPPORTED;
    if (d->basis_dtype != TC_F32 && d->basis_dtype != TC_BF16 && d->basis_dtype != TC_INT8) return TC_ERR_INVALID_ARG;
    if (d->basis_dtype == TC_INT8) {
        // every entry must be an integer in [-127, 127] times the scale
        if (!(d->basis_scale > 0.0) || !std::isfinite(d->basis_scale)) return TC_ERR_INVALID_ARG;
        for (size_t i = 0; i < (size_t)d->c * d->c; ++i) {
            const double n = d->basis[i] / d->basis_scale;
            if (std::fabs(n - std::nearbyint(n)) > 1e-9 || std::fabs(n) > 127.0 + 1e-9) return TC_ERR_INVALID_ARG;
        }
    } else {
        for (size_t i = 0; i < (size_t)d->c * d->c; ++i)
            if (round_to_dtype(d->basis[i], d->basis_dtype) != d->basis[i]) return TC_ERR_INVALID_ARG;
    }
    DeviceGuard guard(ctx->device);
    tc_model *m = new (std::nothrow) tc_model();
    if (!m) return TC_ERR_CUDA;
    m->c = d->c; m->k = d->k; m->bits = d->bits; m->basis_dtype = d->basis_dtype;
    m->lo = d->lo; m->step = d->step; m->device = ctx->device;
    m->basis_scale = d->basis_dtype == TC_INT8 ? d->basis_scale : 1.0;
    m->basis.assign(d->basis, d->basis + (size_t)d->c * d->c);
    m->mean.assign(d->mean, d->mean + d->c);
    if (d->eig) m->eig.assign(d->eig, d->eig + d->c); else m->eig.assign(d->c, 0.0);
    tc_status st = finish_model(m);
    if (st != TC_OK) { tc_model_free(m); return st; }
    *out = m;
    return TC_OK;
}

tc_status tc_model_export(const tc_model *m, tc_model_desc *d)
{
    if (!m || !d) return TC_ERR_INVALID_ARG;
    d->c = m->c; d->k = m->k; d->bits = m->bits; d->basis_dtype = m->basis_dtype;
    d->lo = m->lo; d->step = m->step; d->basis_scale = m->basis_scale;
    if (d->basis) {
        const std::vector<double> *b = host_basis(m);
        if (!b) return TC_ERR_CUDA;
        std::copy(b->begin(), b->end(), d->basis);
    }
    if (d->mean) std::copy(m->mean.begin(), m->mean.end(), d->mean);
    if (d->eig) std::copy(m->eig.begin(), m->eig.end(), d->eig);
    return TC_OK;
}

void tc_model_free(tc_model *m)
{
    if (!m) return;
    DeviceGuard guard(m->device);
    cudaFree(m->d_basis64); cudaFree(m->d_mean64); cudaFree(m->d_basis_bf16);
    cudaFree(m->d_basis_t_bf16); cudaFree(m->d_enc_bias); cudaFree(m->d_dec_bias); cudaFree(m->d_tmu32);
    delete m;
}

static tc_status finish_fit(tc_ctx *ctx, const tc_tensor *range_maps, const tc_fit_params *params, int k,
                            const double *d_mean, const double *d_cov, tc_model **out, cudaStream_t s);

static bool valid_fit_params(const tc_fit_params *params)
{
    return (params->basis_dtype == TC_F32 || params->basis_dtype == TC_BF16 || params->basis_dtype == TC_INT8) &&
           (params->eigensolver == TC_EIG_DEVICE || params->eigensolver == TC_EIG_HOST);
}

tc_status tc_fit_pca(tc_ctx *ctx, const tc_tensor *calib, const tc_fit_params *params, tc_model **out, void *cuda_stream)
{
    if (!ctx || !out || !params || !valid_tensor(calib)) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    const int c = calib->c, hw = calib->h * calib->w, n = calib->n;
    const long long m_samples = (long long)n * hw;
    if (m_samples < 2) return TC_ERR_INVALID_ARG;
    if (params->bits < 1 || params->bits > 8 || c > TC_MAX_C) return TC_ERR_UNSUPPORTED;
    const int k = params->k ? params->k : c;
    if (k < 1 || k > c) return TC_ERR_INVALID_ARG;
    if (!valid_fit_params(params)) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;

    const size_t n_doubles = (size_t)c + (size_t)c * c;
    double *d_buf = nullptr;
    TC_CUDA(cudaMalloc((void **)&d_buf, n_doubles * sizeof(double)));
    double *d_mean = d_buf, *d_cov = d_buf + c;
    struct Free { double *p; ~Free() { cudaFree(p); } } freer{d_buf};
    TC_CUDA(cudaMemsetAsync(d_buf, 0, n_doubles * sizeof(double), s));

    tc_status st = tc_launch_channel_sums(calib->data, calib->dtype, n, c, hw, d_mean, s);
    if (st != TC_OK) return st;
    std::vector<double> mean(c);
    TC_CUDA(cudaMemcpyAsync(mean.data(), d_mean, sizeof(double) * c, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaStreamSynchronize(s));
    for (double &v : mean) v /= (double)m_samples;
    TC_CUDA(cudaMemcpyAsync(d_mean, mean.data(), sizeof(double) * c, cudaMemcpyHostToDevice, s));
    st = tc_launch_covariance(calib->data, calib->dtype, n, c, hw, d_mean, d_cov, s);
    if (st != TC_OK) return st;
    // centred sums in the upper triangle -> covariance, full symmetric, still on the device
    if ((st = tc_launch_scale_mirror(d_cov, c, (double)(m_samples - 1), s)) != TC_OK) return st;
    return finish_fit(ctx, calib, params, k, d_mean, d_cov, out, s);
}

// Second half of a fit, from the mean and the (symmetric, normalised) covariance on the device:
// eigendecomposition (on the device; on the host if the caller asks for that solver), rounding
// of the basis, range of coefficient 0 over `range_maps`, the model's constants.  Only vectors of
// C numbers cross to the host, unless the host solver was asked for.
static tc_status finish_fit(tc_ctx *ctx, const tc_tensor *range_maps, const tc_fit_params *params, int k,
                            const double *d_mean, const double *d_cov, tc_model **out, cudaStream_t s)
{
    const int c = range_maps->c, hw = range_maps->h * range_maps->w, n = range_maps->n;
    const long long m_samples = (long long)n * hw;
    const int range_blocks = tc_range0_max_blocks(m_samples);
    const size_t cc = (size_t)c * c;
    // small: eigenvalues [c], scale [1], min / max per block [2 * range_blocks]
    double *d_small = nullptr, *d_basis = nullptr, *d_mean_copy = nullptr;
    void *d_work = nullptr;
    struct Free {
        double **a, **b, **m; void **w;
        ~Free() { cudaFree(*a); cudaFree(*b); cudaFree(*m); cudaFree(*w); }
    } freer{&d_small, &d_basis, &d_mean_copy, &d_work};
    TC_CUDA(cudaMalloc((void **)&d_small, ((size_t)c + 1 + 2 * (size_t)range_blocks) * sizeof(double)));
    TC_CUDA(cudaMalloc((void **)&d_basis, cc * sizeof(double)));
    TC_CUDA(cudaMalloc((void **)&d_mean_copy, (size_t)c * sizeof(double)));
    double *d_eig = d_small, *d_scale = d_small + c, *d_minmax = d_scale + 1;
    TC_CUDA(cudaMemcpyAsync(d_mean_copy, d_mean, sizeof(double) * c, cudaMemcpyDeviceToDevice, s));
    tc_status st;
    if (params->eigensolver == TC_EIG_HOST) {
        std::vector<double> cov(cc), eig(c), basis(cc);
        TC_CUDA(cudaMemcpyAsync(cov.data(), d_cov, sizeof(double) * cc, cudaMemcpyDeviceToHost, s));
        TC_CUDA(cudaStreamSynchronize(s));
        if (tc_eigh_host(cov.data(), c, eig.data(), basis.data()) != 0) return TC_ERR_NOT_CONVERGED;
        TC_CUDA(cudaMemcpyAsync(d_basis, basis.data(), sizeof(double) * cc, cudaMemcpyHostToDevice, s));
        TC_CUDA(cudaMemcpyAsync(d_eig, eig.data(), sizeof(double) * c, cudaMemcpyHostToDevice, s));
        TC_CUDA(cudaStreamSynchronize(s));
    } else {
        TC_CUDA(cudaMalloc(&d_work, tc_eigh_device_workspace_bytes(c)));
        if ((st = tc_eigh_device(d_cov, c, d_eig, d_basis, d_work, nullptr, s)) != TC_OK) return st;
    }
    if ((st = tc_launch_round_basis(d_basis, c, params->basis_dtype, d_scale, s)) != TC_OK) return st;

    int blocks = 0;
    st = tc_launch_range0(range_maps->data, range_maps->dtype, n, c, hw, d_mean_copy, d_basis, d_minmax, &blocks, s);
    if (st != TC_OK) return st;
    std::vector<double> small((size_t)c + 1 + 2 * (size_t)blocks), mean(c);
    TC_CUDA(cudaMemcpyAsync(small.data(), d_small, sizeof(double) * small.size(), cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(mean.data(), d_mean_copy, sizeof(double) * c, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaStreamSynchronize(s));
    const double *mm = small.data() + c + 1;
    double lo = INFINITY, hi = -INFINITY;
    for (int i = 0; i < blocks; ++i) { lo = std::min(lo, mm[2 * i]); hi = std::max(hi, mm[2 * i + 1]); }
    if (!(hi > lo)) return TC_ERR_INVALID_ARG;    // constant calibration data: no range to quantise

    tc_model *m = new (std::nothrow) tc_model();
    if (!m) return TC_ERR_CUDA;
    m->c = c; m->k = k; m->bits = params->bits; m->basis_dtype = params->basis_dtype; m->device = ctx->device;
    m->step = (hi - lo) / (double)((1 << params->bits) - 1);
    // zero_level: shift the grid so that y = 0 is a level (at most half a step; ties to even)
    m->lo = params->zero_level ? -m->step * std::nearbyint(-lo / m->step) : lo;
    m->basis_scale = params->basis_dtype == TC_INT8 ? small[c] : 1.0;
    m->mean = mean;
    m->eig.assign(small.begin(), small.begin() + c);
    m->d_basis64 = d_basis; d_basis = nullptr;         // the model owns them from here
    m->d_mean64 = d_mean_copy; d_mean_copy = nullptr;
    if (params->basis_dtype == TC_INT8 && !(m->basis_scale > 0.0)) { tc_model_free(m); return TC_ERR_INVALID_ARG; }
    st = finish_model(m);
    if (st != TC_OK) { tc_model_free(m); return st; }
    *out = m;
    return TC_OK;
}

// ---- online fit: running sums ---------------------------------------------------------------

struct tc_fit_state {
    int c = 0, device = 0;
    long long count = 0;
    double *d_sum = nullptr;      // [c]     sum of the pixel vectors
    double *d_outer = nullptr;    // [c][c]  sum of their outer products (upper triangle)
    double *d_zero = nullptr;     // [c]     zeros: the "mean" that makes the covariance kernel add raw products
};

tc_status tc_fit_state_create(tc_ctx *ctx, int32_t c, tc_fit_state **out)
{
    if (!ctx || !out || c < 1) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    if (c > TC_MAX_C) return TC_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    double *buf = nullptr;
    const size_t n = 2 * (size_t)c + (size_t)c * c;
    TC_CUDA(cudaMalloc((void **)&buf, n * sizeof(double)));
    if (cudaMemset(buf, 0, n * sizeof(double)) != cudaSuccess) { cudaFree(buf); return TC_ERR_CUDA; }
    tc_fit_state *st = new tc_fit_state;
    st->c = c; st->device = ctx->device;
    st->d_sum = buf; st->d_zero = buf + c; st->d_outer = buf + 2 * (size_t)c;
    *out = st;
    return TC_OK;
}

void tc_fit_state_free(tc_fit_state *st)
{
    if (!st) return;
    DeviceGuard guard(st->device);
    cudaFree(st->d_sum);          // one allocation holds all three arrays
    delete st;
}

tc_status tc_fit_state_update(tc_ctx *ctx, tc_fit_state *st, const tc_tensor *maps, void *cuda_stream)
{
    if (!ctx || !st || !valid_tensor(maps) || maps->c != st->c || ctx->device != st->device) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int hw = maps->h * maps->w;
    if ((long long)maps->n * hw == 0) return TC_OK;
    tc_status rc = tc_launch_channel_sums(maps->data, maps->dtype, maps->n, st->c, hw, st->d_sum, s);
    if (rc != TC_OK) return rc;
    rc = tc_launch_covariance(maps->data, maps->dtype, maps->n, st->c, hw, st->d_zero, st->d_outer, s);
    if (rc != TC_OK) return rc;
    st->count += (long long)maps->n * hw;
    return TC_OK;
}

tc_status tc_fit_state_export(tc_ctx *ctx, const tc_fit_state *st, int64_t *count, double *sum, double *outer,
                              void *cuda_stream)
{
    if (!ctx || !st || !count || !sum || !outer) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(st->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int c = st->c;
    TC_CUDA(cudaMemcpyAsync(sum, st->d_sum, sizeof(double) * c, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(outer, st->d_outer, sizeof(double) * (size_t)c * c, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaStreamSynchronize(s));
    for (int a = 0; a < c; ++a)                       // the device holds the upper triangle
        for (int b = a + 1; b < c; ++b) outer[(size_t)b * c + a] = outer[(size_t)a * c + b];
    *count = st->count;
    return TC_OK;
}

tc_status tc_fit_state_import(tc_ctx *ctx, tc_fit_state *st, int64_t count, const double *sum, const double *outer,
                              void *cuda_stream)
{
    if (!ctx || !st || count < 0 || !sum || !outer) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(st->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    TC_CUDA(cudaMemcpyAsync(st->d_sum, sum, sizeof(double) * st->c, cudaMemcpyHostToDevice, s));
    TC_CUDA(cudaMemcpyAsync(st->d_outer, outer, sizeof(double) * (size_t)st->c * st->c, cudaMemcpyHostToDevice, s));
    TC_CUDA(cudaStreamSynchronize(s));
    st->count = count;
    return TC_OK;
}

tc_status tc_fit_state_finish(tc_ctx *ctx, const tc_fit_state *st, const tc_tensor *range_maps,
                              const tc_fit_params *params, tc_model **out, void *cuda_stream)
{
    if (!ctx || !st || !out || !params || !valid_tensor(range_maps) || range_maps->c != st->c) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    const int c = st->c;
    if (st->count < 2 || (long long)range_maps->n * range_maps->h * range_maps->w < 1) return TC_ERR_INVALID_ARG;
    if (params->bits < 1 || params->bits > 8) return TC_ERR_UNSUPPORTED;
    const int k = params->k ? params->k : c;
    if (k < 1 || k > c) return TC_ERR_INVALID_ARG;
    if (!valid_fit_params(params)) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // mean = s / M, covariance = (S - s s^T / M) / (M - 1), on the device
    double *d_buf = nullptr;
    TC_CUDA(cudaMalloc((void **)&d_buf, ((size_t)c + (size_t)c * c) * sizeof(double)));
    struct Free { double *p; ~Free() { cudaFree(p); } } freer{d_buf};
    double *d_mean = d_buf, *d_cov = d_buf + c;
    tc_status rc = tc_launch_moments_to_cov(st->d_sum, st->d_outer, st->count, c, d_mean, d_cov, s);
    if (rc != TC_OK) return rc;
    return finish_fit(ctx, range_maps, params, k, d_mean, d_cov, out, s);
}

// ---- folding into the neighbouring convolutions (host arithmetic, fp64) --------------------------

tc_status tc_fold_forward(const tc_model *m, const double *w, const double *bias, const double *scale,
                          const double *shift, int64_t fan, double *w_folded, double *bias_folded)
{
    if (!m || !w || !w_folded || !bias_folded || fan < 1) return TC_ERR_INVALID_ARG;
    const int c = m->c, k = m->k;
    const std::vector<double> *basis = host_basis(m);
    if (!basis) return TC_ERR_CUDA;
    for (int j = 0; j < k; ++j) {
        const double *row = basis->data() + (size_t)j * c;
        for (int64_t f = 0; f < fan; ++f) {
            double acc = 0.0;
            for (int a = 0; a < c; ++a) acc += row[a] * ((scale ? scale[a] : 1.0) * w[(size_t)a * fan + f]);
            w_folded[(size_t)j * fan + f] = acc;
        }
        double b = 0.0;
        for (int a = 0; a < c; ++a)
            b += row[a] * ((scale ? scale[a] : 1.0) * (bias ? bias[a] : 0.0) + (shift ? shift[a] : 0.0) - m->mean[a]);
        bias_folded[j] = b;
    }
    return TC_OK;
}

tc_status tc_fold_inverse(const tc_model *m, const double *w_next, const double *bias_next, int32_t c_out,
                          int32_t taps, double *w_folded, double *bias_folded)
{
    if (!m || !w_next || !w_folded || !bias_folded || c_out < 1 || taps < 1) return TC_ERR_INVALID_ARG;
    const int c = m->c, k = m->k;
    const std::vector<double> *basis = host_basis(m);
    if (!basis) return TC_ERR_CUDA;
    for (int o = 0; o < c_out; ++o) {
        for (int j = 0; j < k; ++j) {
            const double *row = basis->data() + (size_t)j * c;
            for (int t = 0; t < taps; ++t) {
                double acc = 0.0;
                for (int a = 0; a < c; ++a) acc += w_next[((size_t)o * c + a) * taps + t] * row[a];
                w_folded[((size_t)o * k + j) * taps + t] = acc;
            }
        }
        double b = bias_next ? bias_next[o] : 0.0;
        for (int a = 0; a < c; ++a)
            for (int t = 0; t < taps; ++t) b += w_next[((size_t)o * c + a) * taps + t] * m->mean[a];
        bias_folded[o] = b;
    }
    return TC_OK;
}

// ---- codebook ---------------------------------------------------------------------------

tc_status tc_host_huffman_lengths(const uint64_t *counts, int32_t nsym, int32_t max_length, uint8_t *lengths)
{
    return tc_huffman_lengths_host(counts, nsym, max_length, lengths) == 0 ? TC_OK : TC_ERR_INVALID_ARG;
}

tc_status tc_device_eigh(tc_ctx *ctx, const double *a, int32_t n, double *evals, double *evecs, int32_t *sweeps, void *cuda_stream)
{
    if (!ctx || !a || !evals || !evecs || n < 1 || n > TC_MAX_C) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    void *work = nullptr;
    TC_CUDA(cudaMalloc(&work, tc_eigh_device_workspace_bytes(n)));
    int n_sweeps = 0;
    const tc_status st = tc_eigh_device(a, n, evals, evecs, work, &n_sweeps, s);
    cudaStreamSynchronize(s);
    cudaFree(work);
    if (sweeps) *sweeps = n_sweeps;
    return st;
}

tc_status tc_host_eigh(double *a, int32_t n, double *evals, double *evecs)
{
    if (!a || !evals || !evecs || n < 1) return TC_ERR_INVALID_ARG;
    return tc_eigh_host(a, n, evals, evecs) == 0 ? TC_OK : TC_ERR_NOT_CONVERGED;
}

tc_status tc_codebook_import(tc_ctx *ctx, int32_t bits, int32_t groups, const uint8_t *lengths, tc_codebook **out)
{
    if (!ctx || !lengths || !out || groups < 1) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    if (bits < 1 || bits > 8 || groups > TC_MAX_C) return TC_ERR_UNSUPPORTED;
    const int nsym = 1 << bits;
    for (int g = 0; g < groups; ++g) {
        const uint8_t *len = lengths + (size_t)g * nsym;
        for (int s = 0; s < nsym; ++s)
            if (len[s] > TC_MAX_CODE_LEN) return TC_ERR_UNSUPPORTED;
        if (!kraft_complete(len, nsym, TC_MAX_CODE_LEN)) return TC_ERR_INVALID_ARG;
    }
    DeviceGuard guard(ctx->device);
    tc_codebook *cb = new (std::nothrow) tc_codebook();
    if (!cb) return TC_ERR_CUDA;
    cb->bits = bits; cb->groups = groups; cb->device = ctx->device;
    cb->lengths.assign(lengths, lengths + (size_t)groups * nsym);
    tc_status st = finish_codebook(cb);
    if (st != TC_OK) { tc_codebook_free(cb); return st; }
    *out = cb;
    return TC_OK;
}

tc_status tc_build_codebook(tc_ctx *ctx, const tc_model *model, const uint64_t *hist, int hist_on_device,
                            const tc_codebook_params *params, tc_codebook **out)
{
    if (!ctx || !model || !hist || !params || !out) return TC_ERR_INVALID_ARG;
    *out = nullptr;
    const int groups = params->groups;
    if (groups != 1 && groups != model->k) return TC_ERR_INVALID_ARG;
    const int lmax = params->max_length ? params->max_length : TC_MAX_CODE_LEN;
    if (lmax < model->bits) return TC_ERR_INVALID_ARG;
    if (lmax > TC_MAX_CODE_LEN) return TC_ERR_UNSUPPORTED;
    const int nsym = 1 << model->bits;
    std::vector<uint64_t> h((size_t)groups * nsym);
    if (hist_on_device) {
        DeviceGuard guard(ctx->device);
        TC_CUDA(cudaMemcpy(h.data(), hist, h.size() * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    } else {
        std::copy(hist, hist + h.size(), h.begin());
    }
    std::vector<uint8_t> lengths((size_t)groups * nsym);
    for (int g = 0; g < groups; ++g)
        if (tc_huffman_lengths_host(h.data() + (size_t)g * nsym, nsym, lmax, lengths.data() + (size_t)g * nsym) != 0)
            return TC_ERR_INVALID_ARG;
    return tc_codebook_import(ctx, model->bits, groups, lengths.data(), out);
}

tc_status tc_codebook_export(const tc_codebook *cb, int32_t *bits, int32_t *groups, uint8_t *lengths)
{
    if (!cb) return TC_ERR_INVALID_ARG;
    if (bits) *bits = cb->bits;
    if (groups) *groups = cb->groups;
    if (lengths) std::copy(cb->lengths.begin(), cb->lengths.end(), lengths);
    return TC_OK;
}

void tc_codebook_free(tc_codebook *cb)
{
    if (!cb) return;
    DeviceGuard guard(cb->device);
    cudaFree(cb->d_enc);
    cudaFree(cb->d_lut);
    cudaFree(cb->d_lut32);
    delete cb;
}

// ---- encode / decode ----------------------------------------------------------------------

}  // extern "C"

// Argument block and kernel choice shared by tc_encode and tc_encode_noalloc.  `scratch` is
// kEncodeScratchHeader bytes (ticket counter) followed by one 64-bit look-back word per tile;
// it is cleared on the stream here, whoever owns it.
tc_status tc_encode_with_scratch(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const tc_tensor *x, int chunk_pixels,
                                 int splits, void *stream_out, size_t capacity, uint16_t *chunk_len, uint64_t *tile_off,
                                 const tc_debug_out *debug, void *scratch, uint8_t *sym_scratch, cudaStream_t s,
                                 unsigned long long *hist, unsigned long long *clamped, bool scratch_is_zero)
{
    const long long pixels = (long long)x->n * x->h * x->w;
    const long long n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
    if (!scratch_is_zero)
        TC_CUDA(cudaMemsetAsync(scratch, 0, kEncodeScratchHeader + (size_t)n_tiles * sizeof(unsigned long long), s));

    EncodeArgs a{};
    a.x = x->data; a.n = x->n; a.c = x->c; a.hw = x->h * x->w; a.k = m->k; a.bits = m->bits; a.groups = cb->groups;
    a.pixels = pixels; a.n_tiles = n_tiles; a.chunk_pixels = chunk_pixels; a.splits = splits;
    a.basis64 = m->d_basis64; a.mean64 = m->d_mean64; a.lo = m->lo; a.step = m->step;
    a.enc = cb->d_enc; a.stream = (uint32_t *)stream_out;
    a.capacity_bits = (unsigned long long)(capacity & ~(size_t)15) * 8ull;
    a.chunk_len = chunk_len; a.tile_off = (unsigned long long *)tile_off; a.basis_scale = m->basis_scale;
    a.dbg_coef = debug ? debug->coefficients : nullptr;
    a.dbg_sym = debug ? debug->symbols : nullptr;
    a.ticket = (unsigned int *)scratch;
    a.tile_state = (unsigned long long *)((char *)scratch + kEncodeScratchHeader);
    a.status = ctx->d_status; a.clamped = clamped; a.emit = 1;
    a.basis_bf16 = m->d_basis_bf16; a.enc_bias = m->d_enc_bias; a.tmu32 = m->d_tmu32;
    a.basis_map = m->has_basis_map ? &m->basis_map : nullptr;
    a.hist = hist; a.hist_modal = m->center;
    if (hist && !((ctx->force_exact == 0 || ctx->force_exact == 3) && x->dtype == TC_BF16 && tc_encode_tc_supported(ctx, a)))
        return TC_ERR_UNSUPPORTED;                      // only the resident-basis tensor-core encoder counts symbols
    if ((ctx->force_exact == 0 || ctx->force_exact == 3) && x->dtype == TC_BF16 && tc_encode_tc_supported(ctx, a)) {
        ctx->last_encode_path = 1;
        return tc_launch_encode_tc(ctx, a, s);
    }
    if (ctx->force_exact != 1 && x->dtype == TC_BF16 && tc_encode_wide_supported(ctx, a)) {   // wide layers, unaligned rows
        ctx->last_encode_path = 3;
        if (sym_scratch && n_tiles < ctx->sm_count && ((uintptr_t)sym_scratch & 15u) == 0 && tc_pack_symbols_parts(a) > 0) {
            // fewer tiles than SMs: the projection is dealt over the SMs by blocks of coefficients and leaves
            // the symbols in the arena, the entropy coder follows as a kernel of its own (same stream)
            a.sym_park = sym_scratch;
            const tc_status st = tc_launch_encode_wide(ctx, a, s);
            if (st != TC_OK) return st;
            a.sym_park = nullptr;
            return tc_launch_pack_symbols(a, sym_scratch, s);
        }
        return tc_launch_encode_wide(ctx, a, s);
    }
    if (ctx->force_exact != 1 && x->dtype == TC_BF16 && x->c % 2 == 0) {      // shapes the tensor-core kernel does not take
        ctx->last_encode_path = 2;
        return tc_launch_encode_simt_fp32(ctx, a, s);
    }
    ctx->last_encode_path = 0;
    if (sym_scratch && n_tiles < (long long)kExactParallelTilesPerSm * ctx->sm_count) {
        // few pixels: projection and quantiser with one thread per (pixel, coefficient), then the
        // entropy coder of the per-pixel kernel on those symbols -- same arithmetic, same results
        tc_status st = tc_launch_project_quantise(a, x->dtype, sym_scratch, s);
        if (st != TC_OK) return st;
        if (tc_pack_symbols_parts(a) > 0 && ((uintptr_t)sym_scratch & 15u) == 0)
            return tc_launch_pack_symbols(a, sym_scratch, s);      // several threads per pixel code the symbols
        a.sym_in = sym_scratch;
    }
    return tc_launch_encode_simt(ctx, a, x->dtype, s);
}

extern "C" {


static tc_status check_codec_args(const tc_model *m, const tc_codebook *cb, const tc_tensor *x)
{
    if (!m || !cb || !valid_tensor(x)) return TC_ERR_INVALID_ARG;
    if (x->c != m->c || cb->bits != m->bits) return TC_ERR_INVALID_ARG;
    if (cb->groups != 1 && cb->groups != m->k) return TC_ERR_INVALID_ARG;
    if (x->dtype != m->basis_dtype && m->basis_dtype != TC_INT8) return TC_ERR_UNSUPPORTED;   // an 8-bit basis serves both tensor types
    if ((long long)x->n * x->h * x->w > (1ll << 40)) return TC_ERR_UNSUPPORTED;
    return TC_OK;
}

tc_status tc_encode_bound(const tc_model *m, const tc_codebook *cb, const tc_tensor *x, const tc_encode_params *params,
                          tc_stream_layout *out)
{
    if (!out) return TC_ERR_INVALID_ARG;
    tc_status st = check_codec_args(m, cb, x);
    if (st != TC_OK) return st;
    ChunkShape cs;
    if (!resolve_chunks(params, m->k, cb->max_len, &cs)) return TC_ERR_INVALID_ARG;
    const long long pixels = (long long)x->n * x->h * x->w;
    out->n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
    out->n_chunks = cs.chunks(pixels);
    const unsigned long long tile_bits = (unsigned long long)TC_TILE_PIXELS * m->k * cb->max_len;   // multiple of 128
    out->stream_bytes = (size_t)((unsigned long long)out->n_tiles * tile_bits / 8);
    out->chunk_len_bytes = (size_t)out->n_chunks * 2;
    out->tile_off_bytes = (size_t)(out->n_tiles + 1) * 8;
    out->chunk_pixels = cs.cp;
    out->pixel_splits = cs.splits;
    return TC_OK;
}

tc_status tc_encode(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const tc_tensor *x,
                    const tc_encode_params *params, void *stream_out, size_t capacity, uint16_t *chunk_len,
                    uint64_t *tile_off, const tc_debug_out *debug, void *cuda_stream)
{
    if (!ctx || !tile_off) return TC_ERR_INVALID_ARG;
    tc_status st = check_codec_args(m, cb, x);
    if (st != TC_OK) return st;
    ChunkShape cs;
    if (!resolve_chunks(params, m->k, cb->max_len, &cs)) return TC_ERR_INVALID_ARG;
    const long long pixels = (long long)x->n * x->h * x->w;
    if (pixels > 0 && (!stream_out || !chunk_len)) return TC_ERR_INVALID_ARG;
    if (((uintptr_t)stream_out & 15u) != 0 || ((uintptr_t)chunk_len & 3u) != 0) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const long long n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
    if (n_tiles == 0) {
        TC_CUDA(cudaMemsetAsync(tile_off, 0, sizeof(uint64_t), s));
        return TC_OK;
    }
    const size_t lookback = (kEncodeScratchHeader + (size_t)n_tiles * sizeof(unsigned long long) + 255) & ~(size_t)255;
    // small tensors on the exact kernels also park their symbols in the arena (P * K bytes)
    const bool parallel_exact = n_tiles < (long long)kExactParallelTilesPerSm * ctx->sm_count;
    const size_t scratch = lookback + (parallel_exact ? (size_t)pixels * m->k : 0);
    if ((st = ensure_scratch(ctx, scratch)) != TC_OK) return st;
    return tc_encode_with_scratch(ctx, m, cb, x, cs.cp, cs.splits, stream_out, capacity, chunk_len, tile_off, debug,
                                  ctx->scratch, parallel_exact ? (uint8_t *)ctx->scratch + lookback : nullptr, s);
}

// Bytes of symbol scratch a decode of `x_hat` may need: small tensors on the exact kernels park
// their symbols there (whether that route is taken is decided at launch).
static size_t decode_scratch_bytes(const tc_ctx *ctx, const tc_model *m, const tc_tensor *x_hat)
{
    const long long pixels = (long long)x_hat->n * x_hat->h * x_hat->w;
    const long long n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
    return n_tiles < (long long)kExactParallelTilesPerSm * ctx->sm_count ? (((size_t)pixels * m->k + 255) & ~(size_t)255) : 0;
}

// tc_decode with the symbol scratch named by the caller (decode_scratch_bytes of it, or nullptr)
static tc_status decode_with_scratch(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const void *stream, size_t stream_bytes,
                                     const uint16_t *chunk_len, const uint64_t *tile_off, const tc_encode_params *params,
                                     const tc_tensor *x_hat, uint8_t *sym_scratch, void *cuda_stream)
{
    if (!ctx) return TC_ERR_INVALID_ARG;
    tc_status st = check_codec_args(m, cb, x_hat);
    if (st != TC_OK) return st;
    ChunkShape cs;
    if (!resolve_chunks(params, m->k, cb->max_len, &cs)) return TC_ERR_INVALID_ARG;
    const long long pixels = (long long)x_hat->n * x_hat->h * x_hat->w;
    if (pixels == 0) return TC_OK;
    if (!stream || !chunk_len || !tile_off || ((uintptr_t)stream & 15u) != 0 || ((uintptr_t)chunk_len & 3u) != 0)
        return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    DecodeArgs a{};
    a.stream = (const uint32_t *)stream; a.stream_bits = (unsigned long long)(stream_bytes & ~(size_t)3) * 8ull;
    a.chunk_len = chunk_len; a.splits = cs.splits; a.tile_off = (const unsigned long long *)tile_off; a.symbols = nullptr;
    a.n = x_hat->n; a.c = x_hat->c; a.hw = x_hat->h * x_hat->w; a.k = m->k; a.bits = m->bits; a.groups = cb->groups;
    a.pixels = pixels; a.n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS; a.n_chunks = cs.chunks(pixels);
    a.chunk_pixels = cs.cp; a.lut_bits = cb->lut_bits; a.lut = cb->d_lut;
    a.basis64 = m->d_basis64; a.mean64 = m->d_mean64; a.lo = m->lo; a.step = m->step; a.basis_scale = m->basis_scale;
    a.xhat = x_hat->data; a.status = ctx->d_status;
    a.lut32 = cb->d_lut32; a.basis_t_bf16 = m->d_basis_t_bf16; a.dec_bias = m->d_dec_bias; a.center = m->center;
    a.relu = (params && params->relu) ? 1 : 0;
    a.basis_t_map = m->has_basis_t_map ? &m->basis_t_map : nullptr;
    a.modal = cb->modal;
    a.mean_tile_bytes = (params && params->mean_tile_bytes > 0) ? params->mean_tile_bytes : 0;
    // Coefficient j has standard deviation sqrt(eig[j]) on the calibration data; where that exceeds
    // about 0.45 steps more than a quarter of its symbols differ from the zero level and skipping
    // runs of the zero level no longer pays: those leading coefficients are decoded symbol by symbol.
    a.dense_head = 0;
    while (a.dense_head < m->k && a.dense_head < (int)m->eig.size() && std::sqrt(std::max(0.0, m->eig[a.dense_head])) > 0.45 * m->step)
        ++a.dense_head;
    // per-layer code table, up to 256 channels: the run-skipping decoder (it also takes dense tiles)
    if (ctx->force_exact == 0 && x_hat->dtype == TC_BF16 && tc_decode_runs_supported(ctx, a)) {
        ctx->last_decode_path = 1;
        return tc_launch_decode_runs(ctx, a, (cudaStream_t)cuda_stream);
    }
    bool resident = (ctx->force_exact == 0 || ctx->force_exact == 3) && x_hat->dtype == TC_BF16 && tc_decode_tc_supported(ctx, a);
    // High-rate streams (params->mean_tile_bytes): a tile's segment that no longer fits the shared-memory
    // staging of the resident-basis decoder but still fits that of the streaming decoder is better
    // served by the latter (the former would read the stream from global memory word by word).
    const size_t hint = (params && params->mean_tile_bytes > 0) ? (size_t)params->mean_tile_bytes : 0;
    if (resident && hint > tc_decode_tc_staging_bytes(ctx, a) && tc_decode_wide_supported(ctx, a) &&
        hint <= tc_decode_wide_staging_bytes(ctx, a))
        resident = false;
    if (resident) {
        ctx->last_decode_path = 1;
        return tc_launch_decode_tc(ctx, a, (cudaStream_t)cuda_stream);
    }
    if (ctx->force_exact != 1 && x_hat->dtype == TC_BF16 && tc_decode_wide_supported(ctx, a)) {   // wide layers
        ctx->last_decode_path = 3;
        return tc_launch_decode_wide(ctx, a, (cudaStream_t)cuda_stream);
    }
    if (ctx->force_exact != 1 && x_hat->dtype == TC_BF16 && x_hat->c % 2 == 0) {  // shapes the tensor-core kernel does not take
        ctx->last_decode_path = 2;
        return tc_launch_decode_simt_fp32(ctx, a, (cudaStream_t)cuda_stream);
    }
    ctx->last_decode_path = 0;
    if (sym_scratch && a.n_tiles < (long long)kExactParallelTilesPerSm * ctx->sm_count) {
        // few pixels: the per-pixel kernel only decodes the symbols (into the context's arena), the
        // inverse transform runs with one thread per (pixel, channel) -- same arithmetic, same results
        if ((st = tc_launch_unpack_symbols(a, sym_scratch, (cudaStream_t)cuda_stream)) != TC_OK) return st;
        return tc_launch_reconstruct(a, x_hat->dtype, sym_scratch, (cudaStream_t)cuda_stream);
    }
    return tc_launch_decode_simt(ctx, a, x_hat->dtype, (cudaStream_t)cuda_stream);
}

tc_status tc_decode(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const void *stream, size_t stream_bytes,
                    const uint16_t *chunk_len, const uint64_t *tile_off, const tc_encode_params *params,
                    const tc_tensor *x_hat, void *cuda_stream)
{
    if (!ctx || !m || !valid_tensor(x_hat)) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    const size_t scratch = decode_scratch_bytes(ctx, m, x_hat);
    if (scratch) {
        const tc_status st = ensure_scratch(ctx, scratch);
        if (st != TC_OK) return st;
    }
    return decode_with_scratch(ctx, m, cb, stream, stream_bytes, chunk_len, tile_off, params, x_hat,
                               scratch ? (uint8_t *)ctx->scratch : nullptr, cuda_stream);
}

// ---- several tensors per call --------------------------------------------------------------------

static tc_status ensure_many_streams(tc_ctx *ctx)
{
    if (ctx->many_fork) return TC_OK;
    for (int i = 0; i < 4; ++i) {
        TC_CUDA(cudaStreamCreateWithFlags(&ctx->many_streams[i], cudaStreamNonBlocking));
        TC_CUDA(cudaEventCreateWithFlags(&ctx->many_join[i], cudaEventDisableTiming));
    }
    TC_CUDA(cudaEventCreateWithFlags(&ctx->many_fork, cudaEventDisableTiming));
    return TC_OK;
}

// Items in descending order of work: the large ones start first, each on its own stream.
static std::vector<int> by_descending_work(int n, const std::vector<double> &work)
{
    std::vector<int> order(n);
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return work[a] > work[b]; });
    return order;
}

tc_status tc_encode_many(tc_ctx *ctx, const tc_encode_item *items, int32_t n_items, void *cuda_stream)
{
    if (!ctx || n_items < 0 || (n_items > 0 && !items)) return TC_ERR_INVALID_ARG;
    if (n_items == 0) return TC_OK;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // every item is checked before anything is launched
    std::vector<ChunkShape> shape(n_items);
    std::vector<size_t> lookback_at(n_items), symbols_at(n_items, 0);
    std::vector<double> work(n_items);
    size_t lookback_total = 0, total = 0;
    for (int i = 0; i < n_items; ++i) {
        const tc_encode_item &it = items[i];
        if (!it.tile_off) return TC_ERR_INVALID_ARG;
        const tc_status st = check_codec_args(it.model, it.codebook, it.x);
        if (st != TC_OK) return st;
        if (!resolve_chunks(it.params, it.model->k, it.codebook->max_len, &shape[i])) return TC_ERR_INVALID_ARG;
        const long long pixels = (long long)it.x->n * it.x->h * it.x->w;
        if (pixels > 0 && (!it.stream_out || !it.chunk_len)) return TC_ERR_INVALID_ARG;
        if (((uintptr_t)it.stream_out & 15u) != 0 || ((uintptr_t)it.chunk_len & 3u) != 0) return TC_ERR_INVALID_ARG;
        const long long n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
        lookback_at[i] = lookback_total;
        lookback_total += (kEncodeScratchHeader + (size_t)n_tiles * sizeof(unsigned long long) + 255) & ~(size_t)255;
        work[i] = (double)pixels * it.x->c;
    }
    total = lookback_total;
    for (int i = 0; i < n_items; ++i) {
        const tc_encode_item &it = items[i];
        const long long pixels = (long long)it.x->n * it.x->h * it.x->w;
        const long long n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
        if (n_tiles > 0 && n_tiles < (long long)kExactParallelTilesPerSm * ctx->sm_count) {
            symbols_at[i] = total;
            total += ((size_t)pixels * it.model->k + 255) & ~(size_t)255;
        }
    }
    tc_status st = ensure_scratch(ctx, total);
    if (st != TC_OK) return st;
    if ((st = ensure_many_streams(ctx)) != TC_OK) return st;
    // one clear for the look-back state of all items, then the items fan out over the streams
    TC_CUDA(cudaMemsetAsync(ctx->scratch, 0, lookback_total, s));
    TC_CUDA(cudaEventRecord(ctx->many_fork, s));
    const int n_streams = std::min(4, (int)n_items);
    for (int j = 0; j < n_streams; ++j) TC_CUDA(cudaStreamWaitEvent(ctx->many_streams[j], ctx->many_fork, 0));
    const std::vector<int> order = by_descending_work(n_items, work);
    tc_status first_error = TC_OK;
    for (int r = 0; r < n_items; ++r) {
        const int i = order[r];
        const tc_encode_item &it = items[i];
        cudaStream_t ws = ctx->many_streams[r % n_streams];
        const long long pixels = (long long)it.x->n * it.x->h * it.x->w;
        if (pixels == 0) { if (cudaMemsetAsync(it.tile_off, 0, sizeof(uint64_t), ws) != cudaSuccess && first_error == TC_OK) first_error = TC_ERR_CUDA; continue; }
        st = tc_encode_with_scratch(ctx, it.model, it.codebook, it.x, shape[i].cp, shape[i].splits, it.stream_out, it.capacity,
                                    it.chunk_len, it.tile_off, nullptr, (char *)ctx->scratch + lookback_at[i],
                                    symbols_at[i] ? (uint8_t *)ctx->scratch + symbols_at[i] : nullptr, ws, nullptr, nullptr, true);
        if (st != TC_OK && first_error == TC_OK) first_error = st;
    }
    for (int j = 0; j < n_streams; ++j) {
        TC_CUDA(cudaEventRecord(ctx->many_join[j], ctx->many_streams[j]));
        TC_CUDA(cudaStreamWaitEvent(s, ctx->many_join[j], 0));
    }
    return first_error;
}

tc_status tc_decode_many(tc_ctx *ctx, const tc_decode_item *items, int32_t n_items, void *cuda_stream)
{
    if (!ctx || n_items < 0 || (n_items > 0 && !items)) return TC_ERR_INVALID_ARG;
    if (n_items == 0) return TC_OK;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    std::vector<size_t> symbols_at(n_items, 0), symbols_bytes(n_items, 0);
    std::vector<double> work(n_items);
    size_t total = 0;
    for (int i = 0; i < n_items; ++i) {
        const tc_decode_item &it = items[i];
        const tc_status st = check_codec_args(it.model, it.codebook, it.x_hat);
        if (st != TC_OK) return st;
        ChunkShape cs;
        if (!resolve_chunks(it.params, it.model->k, it.codebook->max_len, &cs)) return TC_ERR_INVALID_ARG;
        const long long pixels = (long long)it.x_hat->n * it.x_hat->h * it.x_hat->w;
        if (pixels > 0 && (!it.stream || !it.chunk_len || !it.tile_off || ((uintptr_t)it.stream & 15u) != 0 ||
                           ((uintptr_t)it.chunk_len & 3u) != 0))
            return TC_ERR_INVALID_ARG;
        symbols_bytes[i] = decode_scratch_bytes(ctx, it.model, it.x_hat);
        symbols_at[i] = total;
        total += symbols_bytes[i];
        work[i] = (double)pixels * it.x_hat->c;
    }
    tc_status st;
    if (total && (st = ensure_scratch(ctx, total)) != TC_OK) return st;
    if ((st = ensure_many_streams(ctx)) != TC_OK) return st;
    TC_CUDA(cudaEventRecord(ctx->many_fork, s));
    const int n_streams = std::min(4, (int)n_items);
    for (int j = 0; j < n_streams; ++j) TC_CUDA(cudaStreamWaitEvent(ctx->many_streams[j], ctx->many_fork, 0));
    const std::vector<int> order = by_descending_work(n_items, work);
    tc_status first_error = TC_OK;
    for (int r = 0; r < n_items; ++r) {
        const int i = order[r];
        const tc_decode_item &it = items[i];
        st = decode_with_scratch(ctx, it.model, it.codebook, it.stream, it.stream_bytes, it.chunk_len, it.tile_off, it.params,
                                 it.x_hat, symbols_bytes[i] ? (uint8_t *)ctx->scratch + symbols_at[i] : nullptr,
                                 ctx->many_streams[r % n_streams]);
        if (st != TC_OK && first_error == TC_OK) first_error = st;
    }
    for (int j = 0; j < n_streams; ++j) {
        TC_CUDA(cudaEventRecord(ctx->many_join[j], ctx->many_streams[j]));
        TC_CUDA(cudaStreamWaitEvent(s, ctx->many_join[j], 0));
    }
    return first_error;
}

tc_status tc_roundtrip_host(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const void *x_host, void *x_hat_host,
                            int32_t n, int32_t c, int32_t h, int32_t w, int32_t dtype, const tc_encode_params *params,
                            uint64_t *stream_bits, void *cuda_stream)
{
    if (!ctx || !x_host || !x_hat_host) return TC_ERR_INVALID_ARG;
    tc_tensor x{nullptr, n, c, h, w, dtype};
    x.data = (void *)x_host;                      // only for the shape checks of tc_encode_bound
    tc_stream_layout lay;
    tc_status st = tc_encode_bound(m, cb, &x, params, &lay);
    if (st != TC_OK) return st;
    if (lay.n_tiles == 0) { if (stream_bits) *stream_bits = 0; return TC_OK; }
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t elem = dtype == TC_F32 ? 4 : 2;
    const size_t image_bytes = (size_t)c * h * w * elem;
    // The batch is cut into chunks of whole tiles (so that the stream is the one a single call
    // would write) of about 24 MB, and two chunks are in flight: while one is encoded and decoded
    // on the caller's stream, the next one is copied in and the previous one is copied out on
    // two streams of the context -- the link to the host carries both directions at once.
    const int hw = h * w;
    int unit = 1;                                   // images per chunk must be a multiple of this
    while (((long long)unit * hw) % TC_TILE_PIXELS != 0) unit <<= 1;      // at most 128
    long long chunk_n = (long long)((24ull << 20) / image_bytes);
    chunk_n = std::max<long long>(chunk_n, ((long long)n + kMaxRoundtripChunks - 1) / kMaxRoundtripChunks);
    chunk_n = std::max<long long>(unit, (chunk_n + unit - 1) / unit * unit);
    if (chunk_n >= n) chunk_n = n;
    const int n_chunks = (int)(((long long)n + chunk_n - 1) / chunk_n);
    if (n_chunks > kMaxRoundtripChunks) return TC_ERR_UNSUPPORTED;
    if (!ctx->copy_in) {
        TC_CUDA(cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking));
        TC_CUDA(cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            TC_CUDA(cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming));
            TC_CUDA(cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming));
            TC_CUDA(cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming));
        }
        TC_CUDA(cudaMallocHost((void **)&ctx->chunk_bits, sizeof(unsigned long long) * kMaxRoundtripChunks));
    }
    tc_tensor xc{nullptr, (int32_t)chunk_n, c, h, w, dtype};
    xc.data = (void *)x_host;
    tc_stream_layout clay;
    if ((st = tc_encode_bound(m, cb, &xc, params, &clay)) != TC_OK) return st;
    const size_t chunk_bytes = (size_t)chunk_n * image_bytes;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t off_xhat = up(chunk_bytes), off_stream = off_xhat + up(chunk_bytes), off_chunk = off_stream + up(clay.stream_bytes),
                 off_tile = off_chunk + up(clay.chunk_len_bytes), slot_bytes = off_tile + up(clay.tile_off_bytes);
    const int n_slots = n_chunks > 1 ? 2 : 1;
    const size_t total = slot_bytes * n_slots;
    if (total > ctx->host_arena_bytes) {
        if (ctx->host_arena) { TC_CUDA(cudaDeviceSynchronize()); cudaFree(ctx->host_arena); ctx->host_arena = nullptr; ctx->host_arena_bytes = 0; }
        TC_CUDA(cudaMalloc(&ctx->host_arena, total));
        ctx->host_arena_bytes = total;
    }
    // the copy-in stream starts after whatever the caller queued before this call
    TC_CUDA(cudaEventRecord(ctx->ev_done[0], s));
    TC_CUDA(cudaStreamWaitEvent(ctx->copy_in, ctx->ev_done[0], 0));
    for (int i = 0; i < n_chunks; ++i) {
        const int slot = i % n_slots;
        char *base = (char *)ctx->host_arena + slot_bytes * slot;
        const long long first = (long long)i * chunk_n;
        const int32_t cn = (int32_t)std::min<long long>(chunk_n, n - first);
        const size_t cbytes = (size_t)cn * image_bytes;
        tc_tensor xd{base, cn, c, h, w, dtype}, xh{base + off_xhat, cn, c, h, w, dtype};
        tc_stream_layout l;
        if ((st = tc_encode_bound(m, cb, &xd, params, &l)) != TC_OK) return st;
        // copy in: the slot's tensor was last read by the encode of chunk i - 2
        if (i >= n_slots) TC_CUDA(cudaStreamWaitEvent(ctx->copy_in, ctx->ev_done[slot], 0));
        TC_CUDA(cudaMemcpyAsync(xd.data, (const char *)x_host + (size_t)first * image_bytes, cbytes, cudaMemcpyHostToDevice, ctx->copy_in));
        TC_CUDA(cudaEventRecord(ctx->ev_in[slot], ctx->copy_in));
        // encode + decode: after the copy, and after chunk i - 2 has left the slot's reconstruction
        TC_CUDA(cudaStreamWaitEvent(s, ctx->ev_in[slot], 0));
        if (i >= n_slots) TC_CUDA(cudaStreamWaitEvent(s, ctx->ev_out[slot], 0));
        st = tc_encode(ctx, m, cb, &xd, params, base + off_stream, clay.stream_bytes, (uint16_t *)(base + off_chunk),
                       (uint64_t *)(base + off_tile), nullptr, s);
        if (st != TC_OK) return st;
        st = tc_decode(ctx, m, cb, base + off_stream, clay.stream_bytes, (const uint16_t *)(base + off_chunk),
                       (const uint64_t *)(base + off_tile), params, &xh, s);
        if (st != TC_OK) return st;
        TC_CUDA(cudaEventRecord(ctx->ev_done[slot], s));
        // copy out
        TC_CUDA(cudaStreamWaitEvent(ctx->copy_out, ctx->ev_done[slot], 0));
        TC_CUDA(cudaMemcpyAsync((char *)x_hat_host + (size_t)first * image_bytes, xh.data, cbytes, cudaMemcpyDeviceToHost, ctx->copy_out));
        TC_CUDA(cudaMemcpyAsync(&ctx->chunk_bits[i], base + off_tile + (size_t)l.n_tiles * 8, 8, cudaMemcpyDeviceToHost, ctx->copy_out));
        TC_CUDA(cudaEventRecord(ctx->ev_out[slot], ctx->copy_out));
    }
    // the caller's stream ends after the last copy out, as the one-stream version did
    TC_CUDA(cudaStreamWaitEvent(s, ctx->ev_out[(n_chunks - 1) % n_slots], 0));
    if (n_slots > 1 && n_chunks > 1) TC_CUDA(cudaStreamWaitEvent(s, ctx->ev_out[(n_chunks - 2) % n_slots], 0));
    TC_CUDA(cudaStreamSynchronize(s));
    uint64_t bits = 0;
    for (int i = 0; i < n_chunks; ++i) bits += ctx->chunk_bits[i];
    if (stream_bits) *stream_bits = bits;
    return tc_get_status(ctx, s);
}

// ---- statistics ---------------------------------------------------------------------------

// Statistics of a bf16 tensor on the tensor-core kernels: the batch is worked through in chunks of
// whole tiles; every chunk is encoded (the encoder counts its symbols per coefficient channel and
// the coefficients outside the quantiser's range while it codes), decoded again, and compared with
// the input.  The stream is coded with `cb` when that is a per-layer table, else with a
// fixed-length code of the model's bit width.  Buffers live in the context's arena (grown on
// demand, kept between calls).  Returns TC_ERR_UNSUPPORTED for shapes those kernels do not take.
static tc_status stats_tensor_core(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const tc_tensor *x,
                                   std::vector<unsigned long long> &hist, double &sq, unsigned long long &zeros,
                                   unsigned long long &clamped, cudaStream_t s)
{
    if (x->dtype != TC_BF16 || ctx->force_exact == 1 || ctx->force_exact == 2) return TC_ERR_UNSUPPORTED;
    if (m->c % 16 != 0 || m->k % 16 != 0 || m->k < 16 || m->c > 256 || (x->h * x->w) % 4 != 0 || ((uintptr_t)x->data & 7u) != 0)
        return TC_ERR_UNSUPPORTED;
    const int nsym = 1 << m->bits;
    const tc_codebook *code = (cb && cb->groups == 1) ? cb : nullptr;
    if (!code) {
        if (!ctx->stats_cb[m->bits]) {
            std::vector<uint8_t> lengths(nsym, (uint8_t)m->bits);
            tc_status st = tc_codebook_import(ctx, m->bits, 1, lengths.data(), &ctx->stats_cb[m->bits]);
            if (st != TC_OK) return st;
        }
        code = ctx->stats_cb[m->bits];
    }
    const int hw = x->h * x->w;
    const size_t image_bytes = (size_t)m->c * hw * 2;
    int unit = 1;                                   // images per chunk: whole tiles
    while (((long long)unit * hw) % TC_TILE_PIXELS != 0) unit <<= 1;
    long long chunk_n = std::max<long long>(1, (long long)((32ull << 20) / image_bytes));
    chunk_n = std::max<long long>(unit, chunk_n / unit * unit);
    if (chunk_n > x->n) chunk_n = x->n;
    tc_tensor xc{x->data, (int32_t)chunk_n, x->c, x->h, x->w, x->dtype};
    tc_stream_layout lay;
    tc_status st = tc_encode_bound(m, code, &xc, nullptr, &lay);
    if (st != TC_OK) return st;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t hist_bytes = (size_t)m->k * nsym * sizeof(unsigned long long);
    const size_t off_stream = up((size_t)chunk_n * image_bytes), off_chunk = off_stream + up(lay.stream_bytes),
                 off_tile = off_chunk + up(lay.chunk_len_bytes), off_hist = off_tile + up(lay.tile_off_bytes),
                 off_small = off_hist + up(hist_bytes), total = off_small + 64;
    if (total > ctx->host_arena_bytes) {
        if (ctx->host_arena) { TC_CUDA(cudaDeviceSynchronize()); cudaFree(ctx->host_arena); ctx->host_arena = nullptr; ctx->host_arena_bytes = 0; }
        TC_CUDA(cudaMalloc(&ctx->host_arena, total));
        ctx->host_arena_bytes = total;
    }
    char *base = (char *)ctx->host_arena;
    unsigned long long *d_hist = (unsigned long long *)(base + off_hist);
    double *d_sq = (double *)(base + off_small);
    unsigned long long *d_zeros = (unsigned long long *)(base + off_small + 8), *d_clamped = (unsigned long long *)(base + off_small + 16);
    TC_CUDA(cudaMemsetAsync(base + off_hist, 0, up(hist_bytes) + 64, s));
    const long long tiles_max = ((long long)chunk_n * hw + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS;
    const size_t lookback = kEncodeScratchHeader + (size_t)tiles_max * sizeof(unsigned long long);
    if ((st = ensure_scratch(ctx, lookback)) != TC_OK) return st;
    tc_encode_params prm{lay.chunk_pixels, lay.pixel_splits, 0, 0};
    for (long long first = 0; first < x->n; first += chunk_n) {
        const int32_t cn = (int32_t)std::min<long long>(chunk_n, x->n - first);
        tc_tensor xi{(char *)x->data + (size_t)first * image_bytes, cn, x->c, x->h, x->w, x->dtype};
        tc_tensor xh{base, cn, x->c, x->h, x->w, x->dtype};
        st = tc_encode_with_scratch(ctx, m, code, &xi, lay.chunk_pixels, lay.pixel_splits, base + off_stream, lay.stream_bytes,
                                    (uint16_t *)(base + off_chunk), (uint64_t *)(base + off_tile), nullptr, ctx->scratch, nullptr, s,
                                    d_hist, d_clamped);
        if (st != TC_OK) return st;
        st = tc_decode(ctx, m, code, base + off_stream, lay.stream_bytes, (const uint16_t *)(base + off_chunk),
                       (const uint64_t *)(base + off_tile), &prm, &xh, s);
        if (st != TC_OK) return st;
        if ((st = tc_launch_sqerr(xi.data, xh.data, x->dtype, (long long)cn * m->c * hw, d_sq, d_zeros, s)) != TC_OK) return st;
    }
    hist.assign((size_t)m->k * nsym, 0ull);
    TC_CUDA(cudaMemcpyAsync(hist.data(), d_hist, hist_bytes, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(&sq, d_sq, 8, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(&zeros, d_zeros, 8, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(&clamped, d_clamped, 8, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaStreamSynchronize(s));
    // the encoder counts every symbol but the zero level (m->center): that one takes the rest of the pixels
    const unsigned long long pixels = (unsigned long long)x->n * hw;
    for (int j = 0; j < m->k; ++j) {
        unsigned long long others = 0;
        for (int q = 0; q < nsym; ++q)
            if (q != m->center) others += hist[(size_t)j * nsym + q];
        hist[(size_t)j * nsym + m->center] = pixels - others;
    }
    return TC_OK;
}

// The same on the fp64 kernels: project + quantise (symbols to memory), histogram, reconstruct,
// squared error; the buffers (P * K + V * element bytes) are allocated for the call.
static tc_status stats_exact(tc_ctx *ctx, const tc_model *m, const tc_tensor *x, std::vector<unsigned long long> &hist_out,
                             double &sq, unsigned long long &zeros, unsigned long long &clamped, cudaStream_t s)
{
    const long long pixels = (long long)x->n * x->h * x->w;
    const int nsym = 1 << m->bits;
    const size_t elem = (x->dtype == TC_F32) ? 4 : 2;
    const size_t values = (size_t)pixels * m->c, symbols = (size_t)pixels * m->k;
    const size_t hist_bytes = (size_t)m->k * nsym * sizeof(unsigned long long);

    char *buf = nullptr;
    const size_t off_xhat = (symbols + 255) & ~(size_t)255;
    const size_t off_hist = off_xhat + ((values * elem + 255) & ~(size_t)255);
    const size_t off_small = off_hist + hist_bytes;
    TC_CUDA(cudaMalloc((void **)&buf, off_small + 64));
    struct Free { char *p; ~Free() { cudaFree(p); } } freer{buf};
    uint8_t *d_sym = (uint8_t *)buf;
    void *d_xhat = buf + off_xhat;
    unsigned long long *d_hist = (unsigned long long *)(buf + off_hist);   // always per channel
    double *d_sq = (double *)(buf + off_small);
    unsigned long long *d_zeros = (unsigned long long *)(buf + off_small + 8);
    unsigned long long *d_clamped = (unsigned long long *)(buf + off_small + 16);
    TC_CUDA(cudaMemsetAsync(buf + off_hist, 0, hist_bytes + 64, s));

    EncodeArgs e{};
    e.x = x->data; e.n = x->n; e.c = x->c; e.hw = x->h * x->w; e.k = m->k; e.bits = m->bits; e.groups = 1;
    e.pixels = pixels; e.n_tiles = (pixels + TC_TILE_PIXELS - 1) / TC_TILE_PIXELS; e.chunk_pixels = 1; e.splits = 1;
    e.basis64 = m->d_basis64; e.mean64 = m->d_mean64; e.lo = m->lo; e.step = m->step; e.basis_scale = m->basis_scale;
    e.enc = nullptr; e.dbg_sym = d_sym; e.status = ctx->d_status; e.clamped = d_clamped; e.emit = 0;
    e.bits = m->bits;
    // statistics mode stages no code table: give it an empty one
    e.groups = 0;
    tc_status st = tc_launch_encode_simt(ctx, e, x->dtype, s);
    if (st != TC_OK) return st;
    if ((st = tc_launch_histogram(d_sym, pixels, m->k, m->k, m->bits, d_hist, s)) != TC_OK) return st;

    DecodeArgs d{};
    d.symbols = d_sym; d.n = x->n; d.c = x->c; d.hw = x->h * x->w; d.k = m->k; d.bits = m->bits; d.groups = 1;
    d.pixels = pixels; d.n_tiles = e.n_tiles; d.n_chunks = pixels; d.chunk_pixels = 1; d.splits = 1;
    d.basis64 = m->d_basis64; d.mean64 = m->d_mean64; d.lo = m->lo; d.step = m->step; d.basis_scale = m->basis_scale;
    d.xhat = d_xhat; d.status = ctx->d_status;
    if ((st = tc_launch_decode_simt(ctx, d, x->dtype, s)) != TC_OK) return st;
    if ((st = tc_launch_sqerr(x->data, d_xhat, x->dtype, (long long)values, d_sq, d_zeros, s)) != TC_OK) return st;

    hist_out.assign((size_t)m->k * nsym, 0ull);
    TC_CUDA(cudaMemcpyAsync(hist_out.data(), d_hist, hist_bytes, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(&sq, d_sq, 8, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(&zeros, d_zeros, 8, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaMemcpyAsync(&clamped, d_clamped, 8, cudaMemcpyDeviceToHost, s));
    TC_CUDA(cudaStreamSynchronize(s));
    return TC_OK;
}

tc_status tc_stats(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const tc_tensor *x, tc_stats_out *out,
                   void *cuda_stream)
{
    if (!ctx || !m || !out || !valid_tensor(x)) return TC_ERR_INVALID_ARG;
    if (x->c != m->c) return TC_ERR_INVALID_ARG;
    if (x->dtype != m->basis_dtype && m->basis_dtype != TC_INT8) return TC_ERR_UNSUPPORTED;   // an 8-bit basis serves both tensor types
    if (out->groups != 1 && out->groups != m->k) return TC_ERR_INVALID_ARG;
    if (cb && (cb->bits != m->bits || (cb->groups != 1 && cb->groups != m->k))) return TC_ERR_INVALID_ARG;
    const long long pixels = (long long)x->n * x->h * x->w;
    if (pixels == 0) return TC_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int nsym = 1 << m->bits, groups = out->groups;
    const size_t values = (size_t)pixels * m->c, symbols = (size_t)pixels * m->k;

    std::vector<unsigned long long> hist;
    double sq = 0.0;
    unsigned long long zeros = 0, clamped = 0;
    // bf16 tensors of up to 256 channels: the tensor-core kernels, which count while they code;
    // everything else: the fp64 kernels
    tc_status st = stats_tensor_core(ctx, m, cb, x, hist, sq, zeros, clamped, s);
    if (st == TC_ERR_UNSUPPORTED) st = stats_exact(ctx, m, x, hist, sq, zeros, clamped, s);
    if (st != TC_OK) return st;

    // fold the per-channel counts to the requested granularity
    std::vector<unsigned long long> folded((size_t)groups * nsym, 0ull);
    for (int j = 0; j < m->k; ++j)
        for (int v = 0; v < nsym; ++v) folded[(size_t)(groups == 1 ? 0 : j) * nsym + v] += hist[(size_t)j * nsym + v];
    if (out->hist)
        TC_CUDA(cudaMemcpy(out->hist, folded.data(), folded.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice));
    double entropy = 0.0, mean_len = 0.0;
    for (int g = 0; g < groups; ++g) {
        double tot = 0.0, h = 0.0;
        for (int v = 0; v < nsym; ++v) tot += (double)folded[(size_t)g * nsym + v];
        for (int v = 0; v < nsym; ++v) {
            const double cnt = (double)folded[(size_t)g * nsym + v];
            if (cnt > 0) h -= cnt / tot * std::log2(cnt / tot);
        }
        entropy += h / groups;
    }
    if (cb) {
        double tot = 0.0, acc = 0.0;
        for (int j = 0; j < m->k; ++j)
            for (int v = 0; v < nsym; ++v) {
                const double cnt = (double)hist[(size_t)j * nsym + v];
                tot += cnt;
                acc += cnt * cb->lengths[(size_t)(cb->groups == 1 ? 0 : j) * nsym + v];
            }
        mean_len = acc / tot;
    }
    out->entropy = entropy;
    out->mean_length = mean_len;
    out->mse = sq / (double)values;
    out->clamped_fraction = (double)clamped / (double)symbols;
    out->zero_fraction = (double)zeros / (double)values;
    double total_energy = 0.0, run = 0.0;
    for (double v : m->eig) total_energy += v;
    int need = m->c;
    for (int j = 0; j < m->c && total_energy > 0.0; ++j) {
        run += m->eig[j];
        if (run >= 0.9 * total_energy) { need = j + 1; break; }
    }
    out->energy_ratio_90 = (double)need / (double)m->c;
    return TC_OK;
}

}  // extern "C"
