// Exact (fp64) encode and decode kernels: one thread per pixel, plain FMA-free double
// arithmetic in the order the definition states, so that fp32 tensors -- whose products do not
// fit the bf16 tensor-core path -- are coded without any rounding of their own.  They are
// also the validation path and the statistics mode.
//
// The same kernels have an fp32 mode (kFp32) for bf16 tensors whose shape the tensor-core
// kernels do not take (channel or coefficient counts that are not multiples of 16): bf16 x bf16 products are exact
// in fp32, accumulation is fp32 with fused multiply-adds, and the quantiser / dequantiser use
// the same folded constants as the tensor-core kernels (acc / step + bias, step * acc + bias
// around the centre symbol), so that the two bf16 routes take their decisions alike.
//
// Encode (Section 3: transform, quantiser, VLC): y_j = sum_c T[j][c] (x_c - mu_c),
// q = clamp(rint((y - lo)/step)), code lookup, bit offsets by scan + tile look-back, pack.
// Decode (Section 3: VLD, inverse quantiser, inverse transform): table-driven canonical
// Huffman decode per chunk, y_hat = lo + q*step, x_hat_c = sum_j T[j][c] y_hat_j + mu_c.
#include "device_utils.cuh"

namespace {

constexpr int kThreads = TC_TILE_PIXELS;
constexpr int kRowBlock = 8;           // basis rows (encode) / columns (decode) per pass, fp64 mode
constexpr int kRowBlock32 = 16;        // the same in fp32 mode
constexpr int kEncSmemEntries = 2048;  // code tables up to this many entries are staged

using namespace tcdev;

template <typename TIn, bool kFp32>
__global__ void __launch_bounds__(kThreads) encode_simt_kernel(EncodeArgs a)
{
    constexpr int RB = kFp32 ? kRowBlock32 : kRowBlock;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_mean = reinterpret_cast<double *>(smem_raw);            // [C]  (fp64 mode)
    double *s_panel = s_mean + a.c;                                    // [RB][C] doubles, or [C][RB] floats in fp32 mode
    float *s_panel32 = reinterpret_cast<float *>(s_panel);
    uint32_t *s_enc = reinterpret_cast<uint32_t *>(s_panel + kRowBlock * a.c);      // 8 doubles = 16 floats per channel
    const int nsym = 1 << a.bits;
    const int enc_entries = a.groups * nsym;
    const bool enc_in_smem = enc_entries <= kEncSmemEntries;
    uint8_t *s_q = reinterpret_cast<uint8_t *>(s_enc + (enc_in_smem ? enc_entries : 0));  // [K][128]

    __shared__ long long s_tile;
    __shared__ unsigned int s_warp_sums[4];
    __shared__ unsigned long long s_base;
    __shared__ int s_write_ok;
    __shared__ unsigned int s_pixel_off[TC_TILE_PIXELS + 1];   // bit offset of every pixel in the tile, then the tile's bits

    const int t = threadIdx.x;
    if (t == 0) s_tile = a.emit ? (long long)atomicAdd(a.ticket, 1u) : (long long)blockIdx.x;
    for (int i = t; i < a.c; i += kThreads) s_mean[i] = a.mean64[i];
    if (enc_in_smem)
        for (int i = t; i < enc_entries; i += kThreads) s_enc[i] = a.enc[i];
    __syncthreads();
    const long long tile = s_tile;
    const uint32_t *enc = enc_in_smem ? s_enc : a.enc;

    const long long p = tile * TC_TILE_PIXELS + t;
    const bool valid = p < a.pixels;
    const TIn *xin = reinterpret_cast<const TIn *>(a.x);
    long long xbase = 0;
    if (valid) {
        const long long img = p / a.hw;
        const long long s = p - img * a.hw;
        xbase = img * a.c * (long long)a.hw + s;
    }
    const double top = (double)(nsym - 1);
    unsigned int clamped = 0;

    if (a.sym_in) {
        // the symbols were computed by the one-thread-per-value projection kernel
        if (valid)
            for (int j = 0; j < a.k; ++j) s_q[j * kThreads + t] = a.sym_in[p * a.k + j];
    } else
    for (int j0 = 0; j0 < a.k; j0 += RB) {
        __syncthreads();
        if constexpr (kFp32) {
            // [C][RB] floats: the RB coefficients of one channel are one 64-byte row
            for (int i = t; i < RB * a.c; i += kThreads) {
                const int jj = i / a.c, cc = i - jj * a.c;
                s_panel32[cc * RB + jj] = (j0 + jj < a.k) ? __bfloat162float(a.basis_bf16[(long long)(j0 + jj) * a.c + cc]) : 0.f;
            }
        } else {
            for (int i = t; i < kRowBlock * a.c; i += kThreads) {
                const int jj = i / a.c, cc = i - jj * a.c;
                s_panel[i] = (j0 + jj < a.k) ? a.basis64[(long long)(j0 + jj) * a.c + cc] : 0.0;
            }
        }
        __syncthreads();
        if constexpr (kFp32) {
            if (valid) {
                float acc[RB];
#pragma unroll
                for (int jj = 0; jj < RB; ++jj) acc[jj] = 0.f;
                for (int cc = 0; cc < a.c; ++cc) {
                    const float xv = (float)load_as_double(xin + xbase + (long long)cc * a.hw);
                    const float4 *row = reinterpret_cast<const float4 *>(s_panel32 + cc * RB);
#pragma unroll
                    for (int q4 = 0; q4 < RB / 4; ++q4) {
                        const float4 w = row[q4];
                        acc[4 * q4 + 0] = fmaf(w.x, xv, acc[4 * q4 + 0]);
                        acc[4 * q4 + 1] = fmaf(w.y, xv, acc[4 * q4 + 1]);
                        acc[4 * q4 + 2] = fmaf(w.z, xv, acc[4 * q4 + 2]);
                        acc[4 * q4 + 3] = fmaf(w.w, xv, acc[4 * q4 + 3]);
                    }
                }
                const float inv_step = (float)(a.basis_scale / a.step);     // the operand holds basis / basis_scale
#pragma unroll
                for (int jj = 0; jj < RB; ++jj) {
                    const int j = j0 + jj;
                    if (j < a.k) {
                        const float u = fmaf(acc[jj], inv_step, a.enc_bias[j]);      // (y - lo) / step
                        if (u < 0.f || u > (float)top) ++clamped;
                        const float r = fminf(fmaxf(rintf(u), 0.f), (float)top);
                        const unsigned int q = (unsigned int)r;
                        s_q[j * kThreads + t] = (uint8_t)q;
                        if (a.dbg_coef) a.dbg_coef[p * a.k + j] = fmaf(acc[jj], (float)a.basis_scale, -a.tmu32[j]);
                        if (a.dbg_sym) a.dbg_sym[p * a.k + j] = (uint8_t)q;
                    }
                }
            }
        } else if (valid) {
            double acc[kRowBlock];
#pragma unroll
            for (int jj = 0; jj < kRowBlock; ++jj) acc[jj] = 0.0;
            for (int cc = 0; cc < a.c; ++cc) {
                const double d = __dsub_rn(load_as_double(xin + xbase + (long long)cc * a.hw), s_mean[cc]);
#pragma unroll
                for (int jj = 0; jj < kRowBlock; ++jj)
                    acc[jj] = __dadd_rn(acc[jj], __dmul_rn(s_panel[jj * a.c + cc], d));
            }
#pragma unroll
            for (int jj = 0; jj < kRowBlock; ++jj) {
                const int j = j0 + jj;
                if (j < a.k) {
                    const double y = acc[jj];
                    const double u = __ddiv_rn(__dsub_rn(y, a.lo), a.step);
                    double r = rint(u);
                    if (u < 0.0 || u > top) ++clamped;
                    r = fmin(fmax(r, 0.0), top);
                    const unsigned int q = (unsigned int)r;
                    s_q[j * kThreads + t] = (uint8_t)q;
                    if (a.dbg_coef) a.dbg_coef[p * a.k + j] = (float)y;
                    if (a.dbg_sym) a.dbg_sym[p * a.k + j] = (uint8_t)q;
                }
            }
        }
    }
    if (a.clamped) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) clamped += __shfl_xor_sync(0xffffffffu, clamped, d);
        if ((t & 31) == 0 && clamped) atomicAdd(a.clamped, (unsigned long long)clamped);
    }
    if (!a.emit) return;

    // ---- bit lengths, offsets --------------------------------------------------------
    unsigned int my_bits = 0;
    unsigned int part_bits[4] = {0u, 0u, 0u, 0u};             // per run of K / splits coefficients
    const int k_part = a.k / a.splits;
    if (valid)
        for (int j = 0; j < a.k; ++j) {
            const int g = (a.groups == 1) ? 0 : j;
            const unsigned int l = enc[g * nsym + s_q[j * kThreads + t]] & 0xffu;
            my_bits += l;
            part_bits[j / k_part] += l;
        }
    unsigned int tile_bits;
    const unsigned int my_off = group_exclusive_scan_128(my_bits, s_warp_sums, t, 1, tile_bits);
    const unsigned long long padded = ((unsigned long long)tile_bits + 127ull) & ~127ull;
    if (t < 32) {
        bool ok;
        const unsigned long long base = tile_lookback(a.tile_state, tile, padded, a.status, ok);
        if (t == 0) {
            bool fits = base + padded <= a.capacity_bits;
            if (ok && !fits) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
            s_base = base;
            s_write_ok = (ok && fits) ? 1 : 0;
            a.tile_off[tile] = base;
            if (tile == a.n_tiles - 1) a.tile_off[a.n_tiles] = base + padded;
        }
    }
    __syncthreads();
    const unsigned long long base = s_base;
    // chunk lengths: a chunk is chunk_pixels pixels, or one of `splits` runs of one pixel
    s_pixel_off[t] = my_off;
    if (t == 0) s_pixel_off[TC_TILE_PIXELS] = tile_bits;
    __syncthreads();
    if (valid) {
        if (a.splits > 1) {
            for (int sp = 0; sp < a.splits; ++sp) a.chunk_len[p * a.splits + sp] = (uint16_t)part_bits[sp];
        } else if ((p % a.chunk_pixels) == 0) {
            const int last = min(t + a.chunk_pixels, TC_TILE_PIXELS);
            a.chunk_len[p / a.chunk_pixels] = (uint16_t)(s_pixel_off[last] - my_off);
        }
    }
    if (!s_write_ok) return;

    // ---- zero the tile's words, then pack --------------------------------------------
    {
        uint4 *dst = reinterpret_cast<uint4 *>(a.stream + (base >> 5));
        const unsigned int n16 = (unsigned int)(padded >> 7);
        for (unsigned int i = t; i < n16; i += kThreads) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    if (valid) {
        BitWriter w;
        w.init(a.stream, base + my_off);
        for (int j = 0; j < a.k; ++j) {
            const int g = (a.groups == 1) ? 0 : j;
            const uint32_t e = enc[g * nsym + s_q[j * kThreads + t]];
            w.put(e >> 8, (int)(e & 0xffu));
        }
        w.finish();
    }
}

// Sequential reader of an MSB-first bit stream with a 64-bit window; words past `end_word`
// read as zero so that a corrupt offset can never cause an out-of-bounds load.
struct BitReader {
    const uint32_t *words;
    unsigned long long window;   // upcoming bits, left-aligned
    int avail;
    unsigned long long next_word, end_word;

    __device__ __forceinline__ uint32_t fetch()
    {
        const uint32_t v = (next_word < end_word) ? __ldg(words + next_word) : 0u;
        ++next_word;
        return v;
    }
    __device__ __forceinline__ void init(const uint32_t *base, unsigned long long bitpos, unsigned long long end_bits)
    {
        words = base;
        next_word = bitpos >> 5;
        end_word = end_bits >> 5;
        const unsigned long long hi = fetch();
        const unsigned long long lo = fetch();
        const int sh = (int)(bitpos & 31);
        window = ((hi << 32) | lo) << sh;
        avail = 64 - sh;
    }
    __device__ __forceinline__ uint32_t peek(int nbits) const { return (uint32_t)(window >> (64 - nbits)); }
    __device__ __forceinline__ void skip(int nbits)
    {
        window <<= nbits;
        avail -= nbits;
        if (avail <= 32) {
            window |= (unsigned long long)fetch() << (32 - avail);
            avail += 32;
        }
    }
};

template <typename TOut, bool kFp32>
__global__ void __launch_bounds__(kThreads) decode_simt_kernel(DecodeArgs a)
{
    constexpr int RB = kFp32 ? kRowBlock32 : kRowBlock;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_mean = reinterpret_cast<double *>(smem_raw);        // [C]  (fp64 mode)
    double *s_panel = s_mean + a.c;                                // [K][RB] doubles (fp64) or floats (fp32: same bytes)
    float *s_panel32 = reinterpret_cast<float *>(s_panel);
    uint8_t *s_q = reinterpret_cast<uint8_t *>(s_panel + (size_t)a.k * kRowBlock);   // [K][128]
    __shared__ int s_bad;
    __shared__ uint16_t s_len[4 * TC_TILE_PIXELS];                 // chunk lengths of the tile

    const int t = threadIdx.x;
    const long long tile = blockIdx.x;
    const long long p = tile * TC_TILE_PIXELS + t;
    const bool valid = p < a.pixels;
    for (int i = t; i < a.c; i += kThreads) s_mean[i] = a.mean64[i];
    if (t == 0) s_bad = 0;
    __syncthreads();

    if (a.symbols) {
        if (valid)
            for (int j = 0; j < a.k; ++j) s_q[j * kThreads + t] = a.symbols[p * a.k + j];
    } else {
        const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
        const bool tile_ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
        if (!tile_ok) {
            if (t == 0) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
            return;
        }
        const int chunks_per_tile = a.splits * TC_TILE_PIXELS / a.chunk_pixels;      // at most 512
        const int chunk_symbols = a.chunk_pixels * a.k / a.splits;
        for (int ci = t; ci < chunks_per_tile; ci += kThreads) {
            const long long ch = tile * chunks_per_tile + ci;
            s_len[ci] = ch < a.n_chunks ? a.chunk_len[ch] : (uint16_t)0;
        }
        __syncthreads();
        const int lut_size = 1 << a.lut_bits;
        for (int ci = t; ci < chunks_per_tile; ci += kThreads) {
            if (tile * chunks_per_tile + ci >= a.n_chunks) break;
            // the chunk starts after the tile's earlier chunks and must end after its own length
            unsigned long long off = 0;
            for (int i = 0; i < ci; ++i) off += s_len[i];
            const unsigned int want = s_len[ci];
            bool bad = base + off + want > end;
            if (!bad) {
                BitReader r;
                r.init(a.stream, base + off, end);
                unsigned int used = 0;
                const int first = ci * chunk_symbols;                 // first symbol, counted inside the tile
                for (int n = first; n < first + chunk_symbols; ++n) {
                    const int lp = n / a.k, j = n - lp * a.k;           // pixel inside the tile, coefficient
                    if (tile * TC_TILE_PIXELS + lp >= a.pixels) break;
                    const int g = (a.groups == 1) ? 0 : j;
                    const uint32_t e = __ldg(a.lut + (size_t)g * lut_size + r.peek(a.lut_bits));
                    const int len = (int)(e & 0xffu);
                    s_q[j * kThreads + lp] = (uint8_t)(e >> 8);
                    r.skip(len);
                    used += len;
                    if (len == 0) bad = true;
                }
                if (used != want) bad = true;
            }
            if (bad) s_bad = 1;
        }
        __syncthreads();
        if (s_bad) {
            if (t == 0) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
            return;
        }
    }

    if (a.sym_out) {
        // the reconstruction runs in the one-thread-per-value kernel
        if (valid)
            for (int j = 0; j < a.k; ++j) a.sym_out[p * a.k + j] = s_q[j * kThreads + t];
        return;
    }
    TOut *out = reinterpret_cast<TOut *>(a.xhat);
    long long obase = 0;
    if (valid) {
        const long long img = p / a.hw;
        const long long s = p - img * a.hw;
        obase = img * a.c * (long long)a.hw + s;
    }
    for (int c0 = 0; c0 < a.c; c0 += RB) {
        __syncthreads();
        if constexpr (kFp32) {
            for (int i = t; i < a.k * RB; i += kThreads) {
                const int cc = i / a.k, j = i - cc * a.k;             // consecutive threads read consecutive j of one channel row
                s_panel32[j * RB + cc] = (c0 + cc < a.c) ? __bfloat162float(a.basis_t_bf16[(long long)(c0 + cc) * a.k + j]) : 0.f;
            }
        } else {
            for (int i = t; i < a.k * kRowBlock; i += kThreads) {
                const int j = i / kRowBlock, cc = i - j * kRowBlock;
                s_panel[i] = (c0 + cc < a.c) ? a.basis64[(long long)j * a.c + c0 + cc] : 0.0;
            }
        }
        __syncthreads();
        if constexpr (kFp32) {
            if (valid) {
                float acc[RB];
#pragma unroll
                for (int cc = 0; cc < RB; ++cc) acc[cc] = 0.f;
                for (int j = 0; j < a.k; ++j) {
                    const float qv = (float)((int)s_q[j * kThreads + t] - a.center);
                    const float4 *row = reinterpret_cast<const float4 *>(s_panel32 + j * RB);
#pragma unroll
                    for (int q4 = 0; q4 < RB / 4; ++q4) {
                        const float4 w = row[q4];
                        acc[4 * q4 + 0] = fmaf(w.x, qv, acc[4 * q4 + 0]);
                        acc[4 * q4 + 1] = fmaf(w.y, qv, acc[4 * q4 + 1]);
                        acc[4 * q4 + 2] = fmaf(w.z, qv, acc[4 * q4 + 2]);
                        acc[4 * q4 + 3] = fmaf(w.w, qv, acc[4 * q4 + 3]);
                    }
                }
                const float step = (float)(a.step * a.basis_scale);        // the operand holds basis / basis_scale
#pragma unroll
                for (int cc = 0; cc < RB; ++cc)
                    if (c0 + cc < a.c)
                        {
                        float v = fmaf(acc[cc], step, a.dec_bias[c0 + cc]);
                        if (a.relu) v = fmaxf(v, 0.f);
                        store_rounded(out + obase + (long long)(c0 + cc) * a.hw, (double)v);
                    }
            }
        } else if (valid) {
            double acc[kRowBlock];
#pragma unroll
            for (int cc = 0; cc < kRowBlock; ++cc) acc[cc] = 0.0;
            for (int j = 0; j < a.k; ++j) {
                const double yh = __dadd_rn(a.lo, __dmul_rn((double)s_q[j * kThreads + t], a.step));
#pragma unroll
                for (int cc = 0; cc < kRowBlock; ++cc)
                    acc[cc] = __dadd_rn(acc[cc], __dmul_rn(s_panel[j * kRowBlock + cc], yh));
            }
#pragma unroll
            for (int cc = 0; cc < kRowBlock; ++cc)
                if (c0 + cc < a.c)
                    {
                    double v = __dadd_rn(acc[cc], s_mean[c0 + cc]);
                    if (a.relu && v < 0.0) v = 0.0;
                    store_rounded(out + obase + (long long)(c0 + cc) * a.hw, v);
                }
        }
    }
}

size_t encode_smem_bytes(const EncodeArgs &a)
{
    const int entries = a.groups << a.bits;
    return sizeof(double) * (size_t)a.c * (1 + kRowBlock) + (entries <= kEncSmemEntries ? entries * 4u : 0u) +
           (size_t)a.k * kThreads;
}
size_t decode_smem_bytes(const DecodeArgs &a)
{
    return sizeof(double) * ((size_t)a.c + (size_t)a.k * kRowBlock) + (size_t)a.k * kThreads;
}

template <typename K, typename A>
tc_status launch(K kernel, const A &a, size_t smem, const tc_ctx *ctx, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    if (smem > (size_t)ctx->max_smem_optin) return TC_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TC_ERR_CUDA;
    kernel<<<(unsigned int)a.n_tiles, kThreads, smem, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

}  // namespace

tc_status tc_launch_encode_simt(const tc_ctx *ctx, const EncodeArgs &a, int dtype, cudaStream_t s)
{
    const size_t smem = encode_smem_bytes(a);
    if (dtype == TC_F32) return launch(encode_simt_kernel<float, false>, a, smem, ctx, s);
    return launch(encode_simt_kernel<__nv_bfloat16, false>, a, smem, ctx, s);
}

tc_status tc_launch_decode_simt(const tc_ctx *ctx, const DecodeArgs &a, int dtype, cudaStream_t s)
{
    const size_t smem = decode_smem_bytes(a);
    if (dtype == TC_F32) return launch(decode_simt_kernel<float, false>, a, smem, ctx, s);
    return launch(decode_simt_kernel<__nv_bfloat16, false>, a, smem, ctx, s);
}

// fp32 mode, bf16 tensors only (the shared-memory carve-up is the fp64 mode's: 16 floats take
// the room of 8 doubles)
tc_status tc_launch_encode_simt_fp32(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s)
{
    if (!a.basis_bf16 || !a.enc_bias || !a.tmu32) return TC_ERR_UNSUPPORTED;
    return launch(encode_simt_kernel<__nv_bfloat16, true>, a, encode_smem_bytes(a), ctx, s);
}

tc_status tc_launch_decode_simt_fp32(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s)
{
    if (!a.basis_t_bf16 || !a.dec_bias) return TC_ERR_UNSUPPORTED;
    return launch(decode_simt_kernel<__nv_bfloat16, true>, a, decode_smem_bytes(a), ctx, s);
}
