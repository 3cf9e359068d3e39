// Fused tensor-core decode for bf16 tensors (Section 3: VLD, inverse quantiser, inverse
// transform).
//
// One persistent block per SM; two tiles of 128 pixels are in flight at a time.  Warp roles:
//   warps 0-3, 4-7     two VLD groups (alternating tiles): one thread per chunk walks its part
//                      of the bit stream with a table-driven canonical Huffman decoder and
//                      writes the symbols, as exact bf16 integers, into the K-major A operand
//   warps 8-11, 12-15  two epilogue groups: TMEM -> registers, x_hat = step * acc + bias,
//                      round to bf16, NCHW stores
//   warps 16, 17       one thread each issues the tcgen05.mma of its group:
//                      D[pixel][c] = (Q[pixel][j] - center) * T[j][c]
// The transposed basis (bf16, C x K, K-major) stays resident in shared memory; dequantisation
// is folded into the epilogue so that the MMA consumes integers exactly: the symbols minus the
// symbol `center` whose level is nearest to y = 0 (most coefficients sit there, so the
// accumulators stay small and nothing large cancels in fp32), with
// bias_c = mu_c + (lo + center*step) * sum_j T[j][c].
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace tcdev;
using namespace sm100;

constexpr int kPanelK = 64;                                   // coefficients per ring stage
constexpr int kStageBytes = kPanelK * TC_TILE_PIXELS * 2;     // 16 KB
constexpr int kThreads = 18 * 32;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kMaxStages = 4;                                 // per group

struct SmemLayout {
    uint32_t basis, ring, lut, bias, total;
    int stages;                                               // ring stages per group
};

__host__ __device__ inline SmemLayout smem_layout(int c, int k, int lut_entries, int chunk_pixels, int budget)
{
    SmemLayout l;
    l.basis = 0;
    l.lut = (uint32_t)(((size_t)c * k * 2 + 1023) & ~(size_t)1023);
    l.bias = l.lut + (uint32_t)lut_entries * 4;
    l.ring = (l.bias + (uint32_t)c * 4 + 1023) & ~1023u;
    const int n_panels = (k + kPanelK - 1) / kPanelK;
    // a chunk of several pixels is decoded pixel by pixel, so every panel of the tile has to
    // stay resident until the chunk's last pixel is done; single-pixel chunks stream through
    // two stages
    int want = chunk_pixels > 1 ? n_panels : 2;
    if (want < 2) want = 2;
    l.stages = want;
    l.total = l.ring + 2u * (uint32_t)want * kStageBytes;
    if ((int)l.total > budget || want > kMaxStages) l.stages = 0;
    return l;
}

// MSB-first reader over 32-bit words with a 64-bit window held in two registers.  Words at or
// past `end` read as zero, so a corrupt offset can never cause an out-of-bounds load.
struct WindowReader {
    const uint32_t *words;
    unsigned long long next, end;     // word indices
    uint32_t hi, lo;                  // upcoming bits, left-aligned in hi:lo
    int avail;                        // valid bits in the window

    __device__ __forceinline__ uint32_t fetch()
    {
        const uint32_t w = (next < end) ? __ldg(words + next) : 0u;
        ++next;
        return w;
    }
    __device__ __forceinline__ void init(const uint32_t *base, unsigned long long bitpos, unsigned long long end_bits)
    {
        words = base;
        next = bitpos >> 5;
        end = end_bits >> 5;
        const uint32_t w0 = fetch(), w1 = fetch();
        const int sh = (int)(bitpos & 31);
        hi = __funnelshift_l(w1, w0, sh);
        lo = w1 << sh;
        avail = 64 - sh;
    }
    __device__ __forceinline__ uint32_t peek(int nbits) const { return hi >> (32 - nbits); }
    // nbits < 32
    __device__ __forceinline__ void skip(int nbits)
    {
        hi = __funnelshift_l(lo, hi, nbits);
        lo <<= nbits;
        avail -= nbits;
    }
    // keeps more than 32 valid bits in the window
    __device__ __forceinline__ void refill()
    {
        if (avail <= 32) {
            const uint32_t w = fetch();
            const int s = 32 - avail;                 // 0..31
            hi |= __funnelshift_l(w, 0u, s);
            lo |= w << s;
            avail += 32;
        }
    }
};

template <bool kPerChannel>
__global__ void __launch_bounds__(kThreads, 1) decode_tc_kernel(DecodeArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_full[2][kMaxStages], s_empty[2][kMaxStages], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lut_size = 1 << a.lut_bits;
    const SmemLayout L = smem_layout(a.c, a.k, kPerChannel ? 0 : lut_size, a.chunk_pixels, 1 << 30);
    const int stages = L.stages;
    unsigned char *s_basis = smem + L.basis;
    uint32_t *s_lut = reinterpret_cast<uint32_t *>(smem + L.lut);
    float *s_bias = reinterpret_cast<float *>(smem + L.bias);
    const uint32_t ring_addr = smem_u32(smem + L.ring);
    const uint32_t basis_addr = smem_u32(s_basis);
    const uint32_t lut_addr = smem_u32(s_lut);
    const int n_panels = (a.k + kPanelK - 1) / kPanelK;

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int g = 0; g < 2; ++g) {
            for (int s = 0; s < kMaxStages; ++s) { mbar_init(smem_u32(&s_full[g][s]), 128); mbar_init(smem_u32(&s_empty[g][s]), 1); }
            mbar_init(smem_u32(&s_tfull[g]), 1);
            mbar_init(smem_u32(&s_tempty[g]), 128);
        }
        mbar_fence_init();
    }
    if (warp == 16) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    {
        // transposed basis [c][j] -> K-major core matrices: (c/8)*sbo + (j/8)*128 + (c%8)*16 + (j%8)*2
        const uint32_t sbo = (uint32_t)(a.k / 8) * 128u;
        const int chunks_per_row = a.k / 8;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.basis_t_bf16);
        for (int i = tid; i < a.c * chunks_per_row; i += kThreads) {
            const int ch = i / chunks_per_row, j8 = i - ch * chunks_per_row;
            *reinterpret_cast<uint4 *>(s_basis + (ch >> 3) * sbo + j8 * 128 + (ch & 7) * 16) = __ldg(src + i);
        }
        for (int i = tid; i < a.c; i += kThreads) s_bias[i] = a.dec_bias[i];
        if (!kPerChannel)
            for (int i = tid; i < lut_size; i += kThreads) {
                // table entry: bf16(symbol - center) << 16 | symbol << 8 | length
                const uint32_t e = a.lut32[i];
                const float centred = (float)((int)((e >> 8) & 0xffu) - a.center);
                s_lut[i] = (__float_as_uint(centred) & 0xffff0000u) | (e & 0xffffu);
            }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    const long long my_tiles = (a.n_tiles > blockIdx.x) ? (a.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp < 8) {
        // ================= VLD groups =================
        const int grp = warp >> 2;
        const int t = tid & 127;
        const int cp = a.chunk_pixels;
        const int chunks_per_tile = TC_TILE_PIXELS / cp;
        const uint32_t ring_g = ring_addr + (uint32_t)grp * stages * kStageBytes;
        long long it = 0;                       // panels produced by this group so far
        bool alive = true;
        for (long long tl = grp; tl < my_tiles && alive; tl += 2) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
            const bool tile_ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
            const long long ch = tile * chunks_per_tile + t;
            bool active = tile_ok && t < chunks_per_tile && ch < a.n_chunks;
            bool bad = !tile_ok;
            WindowReader r;
            unsigned long long used = 0;
            if (active) {
                const unsigned long long off = a.chunk_off[ch];
                if (base + off > end) { bad = true; active = false; }
                else { r.init(a.stream, base + off, end); used = base + off; }
            }
            const int n_pix = active ? (int)min((long long)cp, a.pixels - (tile * TC_TILE_PIXELS + (long long)t * cp)) : 0;
            for (int pp = 0; pp < cp && alive; ++pp) {
                const bool decode = pp < n_pix;
                const int row = t * cp + pp;       // only meaningful while t < chunks_per_tile
                for (int kp = 0; kp < n_panels; ++kp) {
                    const long long pit = it + kp;
                    const int s = (int)(pit % stages);
                    if (pp == 0 && !mbar_wait(smem_u32(&s_empty[grp][s]), (uint32_t)(((pit / stages) & 1) ^ 1))) { alive = false; break; }
                    if (decode) {
                        const int k0 = kp * kPanelK;
                        const int nk8 = min(kPanelK, a.k - k0) >> 3;
                        const uint32_t dst = ring_g + s * kStageBytes + (row >> 3) * 128 + (row & 7) * 16;
                        for (int k8 = 0; k8 < nk8; ++k8) {
                            uint32_t pk[4];
#pragma unroll
                            for (int i = 0; i < 8; i += 2) {
                                r.refill();
                                uint32_t e0, e1;
                                if constexpr (kPerChannel) e0 = __ldg(a.lut32 + (size_t)(k0 + k8 * 8 + i) * lut_size + r.peek(a.lut_bits));
                                else asm("ld.shared.u32 %0, [%1];" : "=r"(e0) : "r"(lut_addr + r.peek(a.lut_bits) * 4u));
                                r.skip((int)(e0 & 0xffu));
                                if constexpr (kPerChannel) e1 = __ldg(a.lut32 + (size_t)(k0 + k8 * 8 + i + 1) * lut_size + r.peek(a.lut_bits));
                                else asm("ld.shared.u32 %0, [%1];" : "=r"(e1) : "r"(lut_addr + r.peek(a.lut_bits) * 4u));
                                r.skip((int)(e1 & 0xffu));
                                used += (e0 & 0xffu) + (e1 & 0xffu);
                                if constexpr (kPerChannel) {   // tables in global memory hold the plain symbol
                                    e0 = __float_as_uint((float)((int)((e0 >> 8) & 0xffu) - a.center));
                                    e1 = __float_as_uint((float)((int)((e1 >> 8) & 0xffu) - a.center));
                                }
                                pk[i >> 1] = __byte_perm(e0, e1, 0x7632);     // bf16(sym0) | bf16(sym1) << 16
                            }
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + k8 * 2048), "r"(pk[0]),
                                         "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                        }
                    }
                    if (pp == cp - 1) {
                        fence_proxy_async_smem();
                        mbar_arrive(smem_u32(&s_full[grp][s]));
                    }
                }
            }
            it += n_panels;
            if (active && used > end) bad = true;
            if (bad) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
        }
        if (!alive && t == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else if (warp < 16) {
        // ================= epilogue groups =================
        const int grp = (warp - 8) >> 2;
        const int t = tid & 127;
        const int wq = warp & 3;
        const float step = (float)a.step;
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.xhat);
        bool alive = true;
        for (long long tl = grp; tl < my_tiles && alive; tl += 2) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            const long long p = tile * TC_TILE_PIXELS + t;
            const bool valid = p < a.pixels;
            const long long img = valid ? p / a.hw : 0;
            __nv_bfloat16 *dst = out + img * a.c * (long long)a.hw + (valid ? p - img * a.hw : 0);
            if (!mbar_wait(smem_u32(&s_tfull[grp]), (uint32_t)((tl >> 1) & 1))) { alive = false; break; }
            tc_fence_after_sync();
            const uint32_t trow = tmem_base + grp * kAccCols + ((uint32_t)(wq * 32) << 16);
            for (int c0 = 0; c0 < a.c; c0 += 32) {
                uint32_t r[32];
                const bool full = a.c - c0 >= 32;
                if (full) tmem_ld_32x32b_x32(trow + c0, r);
                else {
                    uint32_t r16[16];
                    tmem_ld_32x32b_x16(trow + c0, r16);
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = r16[i];
                }
                tmem_ld_wait();
                if (valid) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        if (i < 16 || full) {
                            const float v0 = fmaf(__uint_as_float(r[i]), step, s_bias[c0 + i]);
                            const float v1 = fmaf(__uint_as_float(r[i + 1]), step, s_bias[c0 + i + 1]);
                            const __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                            dst[(long long)(c0 + i) * a.hw] = h.x;
                            dst[(long long)(c0 + i + 1) * a.hw] = h.y;
                        }
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&s_tempty[grp]));
        }
        if (!alive && t == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else {
        // ================= MMA issuers (one per group) =================
        const int grp = warp - 16;
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(TC_TILE_PIXELS, a.c, /*A K-major*/ false, /*B K-major*/ false);
            const uint32_t b_sbo = (uint32_t)(a.k / 8) * 128u;
            const uint32_t ring_g = ring_addr + (uint32_t)grp * stages * kStageBytes;
            long long it = 0;
            bool alive = true;
            for (long long tl = grp; tl < my_tiles && alive; tl += 2) {
                if (!mbar_wait(smem_u32(&s_tempty[grp]), (uint32_t)(((tl >> 1) & 1) ^ 1))) { alive = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + grp * kAccCols;
                for (int kp = 0; kp < n_panels; ++kp, ++it) {
                    const int s = (int)(it % stages);
                    if (!mbar_wait(smem_u32(&s_full[grp][s]), (uint32_t)((it / stages) & 1))) { alive = false; break; }
                    tc_fence_after_sync();
                    const int k0 = kp * kPanelK;
                    const int nk16 = min(kPanelK, a.k - k0) >> 4;
                    for (int q = 0; q < nk16; ++q) {
                        const uint64_t adesc = make_smem_desc(ring_g + s * kStageBytes + q * 4096, 2048, 128);
                        const uint64_t bdesc = make_smem_desc(basis_addr + ((k0 + 16 * q) >> 3) * 128, 128, b_sbo);
                        mma_bf16_ss(d_tmem, adesc, bdesc, idesc, (kp | q) != 0 ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&s_empty[grp][s]));
                }
                if (alive) mma_commit(smem_u32(&s_tfull[grp]));
            }
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    }

    // ---- teardown ---------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 16) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

bool tc_decode_tc_supported(const tc_ctx *ctx, const DecodeArgs &a)
{
    if (a.c % 16 != 0 || a.k != a.c || a.c > 256) return false;
    if (a.groups != 1 && a.groups != a.k) return false;
    if (a.lut_bits > TC_MAX_CODE_LEN) return false;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, a.chunk_pixels,
                                     ctx->max_smem_optin - 512);
    return l.stages > 0;
}

tc_status tc_launch_decode_tc(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, a.chunk_pixels,
                                     ctx->max_smem_optin - 512);
    if (l.stages == 0) return TC_ERR_UNSUPPORTED;
    void (*kernel)(DecodeArgs) = a.groups != 1 ? decode_tc_kernel<true> : decode_tc_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.total) != cudaSuccess)
        return TC_ERR_CUDA;
    const unsigned int grid = (unsigned int)((a.n_tiles < ctx->sm_count) ? a.n_tiles : ctx->sm_count);
    kernel<<<grid, kThreads, l.total, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
