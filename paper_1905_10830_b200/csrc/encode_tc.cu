// Fused tensor-core encode for bf16 tensors (Section 3: transform, quantiser, VLC).
//
// One persistent block per SM walks tiles of 128 consecutive pixels.  Warp roles:
//   warps 0-3, 4-7  two epilogue groups (alternating tiles): TMEM -> registers, quantise,
//                   code lookup, bit offsets (scan + tile look-back), pack, 128-bit stores
//   warps 8-11      loaders: cp.async NCHW -> shared memory in the MMA's MN-major layout
//   warp 12         one thread issues tcgen05.mma:  D[pixel][coef] = X_tile[pixel][c] * T[coef][c]
// The basis T (bf16, K x C) stays resident in shared memory; the X tile streams through a ring
// of 64-channel panels; the fp32 accumulators are double-buffered in tensor memory so that the
// epilogue of one tile overlaps the loads and MMAs of the next.
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace tcdev;
using namespace sm100;

constexpr int kPanelCh = 64;                      // channels per ring stage
constexpr int kStages = 4;
constexpr int kStageBytes = kPanelCh * TC_TILE_PIXELS * 2;   // 16 KB
constexpr int kLag = 3;                           // cp.async groups kept in flight per loader thread
constexpr int kStagingBytes = 16384;              // packed-bit staging per epilogue group
constexpr int kThreads = 13 * 32;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;

struct SmemLayout {
    uint32_t basis, ring, staging, enc, bias, total;
};

__host__ __device__ inline SmemLayout smem_layout(int c, int k, int enc_entries)
{
    SmemLayout l;
    l.basis = 0;
    l.ring = (uint32_t)(((size_t)k * c * 2 + 1023) & ~(size_t)1023);
    l.staging = l.ring + kStages * kStageBytes;
    l.enc = l.staging + 2 * kStagingBytes;
    l.bias = l.enc + (uint32_t)enc_entries * 4;
    l.total = l.bias + (uint32_t)k * 4;
    return l;
}

__global__ void __launch_bounds__(kThreads, 1) encode_tc_kernel(EncodeArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_full[kStages], s_empty[kStages], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ unsigned int s_warp_sums[2][4];
    __shared__ unsigned long long s_base[2];
    __shared__ int s_write_ok[2];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nsym = 1 << a.bits;
    const bool enc_in_smem = a.groups == 1;
    const SmemLayout L = smem_layout(a.c, a.k, enc_in_smem ? nsym : 0);
    unsigned char *s_basis = smem + L.basis;
    uint32_t *s_enc = reinterpret_cast<uint32_t *>(smem + L.enc);
    float *s_bias = reinterpret_cast<float *>(smem + L.bias);
    const uint32_t ring_addr = smem_u32(smem + L.ring);
    const uint32_t basis_addr = smem_u32(s_basis);
    const int n_panels = (a.c + kPanelCh - 1) / kPanelCh;

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&s_full[s]), 128); mbar_init(smem_u32(&s_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&s_tfull[b]), 1); mbar_init(smem_u32(&s_tempty[b]), 128); }
        mbar_fence_init();
    }
    if (warp == 12) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    // basis -> K-major core-matrix layout: element (j, ch) at (j/8)*sbo + (ch/8)*128 + (j%8)*16 + (ch%8)*2
    {
        const uint32_t sbo = (uint32_t)(a.c / 8) * 128u;
        const int chunks_per_row = a.c / 8;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.basis_bf16);
        for (int i = tid; i < a.k * chunks_per_row; i += kThreads) {
            const int j = i / chunks_per_row, c8 = i - j * chunks_per_row;
            *reinterpret_cast<uint4 *>(s_basis + (j >> 3) * sbo + c8 * 128 + (j & 7) * 16) = __ldg(src + i);
        }
        for (int i = tid; i < a.k; i += kThreads) s_bias[i] = a.enc_bias[i];
        if (enc_in_smem)
            for (int i = tid; i < nsym; i += kThreads) s_enc[i] = a.enc[i];
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    const long long my_tiles = (a.n_tiles > blockIdx.x) ? (a.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp >= 8 && warp < 12) {
        // ================= loaders =================
        const int lw = warp - 8, kk = lane & 7;
        const __nv_bfloat16 *xin = reinterpret_cast<const __nv_bfloat16 *>(a.x);
        int it = 0;
        bool alive = true;
        for (long long tl = 0; tl < my_tiles && alive; ++tl) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            const __nv_bfloat16 *src[2];
            uint32_t dst_off[2], nbytes[2];
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                const int mg = 8 * lw + (lane >> 3) + 4 * g;          // group of 4 pixels
                const long long p0 = tile * TC_TILE_PIXELS + 4 * mg;
                const bool valid = p0 < a.pixels;
                const long long img = valid ? p0 / a.hw : 0;
                const long long s = valid ? p0 - img * a.hw : 0;
                src[g] = xin + img * a.c * (long long)a.hw + s;
                nbytes[g] = valid ? 8u : 0u;
                dst_off[g] = (uint32_t)((mg >> 1) * 128 + kk * 16 + (mg & 1) * 8);
            }
            for (int kp = 0; kp < n_panels; ++kp, ++it) {
                const int s = it % kStages;
                if (!mbar_wait(smem_u32(&s_empty[s]), ((it / kStages) & 1) ^ 1)) { alive = false; break; }
                const int k0 = kp * kPanelCh;
                const int nk8 = min(kPanelCh, a.c - k0) >> 3;
                const uint32_t stage = ring_addr + s * kStageBytes;
                for (int k8 = 0; k8 < nk8; ++k8) {
                    const long long ch_off = (long long)(k0 + 8 * k8 + kk) * a.hw;
#pragma unroll
                    for (int g = 0; g < 2; ++g) cp_async_8(stage + k8 * 2048 + dst_off[g], src[g] + ch_off, nbytes[g]);
                }
                cp_async_commit();
                if (it >= kLag) {
                    cp_async_wait<kLag>();
                    fence_proxy_async_smem();
                    mbar_arrive(smem_u32(&s_full[(it - kLag) % kStages]));
                }
            }
        }
        if (alive) {
            if (it >= 3) { cp_async_wait<2>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 3) % kStages])); }
            if (it >= 2) { cp_async_wait<1>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 2) % kStages])); }
            if (it >= 1) { cp_async_wait<0>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 1) % kStages])); }
        } else {
            cp_async_wait<0>();
            tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else if (warp == 12) {
        // ================= MMA issuer =================
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(TC_TILE_PIXELS, a.k, /*A MN-major*/ true, /*B K-major*/ false);
            const uint32_t b_sbo = (uint32_t)(a.c / 8) * 128u;
            int it = 0;
            bool alive = true;
            for (long long tl = 0; tl < my_tiles && alive; ++tl) {
                const int acc = (int)(tl & 1);
                if (!mbar_wait(smem_u32(&s_tempty[acc]), (uint32_t)(((tl >> 1) & 1) ^ 1))) { alive = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                for (int kp = 0; kp < n_panels; ++kp, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait(smem_u32(&s_full[s]), (it / kStages) & 1)) { alive = false; break; }
                    tc_fence_after_sync();
                    const int k0 = kp * kPanelCh;
                    const int nk16 = min(kPanelCh, a.c - k0) >> 4;
                    for (int q = 0; q < nk16; ++q) {
                        const uint64_t adesc = make_smem_desc(ring_addr + s * kStageBytes + q * 4096, 2048, 128);
                        const uint64_t bdesc = make_smem_desc(basis_addr + ((k0 + 16 * q) >> 3) * 128, 128, b_sbo);
                        mma_bf16_ss(d_tmem, adesc, bdesc, idesc, (kp | q) != 0 ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&s_empty[s]));
                }
                if (alive) mma_commit(smem_u32(&s_tfull[acc]));
            }
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else {
        // ================= epilogue groups =================
        const int grp = warp >> 2;                 // 0 or 1
        const int t = tid & 127;                   // pixel within the tile = TMEM lane
        const int wq = warp & 3;
        uint32_t *stg = reinterpret_cast<uint32_t *>(smem + L.staging + grp * kStagingBytes);
        const uint32_t *enc = enc_in_smem ? s_enc : a.enc;
        const float inv_step = (float)(1.0 / a.step);
        const int top = nsym - 1;
        const int bar_id = 1 + grp;
        bool alive = true;
        for (long long tl = grp; tl < my_tiles && alive; tl += 2) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            const long long p = tile * TC_TILE_PIXELS + t;
            const bool valid = p < a.pixels;
            if (!mbar_wait(smem_u32(&s_tfull[grp]), (uint32_t)((tl >> 1) & 1))) { alive = false; break; }
            tc_fence_after_sync();
            const uint32_t trow = tmem_base + grp * kAccCols + ((uint32_t)(wq * 32) << 16);

            // pass 1: code lengths
            unsigned int my_bits = 0;
            for (int c0 = 0; c0 < a.k; c0 += 32) {
                uint32_t r[32];
                const int n = min(32, a.k - c0);
                if (n == 32) tmem_ld_32x32b_x32(trow + c0, r);
                else {
                    uint32_t r16[16];
                    tmem_ld_32x32b_x16(trow + c0, r16);
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = r16[i];
                }
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (i < n) {
                        const int j = c0 + i;
                        int q = __float2int_rn(fmaf(__uint_as_float(r[i]), inv_step, s_bias[j]));
                        q = max(0, min(q, top));
                        my_bits += enc[(a.groups == 1 ? 0 : j * nsym) + q] & 0xffu;
                    }
                }
            }
            if (!valid) my_bits = 0;
            unsigned int tile_bits;
            const unsigned int my_off = group_exclusive_scan_128(my_bits, s_warp_sums[grp], t, bar_id, tile_bits);
            const unsigned long long padded = ((unsigned long long)tile_bits + 127ull) & ~127ull;
            if (t == 0) lookback_publish(a.tile_state, tile, padded);
            const bool staged = padded <= (unsigned long long)kStagingBytes * 8ull;

            uint32_t *out_words = stg;
            unsigned long long out_bit = my_off;
            if (staged) {
                uint4 *z = reinterpret_cast<uint4 *>(stg);
                for (unsigned int i = t; i < (unsigned int)(padded >> 7); i += 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
            } else {
                // rare: the tile does not fit the staging buffer -> resolve its position first and
                // pack straight into (zeroed) global memory
                if (wq == 0) {
                    bool ok;
                    const unsigned long long base = lookback_resolve(a.tile_state, tile, padded, a.status, ok);
                    if (lane == 0) {
                        const bool fits = base + padded <= a.capacity_bits;
                        if (ok && !fits) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
                        s_base[grp] = base;
                        s_write_ok[grp] = (ok && fits) ? 1 : 0;
                    }
                }
                named_bar_sync(bar_id, 128);
                if (s_write_ok[grp]) {
                    uint4 *z = reinterpret_cast<uint4 *>(a.stream + (s_base[grp] >> 5));
                    for (unsigned int i = t; i < (unsigned int)(padded >> 7); i += 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
                }
                out_words = a.stream;
                out_bit = s_base[grp] + my_off;
            }
            named_bar_sync(bar_id, 128);

            // pass 2: quantise again, look up codes, pack
            const bool do_pack = valid && (staged || s_write_ok[grp]);
            BitWriter w;
            w.init(out_words, out_bit);
            for (int c0 = 0; c0 < a.k; c0 += 32) {
                uint32_t r[32];
                const int n = min(32, a.k - c0);
                if (n == 32) tmem_ld_32x32b_x32(trow + c0, r);
                else {
                    uint32_t r16[16];
                    tmem_ld_32x32b_x16(trow + c0, r16);
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = r16[i];
                }
                tmem_ld_wait();
                if (do_pack) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (i < n) {
                            const int j = c0 + i;
                            const float accv = __uint_as_float(r[i]);
                            int q = __float2int_rn(fmaf(accv, inv_step, s_bias[j]));
                            q = max(0, min(q, top));
                            const uint32_t e = enc[(a.groups == 1 ? 0 : j * nsym) + q];
                            w.put(e >> 8, (int)(e & 0xffu));
                            if (a.dbg_coef) a.dbg_coef[p * a.k + j] = accv - a.tmu32[j];
                            if (a.dbg_sym) a.dbg_sym[p * a.k + j] = (uint8_t)q;
                        }
                    }
                }
            }
            if (do_pack) w.finish();
            // the accumulator buffer is free for the tile after next
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&s_tempty[grp]));

            if (staged) {
                if (wq == 0) {
                    bool ok;
                    const unsigned long long base = lookback_resolve(a.tile_state, tile, padded, a.status, ok);
                    if (lane == 0) {
                        const bool fits = base + padded <= a.capacity_bits;
                        if (ok && !fits) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
                        s_base[grp] = base;
                        s_write_ok[grp] = (ok && fits) ? 1 : 0;
                    }
                }
                named_bar_sync(bar_id, 128);      // staging complete, base known
                if (s_write_ok[grp]) {
                    uint4 *dst = reinterpret_cast<uint4 *>(a.stream + (s_base[grp] >> 5));
                    const uint4 *srcv = reinterpret_cast<const uint4 *>(stg);
                    for (unsigned int i = t; i < (unsigned int)(padded >> 7); i += 128) dst[i] = srcv[i];
                }
            }
            const unsigned long long base = s_base[grp];
            if (t == 0) {
                a.tile_off[tile] = base;
                if (tile == a.n_tiles - 1) a.tile_off[a.n_tiles] = base + padded;
            }
            if (valid && (p % a.chunk_pixels) == 0) a.chunk_off[p / a.chunk_pixels] = my_off;
            named_bar_sync(bar_id, 128);          // staging and s_base may be reused
        }
        if (!alive && t == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    }

    // ---- teardown ---------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

bool tc_encode_tc_supported(const tc_ctx *ctx, const EncodeArgs &a)
{
    if (a.c % 16 != 0 || a.k != a.c || a.c > 256 || a.hw % 4 != 0) return false;
    if (a.groups != 1 && a.groups != a.k) return false;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.bits) : 0);
    return (int)l.total + 512 <= ctx->max_smem_optin;
}

tc_status tc_launch_encode_tc(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.bits) : 0);
    if (cudaFuncSetAttribute(encode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.total) != cudaSuccess)
        return TC_ERR_CUDA;
    const unsigned int grid = (unsigned int)((a.n_tiles < ctx->sm_count) ? a.n_tiles : ctx->sm_count);
    EncodeArgs args = a;
    void *params[] = {&args};
    // cooperative launch: the grid must be co-resident, which is what makes the look-back safe
    if (cudaLaunchCooperativeKernel((void *)encode_tc_kernel, dim3(grid), dim3(kThreads), params, l.total, s) != cudaSuccess) {
        cudaGetLastError();
        return TC_ERR_CUDA;
    }
    return TC_OK;
}
