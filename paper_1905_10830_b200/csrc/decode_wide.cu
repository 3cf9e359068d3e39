// Tensor-core decode for bf16 tensors of more than 256 channels (Section 3: VLD, inverse
// quantiser, inverse transform), where neither the transposed basis nor a double-buffered
// accumulator for every channel fits on chip.
//
// One persistent block per SM walks work items of NP pixels (two at a time, on two VLD groups,
// up to 256 channels, where the accumulators of two items fit tensor memory): a whole tile of 128 pixels up to
// 512 channels, half a tile beyond (the accumulators of all channels, NP columns per block of
// 128 channels, fill tensor memory exactly).  Per item:
//   warps 0-7     VLD: one thread per chunk walks the bit stream (the item's segment staged in
//                 shared memory when it fits, table-driven canonical Huffman) and writes the symbols minus the centre symbol, as exact
//                 bf16 integers, into the K-major B operand, which holds all K coefficients of
//                 the item's pixels (2 K NP bytes)
//   warps 16-19   loaders: the transposed basis streams from L2 through a ring of
//                 128-channel x 64-coefficient panels (one tiled TMA copy with 128-byte swizzle
//                 per panel, issued by one thread; cp.async copies without a tensor map)
//   warp 20       one thread issues tcgen05.mma:  D[c][pixel] += T[j][c] * (Q[pixel][j] - center)
//   warps 8-15    epilogue: TMEM -> registers (lane = channel), x_hat = step * acc + bias_c,
//                 round to bf16, NCHW stores; runs while the VLD warps decode the next item
// Dequantisation is folded as in the resident-basis kernel:
// bias_c = mu_c + (lo + center * step) * sum_j T[j][c].
#include <cstring>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace tcdev;
using namespace sm100;

constexpr int kVldThreads = 256;
// Warp roles for G VLD groups (G = 1: wide layers; G = 2: layers of up to 256 channels, where two
// work items are in flight, each group with its own B operand and accumulator): VLD warps
// 0 .. 8G-1, eight epilogue warps, loader warps (four; one when only TMA copies are issued), one
// MMA warp.
template <int G>
struct Roles {
    static constexpr int kEpiWarp0 = 8 * G;
    static constexpr int kLoaderWarp0 = kEpiWarp0 + 8;
    static constexpr int kLoaderWarps = G == 2 ? 1 : 4;
    static constexpr int kMmaWarp = kLoaderWarp0 + kLoaderWarps;
    static constexpr int kThreads = (kMmaWarp + 1) * 32;
};
constexpr int kTmemCols = 512;
constexpr int kPanelK = 64;                                   // coefficients per ring stage
constexpr int kStageBytes = 128 * kPanelK * 2;                // 16 KB: 128 channels x 64 coefficients
constexpr int kMaxStages = 6;
constexpr int kLag = 2;
constexpr int kVldBar = 1;
constexpr int kMaxTileChunks = 512;

// Epilogue transpose block of one warp: 32 channel rows of 32 pixels (64 bytes) with 16 bytes
// of padding, which keeps both the 16-byte row writes and the 8-byte reads spread over the banks.
constexpr int kTrRowBytes = 80;
constexpr int kTrWarpBytes = 32 * kTrRowBytes;
constexpr int kSegBytes = 16384;                              // staged stream segment of one work item: at least this,
constexpr int kSegBytesMax = 32768;                           // up to this where four ring stages still fit
constexpr int kSegSlack = 32;                                 // the reader's window may look two words past the end

struct SmemLayout {
    uint32_t ring, bop, bop_bytes, lut, start, start_bytes, tbuf, seg, seg_stride, total;
    int stages, np;
    uint32_t seg_bytes;                                       // size of the segment buffer (0: none)
    bool staged;                                              // room for the segment buffer beside at least three stages
};

__host__ __device__ inline SmemLayout smem_layout(int c, int k, int lut_entries, int budget, int groups = 1, int item_pixels = 0)
{
    SmemLayout l;
    l.np = item_pixels ? item_pixels : ((c + 127) / 128 <= 4) ? 128 : 64;
    l.bop_bytes = 2u * (uint32_t)k * (uint32_t)l.np;
    l.start_bytes = (kMaxTileChunks + 8) * 4u;
    const uint32_t fixed = (uint32_t)groups * (l.bop_bytes + l.start_bytes) + (uint32_t)lut_entries * 4u + 16u + 8u * kTrWarpBytes;
    // the largest segment buffer (per group) that leaves enough ring stages: 32 KB beside four
    // stages, else 16 KB or 8 KB beside three (two with two groups)
    l.seg_bytes = 0;
    int stages = 0;
    const int cands[3] = {kSegBytesMax, kSegBytes, kSegBytes / 2};
    for (int i = 0; i < 3; ++i) {
        const int st = (int)(((long long)budget - (long long)fixed - (long long)groups * (cands[i] + kSegSlack)) / kStageBytes);
        const int need = i == 0 ? 4 : (groups == 2 ? 2 : 3);
        if (st >= need) { l.seg_bytes = (uint32_t)cands[i]; stages = st; break; }
    }
    l.staged = l.seg_bytes != 0;
    if (!l.staged) stages = (int)(((long long)budget - (long long)fixed) / kStageBytes);
    if (stages > kMaxStages) stages = kMaxStages;
    l.stages = stages < 2 ? 0 : stages;
    l.ring = 0;
    l.bop = (uint32_t)(l.stages * kStageBytes);
    l.lut = l.bop + (uint32_t)groups * l.bop_bytes;
    l.start = l.lut + (uint32_t)lut_entries * 4u;
    l.tbuf = (l.start + (uint32_t)groups * l.start_bytes + 15u) & ~15u;      // eight warp-private transpose blocks (epilogue)
    l.seg = l.tbuf + 8u * kTrWarpBytes;
    l.seg_stride = l.seg_bytes + (uint32_t)kSegSlack;
    l.total = l.seg + (l.staged ? (uint32_t)groups * l.seg_stride : 0u);
    return l;
}

// kTma: the panels of the transposed basis arrive by tiled TMA copies (one instruction per stage,
// 128-byte swizzle) instead of 1024 cp.async copies; `tmap` is then its tensor map.
template <bool kPerChannel, bool kTma, int G>
__global__ void __launch_bounds__(Roles<G>::kThreads, 1) decode_wide_kernel(DecodeArgs a, const __grid_constant__ CUtensorMap tmap)
{
    constexpr int kEpiWarp0 = Roles<G>::kEpiWarp0, kLoaderWarp0 = Roles<G>::kLoaderWarp0, kMmaWarp = Roles<G>::kMmaWarp;
    constexpr int kThreads = Roles<G>::kThreads;
    static_assert(G == 1 || kTma, "two groups leave one loader warp: the basis must come by TMA");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // the swizzled panels want their 1 KB atoms aligned; the ring starts the buffer
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ __align__(8) unsigned long long s_full[kMaxStages], s_empty[kMaxStages];
    __shared__ __align__(8) unsigned long long s_bfull[2], s_bfree[2], s_tfull[2], s_tempty[2];   // per group
    __shared__ uint32_t s_tmem_base;
    __shared__ unsigned int s_wsum[2][8];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lut_size = 1 << a.lut_bits;
    const SmemLayout L = smem_layout(a.c, a.k, kPerChannel ? 0 : lut_size, a.smem_budget, G, a.item_pixels);
    const int stages = L.stages, NP = L.np;
    const uint32_t ring_addr = smem_u32(smem + L.ring);
    uint32_t *s_lut = reinterpret_cast<uint32_t *>(smem + L.lut);
    const int n_cblocks = (a.c + 127) / 128;                  // blocks of 128 channels
    const int n_kpanels = (a.k + kPanelK - 1) / kPanelK;
    const int items_per_tile = TC_TILE_PIXELS / NP;
    const long long n_items = a.n_tiles * items_per_tile;
    const long long my_items = (n_items > blockIdx.x) ? (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(smem_u32(&s_full[s]), kTma ? 1 : 128); mbar_init(smem_u32(&s_empty[s]), 1); }
        for (int g = 0; g < 2; ++g) {
            mbar_init(smem_u32(&s_bfull[g]), kVldThreads);
            mbar_init(smem_u32(&s_bfree[g]), 1);
            mbar_init(smem_u32(&s_tfull[g]), 1);
            mbar_init(smem_u32(&s_tempty[g]), 256);
        }
        mbar_fence_init();
    }
    if (warp == kMmaWarp) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    if (!kPerChannel)
        for (int i = tid; i < lut_size; i += kThreads) {
            // per-layer table: bf16(symbol - center) << 16 | code length
            const uint32_t e = a.lut32[i];
            const float f = (float)((int)((e >> 8) & 0xffu) - a.center);
            s_lut[i] = (__float_as_uint(f) & 0xffff0000u) | (e & 0xffu);
        }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    if (warp < kEpiWarp0) {
        // ================= VLD =================
        const int grp = warp >> 3, vw = warp & 7;            // group, warp within the group
        const int t = tid & 255;
        const uint32_t bop_addr = smem_u32(smem + L.bop) + (uint32_t)grp * L.bop_bytes;
        unsigned int *s_start = reinterpret_cast<unsigned int *>(smem + L.start + grp * L.start_bytes);   // start of every chunk of the tile
        unsigned char *seg_ptr = smem + L.seg + grp * L.seg_stride;
        const int vld_bar = kVldBar + grp;
        const int S = a.splits, cp = a.chunk_pixels;
        const int chunks_per_tile = S * TC_TILE_PIXELS / cp;  // at most 512
        const int k_sub = a.k / S;
        const int item_chunks = S * NP / cp;
        const int pix_chunks = NP / cp;                       // chunks of one run of coefficients in an item
        const uint32_t row_bytes = (uint32_t)NP * 16u;        // one group of 8 coefficients of all the item's pixels
        bool alive = true;
        for (long long n = grp; n < my_items && alive; n += G) {
            const long long li = n / G;                       // items this group has taken before
            const long long item = blockIdx.x + n * gridDim.x;
            const long long tile = item / items_per_tile;
            const int h = (int)(item - tile * items_per_tile);
            // chunk lengths of the tile -> start positions (exclusive scan over 2 x 256 values)
            const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
            const bool tile_ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
            unsigned int l0 = 0, l1 = 0;
            {
                const long long ch = tile * chunks_per_tile + 2 * t;
                if (2 * t < chunks_per_tile && ch < a.n_chunks) l0 = a.chunk_len[ch];
                if (2 * t + 1 < chunks_per_tile && ch + 1 < a.n_chunks) l1 = a.chunk_len[ch + 1];
            }
            unsigned int inc = l0 + l1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += up;
            }
            // the B operand and the start positions are free once the previous item's MMAs are done
            if (!mbar_wait(smem_u32(&s_bfree[grp]), (uint32_t)((li & 1) ^ 1))) { alive = false; break; }
            if (lane == 31) s_wsum[grp][vw] = inc;
            named_bar_sync(vld_bar, kVldThreads);
            unsigned int before = 0, tile_total = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const unsigned int sw = s_wsum[grp][w];
                if (w < vw) before += sw;
                tile_total += sw;
            }
            const unsigned int excl = before + inc - (l0 + l1);
            if (2 * t < kMaxTileChunks) { s_start[2 * t] = excl; s_start[2 * t + 1] = excl + l0; }
            named_bar_sync(vld_bar, kVldThreads);
            bool bad = !tile_ok || (unsigned long long)tile_total > end - base;

            // the item's part of the tile's segment, staged in shared memory when it fits: the
            // readers' refills become shared-memory loads instead of dependent global loads
            const int ci_first = (h * NP / cp) * S, ci_end = ((h + 1) * NP / cp) * S;
            const unsigned int seg_lo = s_start[ci_first];
            const unsigned int seg_hi = ci_end < chunks_per_tile ? s_start[ci_end] : tile_total;
            const unsigned int byte_lo = (seg_lo >> 3) & ~15u, byte_hi = ((seg_hi + 127u) >> 7) << 4;
            const bool staged = L.staged && !bad && byte_hi - byte_lo <= L.seg_bytes;
            if (staged) {
                const unsigned char *src = reinterpret_cast<const unsigned char *>(a.stream) + (base >> 3) + byte_lo;
                const uint32_t dst = smem_u32(seg_ptr);
                for (unsigned int i = (unsigned int)t; i < ((byte_hi - byte_lo) >> 4); i += kVldThreads)
                    cp_async_16(dst + i * 16u, src + (size_t)i * 16u, 16u);
            }
            cp_async_commit();
            cp_async_wait<0>();
            named_bar_sync(vld_bar, kVldThreads);       // every thread's part of the segment has landed
            const uint32_t *seg_words = reinterpret_cast<const uint32_t *>(seg_ptr);

            auto decode_chunks = [&](auto &r) {
            for (int u = t; u < item_chunks && !bad; u += kVldThreads) {
                // chunk u of the item: run `sub` of the coefficients of pixel(s) r0 ...
                const int sub = u / pix_chunks, cidx = u - sub * pix_chunks;
                const int r0 = cidx * cp;                                     // first pixel inside the item
                const int ci = (h * NP + r0) / cp * S + sub;                  // chunk inside the tile (S > 1 only with cp = 1)
                const long long p0 = tile * TC_TILE_PIXELS + h * NP + r0;
                if (p0 >= a.pixels) continue;
                const int n_pix = (int)min((long long)cp, a.pixels - p0);
                const unsigned int start = s_start[ci], want = (ci + 1 < chunks_per_tile ? s_start[ci + 1] : tile_total) - start;
                if (staged) r.init(seg_words, (unsigned long long)start - 8ull * byte_lo, 8ull * (byte_hi - byte_lo));
                else r.init(a.stream, base + start, end);
                unsigned int used = 0;
                const int k_first = sub * k_sub;
                for (int pp = 0; pp < n_pix; ++pp) {
                    const uint32_t dst = bop_addr + (uint32_t)(k_first >> 3) * row_bytes + (uint32_t)(r0 + pp) * 16u;
                    for (int k8 = 0; k8 < (k_sub >> 3); ++k8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            r.refill();
                            uint32_t v0, v1, len0, len1;
                            if constexpr (kPerChannel) {
                                const int j = k_first + k8 * 8 + 2 * i;
                                const uint32_t e0 = __ldg(a.lut32 + (size_t)j * lut_size + r.peek(a.lut_bits));
                                len0 = e0 & 0xffu;
                                r.skip((int)len0);
                                const uint32_t e1 = __ldg(a.lut32 + (size_t)(j + 1) * lut_size + r.peek(a.lut_bits));
                                len1 = e1 & 0xffu;
                                r.skip((int)len1);
                                v0 = __float_as_uint((float)((int)((e0 >> 8) & 0xffu) - a.center));
                                v1 = __float_as_uint((float)((int)((e1 >> 8) & 0xffu) - a.center));
                            } else {
                                v0 = s_lut[r.peek(a.lut_bits)];
                                len0 = v0 & 0xffu;
                                r.skip((int)len0);
                                v1 = s_lut[r.peek(a.lut_bits)];
                                len1 = v1 & 0xffu;
                                r.skip((int)len1);
                            }
                            used += len0 + len1;
                            pk[i] = __byte_perm(v0, v1, 0x7632);
                        }
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)k8 * row_bytes), "r"(pk[0]),
                                     "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    }
                }
                // a chunk must end exactly where its recorded length says
                if (used != want) bad = true;
            }
            };
            if (staged) { WindowReaderT<true> r; decode_chunks(r); }
            else { WindowReader r; decode_chunks(r); }
            if (bad) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
            // the writes become visible to the tensor core's proxy, then the operand is handed over
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&s_bfull[grp]));
        }
        if (!alive && t == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else if (warp < kLoaderWarp0) {
        // ================= epilogue =================
        const int ew = warp - kEpiWarp0;
        const int set = ew >> 2, wq = ew & 3;                // two sets of four warps take alternate channel blocks
        const float step = (float)(a.step * a.basis_scale);  // the operand holds basis / basis_scale
        const float floor_v = a.relu ? 0.f : __int_as_float((int)0xff800000u);      // the layer's non-linearity, when it follows the decoder
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.xhat);
        const bool vec = (a.hw & 3) == 0 && ((uintptr_t)a.xhat & 7u) == 0;                    // four aligned pixels lie inside one image, 8-byte aligned
        const long long img_stride = (long long)a.c * a.hw;
        const uint32_t tb = smem_u32(smem + L.tbuf) + (uint32_t)ew * kTrWarpBytes;
        const uint32_t tb_wr = tb + (uint32_t)lane * kTrRowBytes;                              // this thread's channel row
        const uint32_t tb_rd = tb + (uint32_t)(lane >> 3) * kTrRowBytes + (uint32_t)(lane & 7) * 8u;
        bool alive = true;
        for (long long n = 0; n < my_items && alive; ++n) {
            const long long item = blockIdx.x + n * gridDim.x;
            const long long p_first = item * NP;
            const long long left = a.pixels - p_first;
            const int n_valid = (int)(left < (long long)NP ? (left < 0 ? 0 : left) : (long long)NP);
            const long long img0 = left > 0 ? p_first / a.hw : 0;
            const int s0 = left > 0 ? (int)(p_first - img0 * a.hw) : 0;
            const int grp = (int)(n % G);
            if (!mbar_wait(smem_u32(&s_tfull[grp]), (uint32_t)((n / G) & 1))) { alive = false; break; }
            tc_fence_after_sync();
            for (int blk = set; blk < n_cblocks; blk += 2) {
                const int ch = blk * 128 + wq * 32 + lane;
                const bool ch_ok = ch < a.c;
                const float bias = ch_ok ? __ldg(a.dec_bias + ch) : 0.f;
                const uint32_t trow = tmem_base + (uint32_t)(grp * 256 + blk * NP) + ((uint32_t)(wq * 32) << 16);
                if (vec) {
                    // 32 pixels at a time: the thread rounds its channel's values and writes them as one
                    // 64-byte row of the warp's block; the warp then reads the block back four rows per
                    // instruction, so that every channel row leaves as 64 contiguous bytes
                    const int pgrp = lane & 7, r_sub = lane >> 3;
                    const int ch_base = blk * 128 + wq * 32;
                    const long long pg = p_first + 4 * pgrp;
                    long long img = pg < a.pixels ? pg / a.hw : 0;
                    int sp = pg < a.pixels ? (int)(pg - img * a.hw) : 0;
                    for (int c0 = 0; c0 < NP; c0 += 32) {
                        uint32_t r[32];
                        {
                            uint32_t r16[16];
                            tmem_ld_32x32b_x16(trow + c0, r16);
#pragma unroll
                            for (int i = 0; i < 16; ++i) r[i] = r16[i];
                            tmem_ld_32x32b_x16(trow + c0 + 16, r16);
#pragma unroll
                            for (int i = 0; i < 16; ++i) r[16 + i] = r16[i];
                        }
                        tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint32_t h2[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(fmaxf(fmaf(__uint_as_float(r[8 * q + 2 * i]), step, bias), floor_v),
                                                                               fmaxf(fmaf(__uint_as_float(r[8 * q + 2 * i + 1]), step, bias), floor_v));
                                h2[i] = *reinterpret_cast<const uint32_t *>(&h);
                            }
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(tb_wr + q * 16), "r"(h2[0]), "r"(h2[1]),
                                         "r"(h2[2]), "r"(h2[3]) : "memory");
                        }
                        __syncwarp();
                        const bool px_ok = c0 + 4 * pgrp < n_valid;
                        __nv_bfloat16 *row_ptr = out + img * img_stride + (long long)(ch_base + r_sub) * a.hw + sp;
#pragma unroll
                        for (int it = 0; it < 8; ++it) {
                            uint32_t lo2, hi2;
                            asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(lo2), "=r"(hi2) : "r"(tb_rd + it * 4 * kTrRowBytes));
                            if (px_ok && ch_base + 4 * it + r_sub < a.c)
                                *reinterpret_cast<uint2 *>(row_ptr + (long long)(4 * it) * a.hw) = make_uint2(lo2, hi2);
                        }
                        sp += 32;
                        while (sp >= a.hw) { sp -= a.hw; ++img; }
                        __syncwarp();                                   // the block may be overwritten
                    }
                } else {
                    int s = s0;
                    __nv_bfloat16 *dst = out + img0 * img_stride + (long long)(ch_ok ? ch : 0) * a.hw + s;
                    for (int c0 = 0; c0 < NP; c0 += 16) {
                        uint32_t r[16];
                        tmem_ld_32x32b_x16(trow + c0, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const __nv_bfloat16 hv = __float2bfloat16_rn(fmaxf(fmaf(__uint_as_float(r[i]), step, bias), floor_v));
                            if (ch_ok && c0 + i < n_valid) *dst = hv;
                            s += 1;
                            const bool wrap = s == a.hw;
                            dst += wrap ? 1 + img_stride - a.hw : 1;
                            s = wrap ? 0 : s;
                        }
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&s_tempty[grp]));
        }
        if (!alive && lane == 0 && ew == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else if (warp < kMmaWarp) {
        // ================= loaders =================
        const int lt = tid - kLoaderWarp0 * 32;               // 0..127
        int it = 0;
        bool alive = true;
        for (long long n = 0; n < my_items && alive; ++n) {
            if (kTma && lt != 0) break;                       // one thread asks for the boxes
            for (int jp = 0; jp < n_kpanels && alive; ++jp) {
                const int j0 = jp * kPanelK;
                const int nk8 = min(kPanelK, a.k - j0) >> 3;
                for (int blk = 0; blk < n_cblocks; ++blk, ++it) {
                    const int s = it % stages;
                    if (!mbar_wait(smem_u32(&s_empty[s]), ((it / stages) & 1) ^ 1)) { alive = false; break; }
                    const uint32_t stage = ring_addr + s * kStageBytes;
                    if constexpr (kTma) {
                        // box of 128 channels x 64 coefficients at (coefficient j0, channel blk * 128); rows
                        // and columns past the matrix arrive as zeros and count towards the bytes
                        mbar_arrive_expect_tx(smem_u32(&s_full[s]), (uint32_t)kStageBytes);
                        tma_load_2d(stage, &tmap, j0, blk * 128, smem_u32(&s_full[s]));
                        continue;
                    }
                    // transposed basis rows (channels) blk * 128 ..., coefficients j0 ...: K-major core
                    // matrices (row / 8) * 1024 + (j / 8) * 128 + (row % 8) * 16; rows past C are zero
                    for (int i = lt; i < 128 * 8; i += 128) {
                        const int row = i >> 3, j8 = i & 7;
                        const int ch = blk * 128 + row;
                        const bool ok = ch < a.c && j8 < nk8;
                        cp_async_16(stage + (row >> 3) * 1024 + j8 * 128 + (row & 7) * 16,
                                    a.basis_t_bf16 + (ok ? (long long)ch * a.k + j0 + j8 * 8 : 0), ok ? 16u : 0u);
                    }
                    cp_async_commit();
                    if (it >= kLag) {
                        cp_async_wait<kLag>();
                        fence_proxy_async_smem();
                        mbar_arrive(smem_u32(&s_full[(it - kLag) % stages]));
                    }
                }
            }
        }
        if (kTma) {
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        } else if (alive) {
            if (it >= 2) { cp_async_wait<1>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 2) % stages])); }
            if (it >= 1) { cp_async_wait<0>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 1) % stages])); }
        } else {
            cp_async_wait<0>();
            tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else {
        // ================= MMA issuer =================
        if (lane == 0) {
            // A = transposed basis (128 channels per instruction), B = the decoded symbols of NP pixels
            const uint32_t idesc = make_idesc_bf16(128, NP, /*A K-major*/ false, /*B K-major*/ false);
            const uint32_t b_lbo = (uint32_t)NP * 16u;
            int it = 0;
            bool alive = true;
            for (long long n = 0; n < my_items && alive; ++n) {
                const int grp = (int)(n % G);
                const uint32_t par = (uint32_t)((n / G) & 1);
                const uint32_t bop_addr = smem_u32(smem + L.bop) + (uint32_t)grp * L.bop_bytes;
                if (!mbar_wait(smem_u32(&s_bfull[grp]), par)) { alive = false; break; }
                if (!mbar_wait(smem_u32(&s_tempty[grp]), par ^ 1u)) { alive = false; break; }
                fence_proxy_async_smem();
                tc_fence_after_sync();
                for (int jp = 0; jp < n_kpanels && alive; ++jp) {
                    const int j0 = jp * kPanelK;
                    const int nk16 = min(kPanelK, a.k - j0) >> 4;
                    for (int blk = 0; blk < n_cblocks; ++blk, ++it) {
                        const int s = it % stages;
                        if (!mbar_wait(smem_u32(&s_full[s]), (it / stages) & 1)) { alive = false; break; }
                        tc_fence_after_sync();
                        const uint32_t stage = ring_addr + s * kStageBytes;
                        for (int q = 0; q < nk16; ++q) {
                            const uint64_t adesc = kTma ? make_smem_desc_sw128(stage + q * 32, 1024) : make_smem_desc(stage + q * 256, 128, 1024);
                            const uint64_t bdesc = make_smem_desc(bop_addr + (uint32_t)((j0 + 16 * q) >> 3) * b_lbo, b_lbo, 128);
                            mma_bf16_ss(tmem_base + (uint32_t)(grp * 256 + blk * NP), adesc, bdesc, idesc, (jp | q) != 0 ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&s_empty[s]));
                    }
                }
                if (alive) {
                    mma_commit(smem_u32(&s_tfull[grp]));
                    mma_commit(smem_u32(&s_bfree[grp]));
                }
            }
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    }

    // ---- teardown ---------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

// Two VLD groups (two work items in flight, each with its own B operand and accumulator) where
// the accumulators of two items fit tensor memory, i.e. up to 256 channels, the basis comes by
// TMA, and shared memory holds both operands beside two ring stages and the segment buffers.
static int decode_wide_groups(const tc_ctx *ctx, const DecodeArgs &a)
{
    if (!a.basis_t_map || a.c > 256) return 1;
    const SmemLayout l2 = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, ctx->max_smem_optin - 2048, 2);
    if (!(l2.stages >= 2 && l2.staged)) return 1;
    // A stream the caller says is dense (mean tile size above the two-group segment buffers) is better
    // served by one group with a large segment buffer than by two that read it from global memory.
    if (a.mean_tile_bytes > 0 && (unsigned long long)a.mean_tile_bytes > l2.seg_bytes) return 1;
    return 2;
}

bool tc_decode_wide_supported(const tc_ctx *ctx, const DecodeArgs &a)
{
    if (a.c % 16 != 0 || a.k % 16 != 0 || a.k < 16 || a.k > a.c || a.c > TC_MAX_C) return false;
    if (a.splits != 1 && a.splits != 2 && a.splits != 4) return false;
    if (a.splits > 1 && (a.chunk_pixels != 1 || a.k % a.splits != 0 || (a.k / a.splits) % 8 != 0)) return false;
    if (a.groups != 1 && a.groups != a.k) return false;
    if (a.lut_bits > TC_MAX_CODE_LEN) return false;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, ctx->max_smem_optin - 2048,
                                     decode_wide_groups(ctx, a));
    if (l.stages < 2) return false;
    return a.chunk_pixels <= l.np;                            // a chunk lies inside one work item
}

// Bytes of a tile's stream segment this kernel can stage in shared memory (0: none).
size_t tc_decode_wide_staging_bytes(const tc_ctx *ctx, const DecodeArgs &a)
{
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, ctx->max_smem_optin - 2048,
                                     decode_wide_groups(ctx, a));
    return (l.stages >= 2 && l.staged) ? (size_t)l.seg_bytes * (TC_TILE_PIXELS / l.np) : 0u;
}

tc_status tc_launch_decode_wide(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    DecodeArgs args = a;
    args.smem_budget = ctx->max_smem_optin - 2048;            // leaves room for the static shared variables and the alignment
    const int groups = decode_wide_groups(ctx, a);
    SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, args.smem_budget, groups);
    if (l.stages < 2) return TC_ERR_UNSUPPORTED;
    // A tensor of few tiles leaves most SMs without a work item: smaller items (64 or 32 pixels, as
    // long as a chunk still lies inside one) spread it over more of them.  Every item streams the
    // whole basis, so this only pays while there are fewer items than SMs.
    args.item_pixels = 0;
    if (groups == 1) {
        int np = l.np;
        while (np > 32 && np / 2 >= a.chunk_pixels && a.n_tiles * (TC_TILE_PIXELS / np) * 2 <= ctx->sm_count) np /= 2;
        if (np != l.np) {
            const SmemLayout l2 = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, args.smem_budget, groups, np);
            if (l2.stages >= 2) { l = l2; args.item_pixels = np; }
        }
    }
    const bool tma = a.basis_t_map != nullptr, pc = a.groups != 1;
    void (*kernel)(DecodeArgs, const CUtensorMap) =
        groups == 2 ? (pc ? decode_wide_kernel<true, true, 2> : decode_wide_kernel<false, true, 2>)
        : tma       ? (pc ? decode_wide_kernel<true, true, 1> : decode_wide_kernel<false, true, 1>)
                    : (pc ? decode_wide_kernel<true, false, 1> : decode_wide_kernel<false, false, 1>);
    const int threads = groups == 2 ? Roles<2>::kThreads : Roles<1>::kThreads;
    const size_t smem_bytes = (size_t)l.total + 1024;         // room to align the buffer to 1 KB
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
        return TC_ERR_CUDA;
    const long long n_items = a.n_tiles * (TC_TILE_PIXELS / l.np);
    const unsigned int grid = (unsigned int)((n_items < ctx->sm_count) ? n_items : ctx->sm_count);
    CUtensorMap map_arg;
    if (tma) map_arg = *a.basis_t_map;
    else memset(&map_arg, 0, sizeof(map_arg));
    kernel<<<grid, threads, smem_bytes, s>>>(args, map_arg);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
