// Tensor-core encode for bf16 tensors the resident-basis kernel does not take: up to 1024
// channels (the basis no longer fits shared memory) and map sizes whose rows are not 8-byte
// aligned (7 x 7).  Section 3: transform, quantiser, VLC.
//
// One persistent block per SM walks tiles of 128 consecutive pixels.  The coefficients of a
// tile are produced in blocks of up to 256 (one accumulator of tensor memory each, two
// accumulators in flight); for every block the pixels' channels stream through a ring of
// 32-channel panels together with the matching 256 x 32 piece of the basis, both read from L2
// (the basis piece as one tiled TMA copy with 64-byte swizzle, the pixels by the loader warps).
//   warps 0-15    epilogue: four warps per quarter of a block's coefficients (a warp reads its own
//                 32 lanes of tensor memory).  Pass 1 (per block): TMEM -> registers, quantise, code length,
//                 symbols parked in shared memory (one byte each, K x 128 per tile), bits added up
//                 per run of coefficients.  Then: bit offsets (scan over the pixels, tile
//                 look-back), chunk lengths.  Pass 2: codes of the parked symbols packed straight
//                 into the (zeroed) stream words.
//   warps 16-23   loaders: cp.async (or, for unaligned rows, plain 2-byte loads) into the MMA's
//                 shared-memory layouts
//   warp 24       one thread issues tcgen05.mma:  D[pixel][coef] = X[pixel][c] * T[coef][c]
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace tcdev;
using namespace sm100;

constexpr int kPanelCh = 32;                                  // channels per ring stage
constexpr int kBlockCoef = 256;                               // coefficients per accumulator
constexpr int kStageA = kPanelCh * TC_TILE_PIXELS * 2;        // 8 KB: pixels x channels
constexpr int kStageB = kBlockCoef * kPanelCh * 2;            // 16 KB: coefficients x channels
constexpr int kStageBytes = kStageA + kStageB;
constexpr int kMaxStages = 4;
constexpr int kLoaderWarp0 = 16, kMmaWarp = 24;               // warps 0-15 are the epilogue, 16-23 the loaders
constexpr int kThreads = 25 * 32;
constexpr int kEpiThreads = 16 * 32;
constexpr int kTmemCols = 512;
constexpr int kEpiBar = 1;                                    // named barrier of the epilogue threads

struct SmemLayout {
    uint32_t ring, symq, part, bias, enc, len8, total;
    int stages;
};

__host__ __device__ inline SmemLayout smem_layout(int k, int enc_entries, int budget)
{
    SmemLayout l;
    const uint32_t fixed = (uint32_t)k * TC_TILE_PIXELS + 4u * TC_TILE_PIXELS * 4u + (uint32_t)k * 4u +
                           (uint32_t)enc_entries * 4u + (((uint32_t)enc_entries + 15u) & ~15u);
    int stages = ((long long)budget - (long long)fixed) / kStageBytes;
    if (stages > kMaxStages) stages = kMaxStages;
    l.stages = stages < 2 ? 0 : stages;
    l.ring = 0;
    l.symq = (uint32_t)(l.stages * kStageBytes);              // [K / 4][128] words: four symbols of one pixel
    l.part = l.symq + (uint32_t)k * TC_TILE_PIXELS;           // [4][128] bits of each run of coefficients
    l.bias = l.part + 4u * TC_TILE_PIXELS * 4u;
    l.enc = l.bias + (uint32_t)k * 4u;                        // per-layer table: code << 8 | length
    l.len8 = l.enc + (uint32_t)enc_entries * 4u;              // and the lengths once more as bytes
    l.total = l.len8 + (((uint32_t)enc_entries + 15u) & ~15u);
    return l;
}

// Quantiser in fp32 (the same arithmetic as the resident-basis kernel): v = acc/step + bias,
// rounded to the nearest integer (ties to even) by adding 1.5 * 2^23, clamped while a float.
constexpr float kMagic = 12582912.0f;
constexpr uint32_t kMagicBits = 0x4B400000u;
__device__ __forceinline__ uint32_t quantise_bits(uint32_t acc_bits, float inv_step, float bias, float vmax)
{
    return __float_as_uint(fminf(fmaxf(fmaf(__uint_as_float(acc_bits), inv_step, bias) + kMagic, kMagic), vmax));
}

// kTma: the basis pieces arrive by tiled TMA copies (one instruction per stage, 64-byte swizzle)
// instead of 1024 cp.async copies; `bmap` is then the tensor map of the basis.
// kSymOnly: projection and quantiser only.  A tensor of few tiles leaves most SMs without work,
// and a tile of a wide layer takes long; in this mode the unit dealt over the blocks is one
// block of 256 coefficients of one tile, the symbols go to a.sym_park ([P][K] bytes) and the
// entropy coder runs afterwards as a kernel of its own, several threads per pixel.
template <bool kPerChannel, bool kDebug, bool kTma, bool kSymOnly>
__global__ void __launch_bounds__(kThreads, 1) encode_wide_kernel(EncodeArgs a, int smem_budget,
                                                                  const __grid_constant__ CUtensorMap bmap)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // the swizzled basis pieces want their 512-byte atoms aligned; the ring starts the buffer
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ __align__(8) unsigned long long s_full[kMaxStages], s_empty[kMaxStages], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ unsigned int s_warp_sums[4][4];
    __shared__ unsigned long long s_base;
    __shared__ int s_write_ok;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nsym = 1 << a.bits;
    const int enc_entries = (kPerChannel || a.groups != 1) ? 0 : nsym;   // the launcher sizes shared memory by the same rule
    const SmemLayout L = smem_layout(a.k, enc_entries, smem_budget);
    const int stages = L.stages;
    const uint32_t ring_addr = smem_u32(smem + L.ring);
    uint32_t *s_symq = reinterpret_cast<uint32_t *>(smem + L.symq);
    unsigned int *s_part = reinterpret_cast<unsigned int *>(smem + L.part);
    float *s_bias = reinterpret_cast<float *>(smem + L.bias);
    uint32_t *s_enc = reinterpret_cast<uint32_t *>(smem + L.enc);
    unsigned char *s_len8 = smem + L.len8;
    const int n_panels = (a.c + kPanelCh - 1) / kPanelCh;
    const int n_blocks = (a.k + kBlockCoef - 1) / kBlockCoef;

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(smem_u32(&s_full[s]), kTma ? 257 : 256); mbar_init(smem_u32(&s_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&s_tfull[b]), 1); mbar_init(smem_u32(&s_tempty[b]), kEpiThreads); }
        mbar_fence_init();
    }
    if (warp == kMmaWarp) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    for (int i = tid; i < a.k; i += kThreads) s_bias[i] = a.enc_bias[i];
    for (int i = tid; i < enc_entries; i += kThreads) {
        const uint32_t e = a.enc[i];
        s_enc[i] = e;
        s_len8[i] = (unsigned char)(e & 0xffu);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    // units dealt over the blocks: whole tiles, or (tile, coefficient block) pairs
    const long long n_units = kSymOnly ? a.n_tiles * n_blocks : a.n_tiles;
    const long long my_tiles = (n_units > blockIdx.x) ? (n_units - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp >= kLoaderWarp0 && warp < kMmaWarp) {
        // ================= loaders =================
        // 256 threads; every address is a per-thread constant plus a per-stage offset, so that a
        // stage costs a thread four 16-byte copies of the basis and four 8-byte copies (or sixteen
        // element loads) of the pixels and little arithmetic besides.
        const int lt = tid - kLoaderWarp0 * 32;               // 0..255
        const __nv_bfloat16 *xin = reinterpret_cast<const __nv_bfloat16 *>(a.x);
        const bool aligned = (a.hw & 3) == 0 && ((uintptr_t)a.x & 7u) == 0;                 // groups of four pixels are 8-byte aligned and inside one image
        const int lag = stages - 1;                           // 1..3 cp.async groups pending behind the one handed over
        // basis piece of a stage: coefficient rows j0 .. j0 + ncols, channels k0 .. k0 + 32, K-major core
        // matrices (j / 8) * 512 + (ch / 8) * 128 + (j % 8) * 16; this thread copies 16-byte piece
        // c8 of rows jb, jb + 64, jb + 128, jb + 192
        const int jb = lt >> 2, c8 = lt & 3;
        const __nv_bfloat16 *b_src0 = a.basis_bf16 + (long long)jb * a.c + c8 * 8;
        const uint32_t b_dst0 = (uint32_t)((jb >> 3) * 512 + c8 * 128 + (jb & 7) * 16);
        const long long b_row_step = 64ll * a.c;
        // pixels, aligned rows: channel kk (mod 8) of one group of four pixels
        const int lt7 = lt & 127, kk = lt7 & 7;
        const int mg = 8 * (lt7 >> 5) + ((lt7 & 31) >> 3) + 4 * (lt >> 7);
        const uint32_t a_dst0 = (uint32_t)((mg >> 1) * 128 + kk * 16 + (mg & 1) * 8);
        // pixels, unaligned rows: sixteen channels of pixel lt7
        const int ch_half = lt >> 7;
        const uint32_t a_dst1 = (uint32_t)((lt7 >> 3) * 128 + (lt7 & 7) * 2 + ch_half * 2 * 2048);
        int it = 0;
        bool alive = true;
        for (long long tl = 0; tl < my_tiles && alive; ++tl) {
            const long long unit = blockIdx.x + tl * gridDim.x;
            const long long tile = kSymOnly ? unit / n_blocks : unit;
            const int nb_lo = kSymOnly ? (int)(unit - tile * n_blocks) : 0, nb_hi = kSymOnly ? nb_lo + 1 : n_blocks;
            const long long p0 = tile * TC_TILE_PIXELS + 4 * mg;
            const bool valid = p0 < a.pixels;
            const long long img = valid ? p0 / a.hw : 0;
            const __nv_bfloat16 *a_src0 = xin + img * a.c * (long long)a.hw + (valid ? p0 - img * a.hw : 0) + (long long)kk * a.hw;
            const uint32_t a_bytes = valid ? 8u : 0u;
            const long long p1 = tile * TC_TILE_PIXELS + lt7;
            const bool valid1 = p1 < a.pixels;
            const long long img1 = valid1 ? p1 / a.hw : 0;
            const unsigned short *a_src1 = reinterpret_cast<const unsigned short *>(xin) + img1 * a.c * (long long)a.hw +
                                           (valid1 ? p1 - img1 * a.hw : 0) + (long long)(16 * ch_half) * a.hw;
            for (int nb = nb_lo; nb < nb_hi && alive; ++nb) {
                const int j0 = nb * kBlockCoef;
                const int ncols = min(kBlockCoef, a.k - j0);
                const __nv_bfloat16 *b_src = b_src0 + (long long)j0 * a.c;
                for (int kp = 0; kp < n_panels; ++kp, ++it) {
                    const int s = it % stages;
                    if (!mbar_wait(smem_u32(&s_empty[s]), ((it / stages) & 1) ^ 1)) { alive = false; break; }
                    const int k0 = kp * kPanelCh;
                    const int nk8 = min(kPanelCh, a.c - k0) >> 3;
                    const uint32_t stage_a = ring_addr + s * kStageBytes, stage_b = stage_a + kStageA;
                    if constexpr (kTma) {
                        // one thread asks for the 256 x 32 box at (channel k0, coefficient j0); rows and
                        // channels past the matrix arrive as zeros and count towards the bytes
                        if (lt == 0) {
                            mbar_arrive_expect_tx(smem_u32(&s_full[s]), (uint32_t)kStageB);
                            tma_load_2d(stage_b, &bmap, k0, j0, smem_u32(&s_full[s]));
                        }
                    } else {
                        const bool ok = c8 < nk8;
                        const __nv_bfloat16 *src = ok ? b_src + k0 : a.basis_bf16;
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (jb + 64 * u < ncols)
                                cp_async_16(stage_b + b_dst0 + u * 4096, ok ? src + u * b_row_step : src, ok ? 16u : 0u);
                    }
                    if (aligned) {
                        const __nv_bfloat16 *src = a_src0 + (long long)k0 * a.hw;
                        const long long step8 = 8ll * a.hw;
#pragma unroll
                        for (int k8 = 0; k8 < kPanelCh / 8; ++k8)
                            if (k8 < nk8) cp_async_8(stage_a + k8 * 2048 + a_dst0, src + k8 * step8, a_bytes);
                    } else {
                        // every load of the panel is in flight before the first store needs its value
                        const unsigned short *src = a_src1 + (long long)k0 * a.hw;
                        unsigned short v[kPanelCh / 2];
#pragma unroll
                        for (int i = 0; i < kPanelCh / 2; ++i)
                            v[i] = (valid1 && 16 * ch_half + i < nk8 * 8) ? __ldg(src + (long long)i * a.hw) : (unsigned short)0;
#pragma unroll
                        for (int i = 0; i < kPanelCh / 2; ++i)
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(stage_a + (i >> 3) * 2048 + a_dst1 + (i & 7) * 16), "h"(v[i]) : "memory");
                    }
                    cp_async_commit();
                    // every stage of the ring is in flight: the panel issued `lag` iterations ago is
                    // handed over once at most `lag` younger groups are still pending
                    if (it >= lag) {
                        if (lag == 3) cp_async_wait<3>();
                        else if (lag == 2) cp_async_wait<2>();
                        else cp_async_wait<1>();
                        mbar_arrive(smem_u32(&s_full[(it - lag) % stages]));
                    }
                }
            }
        }
        if (alive) {
            if (lag >= 3 && it >= 3) { cp_async_wait<2>(); mbar_arrive(smem_u32(&s_full[(it - 3) % stages])); }
            if (lag >= 2 && it >= 2) { cp_async_wait<1>(); mbar_arrive(smem_u32(&s_full[(it - 2) % stages])); }
            if (it >= 1) { cp_async_wait<0>(); mbar_arrive(smem_u32(&s_full[(it - 1) % stages])); }
        } else {
            cp_async_wait<0>();
            tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else if (warp == kMmaWarp) {
        // ================= MMA issuer =================
        if (lane == 0) {
            int it = 0;
            long long work = 0;                                // (tile, block) pairs issued so far
            bool alive = true;
            for (long long tl = 0; tl < my_tiles && alive; ++tl) {
                const long long unit = blockIdx.x + tl * gridDim.x;
                const int nb_lo = kSymOnly ? (int)(unit % n_blocks) : 0, nb_hi = kSymOnly ? nb_lo + 1 : n_blocks;
                for (int nb = nb_lo; nb < nb_hi && alive; ++nb, ++work) {
                    const int acc = (int)(work & 1);
                    if (!mbar_wait(smem_u32(&s_tempty[acc]), (uint32_t)(((work >> 1) & 1) ^ 1))) { alive = false; break; }
                    tc_fence_after_sync();
                    const int ncols = min(kBlockCoef, a.k - nb * kBlockCoef);
                    const uint32_t idesc = make_idesc_bf16(TC_TILE_PIXELS, ncols, /*A MN-major*/ true, /*B K-major*/ false);
                    const uint32_t d_tmem = tmem_base + acc * kBlockCoef;
                    for (int kp = 0; kp < n_panels; ++kp, ++it) {
                        const int s = it % stages;
                        if (!mbar_wait(smem_u32(&s_full[s]), (it / stages) & 1)) { alive = false; break; }
                        // the panel was written by the 256 loader threads (cp.async, plain stores), all of
                        // which have arrived on the barrier: one proxy fence here, between that
                        // synchronisation and the MMA's operand reads, orders the writes for all of them
                        fence_proxy_async_smem();
                        tc_fence_after_sync();
                        const int nk16 = min(kPanelCh, a.c - kp * kPanelCh) >> 4;
                        const uint32_t stage_a = ring_addr + s * kStageBytes, stage_b = stage_a + kStageA;
                        for (int q = 0; q < nk16; ++q) {
                            const uint64_t adesc = make_smem_desc(stage_a + q * 4096, 2048, 128);
                            const uint64_t bdesc = kTma ? make_smem_desc_sw64(stage_b + q * 32, 512) : make_smem_desc(stage_b + q * 256, 128, 512);
                            mma_bf16_ss(d_tmem, adesc, bdesc, idesc, (kp | q) != 0 ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&s_empty[s]));
                    }
                    if (alive) mma_commit(smem_u32(&s_tfull[acc]));
                }
            }
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else {
        // ================= epilogue =================
        const int part = warp >> 2;                // which quarter of a block's coefficients, and which run of a pixel
        const int wq = warp & 3;                   // TMEM lane quarter
        const int m = wq * 32 + lane;              // pixel within the tile = TMEM lane
        const float inv_step = (float)(a.basis_scale / a.step);   // the operand holds basis / basis_scale
        const float coef_scale = (float)a.basis_scale;
        const float vmax = kMagic + (float)(nsym - 1);
        const uint32_t len8_rel = smem_u32(s_len8) - kMagicBits;  // + (kMagicBits + q) = address of len8[q]
        // Four runs of coefficients whose bits are added up separately, one per thread of a pixel,
        // so that the four pack side by side: the chunks of a pixel, their halves, or quarters
        // of the pixel.  The bounds are multiples of 16 (a chunk is a multiple of 16 coefficients).
        int bnd[5];
        {
            const int n_chunk = a.k / a.splits;                          // coefficients per chunk of a pixel
            const int per = 4 / a.splits;                                // runs per chunk: 4, 2 or 1
            const int step = ((n_chunk + 16 * per - 1) / (16 * per)) * 16;
            for (int v = 0; v <= 4; ++v) {
                const int c = v / per, r = v - c * per;
                bnd[v] = min(c * n_chunk + min(r * step, n_chunk), a.k);
            }
        }
        const int run_lo = part, run_hi = part + 1;                      // this thread packs run `part`
        long long work = 0;
        bool alive = true;

        for (long long tl = 0; tl < my_tiles && alive; ++tl) {
            const long long unit = blockIdx.x + tl * gridDim.x;
            const long long tile = kSymOnly ? unit / n_blocks : unit;
            const int nb_lo = kSymOnly ? (int)(unit - tile * n_blocks) : 0, nb_hi = kSymOnly ? nb_lo + 1 : n_blocks;
            const long long p = tile * TC_TILE_PIXELS + m;
            const bool valid = p < a.pixels;
            if constexpr (!kSymOnly) {
                s_part[part * TC_TILE_PIXELS + m] = 0u;
                named_bar_sync(kEpiBar, kEpiThreads);  // the previous tile's symbols have been packed; the sums are zero
            }

            // pass 1: quantise block by block, park the symbols, add up the code lengths
            for (int nb = nb_lo; nb < nb_hi && alive; ++nb, ++work) {
                const int acc = (int)(work & 1);
                if (!mbar_wait(smem_u32(&s_tfull[acc]), (uint32_t)((work >> 1) & 1))) { alive = false; break; }
                tc_fence_after_sync();
                const int ncols = min(kBlockCoef, a.k - nb * kBlockCoef);
                const int part_cols = ((ncols + 63) / 64) * 16;
                const int col0 = part * part_cols;
                const int my_n = max(0, min(part_cols, ncols - col0));
                const uint32_t trow = tmem_base + acc * kBlockCoef + ((uint32_t)(wq * 32) << 16) + col0;
#pragma unroll 1
                for (int blk = 0; blk * 16 < my_n; ++blk) {
                    const int j0 = nb * kBlockCoef + col0 + blk * 16;
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(trow + blk * 16, r);
                    float4 bias4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) bias4[i] = *reinterpret_cast<const float4 *>(s_bias + j0 + 4 * i);
                    const float *biasv = reinterpret_cast<const float *>(bias4);
                    tmem_ld_wait();
                    unsigned int bits16 = 0;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint32_t vb = quantise_bits(r[i], inv_step, biasv[i], vmax);
                        if constexpr (kSymOnly) {
                        } else if constexpr (kPerChannel) bits16 += __ldg(a.enc + (j0 + i) * nsym + (vb & 0xffu)) & 0xffu;
                        else {
                            uint32_t l;
                            asm("ld.shared.u8 %0, [%1];" : "=r"(l) : "r"(vb + len8_rel));
                            bits16 += l;
                        }
                        if constexpr (kDebug) {
                            if (valid && a.dbg_coef) a.dbg_coef[p * a.k + j0 + i] = fmaf(__uint_as_float(r[i]), coef_scale, -a.tmu32[j0 + i]);
                            if (valid && a.dbg_sym) a.dbg_sym[p * a.k + j0 + i] = (uint8_t)(vb & 0xffu);
                        }
                        r[i] = vb;
                    }
                    uint32_t packed[4];
#pragma unroll
                    for (int i = 0; i < 16; i += 4)          // low bytes of four values -> one word
                        packed[i >> 2] = __byte_perm(__byte_perm(r[i], r[i + 1], 0x0040), __byte_perm(r[i + 2], r[i + 3], 0x0040), 0x5410);
                    if constexpr (kSymOnly) {
                        // sixteen symbols of the pixel's row of [P][K] (K and j0 are multiples of 16)
                        if (valid) *reinterpret_cast<uint4 *>(a.sym_park + p * a.k + j0) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i) s_symq[((j0 >> 2) + i) * TC_TILE_PIXELS + m] = packed[i];
                        const int run = (j0 >= bnd[1] ? 1 : 0) + (j0 >= bnd[2] ? 1 : 0) + (j0 >= bnd[3] ? 1 : 0);
                        if (valid) atomicAdd(&s_part[run * TC_TILE_PIXELS + m], bits16);
                    }
                }
                // the accumulator is free for the block after next
                tc_fence_before_sync();
                mbar_arrive(smem_u32(&s_tempty[acc]));
            }
            if (!alive) break;
            if constexpr (kSymOnly) continue;      // offsets and packing belong to the kernel that follows
            named_bar_sync(kEpiBar, kEpiThreads);  // every run's sum is complete

            // bit offsets: pixel-major, runs in order inside a pixel
            unsigned int run_bits[4], pixel_bits = 0, before_mine = 0, my_bits = 0;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                run_bits[v] = s_part[v * TC_TILE_PIXELS + m];
                if (v < run_lo) before_mine += run_bits[v];
                if (v >= run_lo && v < run_hi) my_bits += run_bits[v];
                pixel_bits += run_bits[v];
            }
            unsigned int inc = pixel_bits;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += up;
            }
            if (lane == 31) s_warp_sums[part][wq] = inc;
            named_bar_sync(kEpiBar, kEpiThreads);
            unsigned int before = 0, tile_bits = 0;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const unsigned int sw = s_warp_sums[part][w];
                if (w < wq) before += sw;
                tile_bits += sw;
            }
            const unsigned int pixel_off = before + inc - pixel_bits;
            const unsigned int my_off = pixel_off + before_mine;
            unsigned int chunk_end = 0;            // end of the chunk of several pixels that starts at this pixel
            if (a.chunk_pixels > 1) {
                const int cpx = a.chunk_pixels;
                if (cpx < 32) {
                    const unsigned int further = __shfl_down_sync(0xffffffffu, pixel_off, cpx);
                    chunk_end = (lane + cpx < 32) ? further : before + s_warp_sums[part][wq];
                } else {
#pragma unroll
                    for (int w = 0; w < 4; ++w)
                        if (w < wq + (cpx >> 5)) chunk_end += s_warp_sums[part][w];
                }
            }
            const unsigned long long padded = ((unsigned long long)tile_bits + 127ull) & ~127ull;
            if (warp == 0) {
                if (lane == 0) lookback_publish(a.tile_state, tile, padded);
                __syncwarp();
                bool ok;
                const unsigned long long base = lookback_resolve(a.tile_state, tile, padded, a.status, ok);
                if (lane == 0) {
                    const bool fits = base + padded <= a.capacity_bits;
                    if (ok && !fits) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
                    s_base = base;
                    s_write_ok = (ok && fits) ? 1 : 0;
                    a.tile_off[tile] = base;
                    if (tile == a.n_tiles - 1) a.tile_off[a.n_tiles] = base + padded;
                }
            }
            // chunk lengths
            if (valid) {
                if (a.splits == 4) {
                    a.chunk_len[p * 4 + part] = (uint16_t)run_bits[part];
                } else if (a.splits == 2) {
                    if ((part & 1) == 0) a.chunk_len[p * 2 + (part >> 1)] = (uint16_t)(run_bits[part] + run_bits[part + 1]);
                } else if (part == 0) {
                    if (a.chunk_pixels == 1) a.chunk_len[p] = (uint16_t)pixel_bits;
                    else if ((p % a.chunk_pixels) == 0) a.chunk_len[p / a.chunk_pixels] = (uint16_t)(chunk_end - pixel_off);
                }
            }
            named_bar_sync(kEpiBar, kEpiThreads);  // the tile's position is known
            const unsigned long long base = s_base;
            const bool write_ok = s_write_ok != 0;
            if (write_ok) {
                uint4 *z = reinterpret_cast<uint4 *>(a.stream + (base >> 5));
                for (unsigned int i = tid; i < (unsigned int)(padded >> 7); i += kEpiThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
            }
            named_bar_sync(kEpiBar, kEpiThreads);  // the tile's words are zero

            // pass 2: codes of the parked symbols, packed into the stream
            if (valid && write_ok && my_bits > 0) {
                BitWriter w;
                w.init(a.stream, base + my_off);
                for (int j = bnd[run_lo]; j < bnd[run_hi]; j += 4) {
                    const uint32_t word = s_symq[(j >> 2) * TC_TILE_PIXELS + m];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t q = (word >> (8 * i)) & 0xffu;
                        uint32_t e;
                        if constexpr (kPerChannel) e = __ldg(a.enc + (j + i) * nsym + q);
                        else e = s_enc[q];
                        w.put(e >> 8, (int)(e & 0xffu));
                    }
                }
                w.finish();
            }
        }
        if (!alive && tid == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
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

bool tc_encode_wide_supported(const tc_ctx *ctx, const EncodeArgs &a)
{
    if (a.c % 16 != 0 || a.k % 16 != 0 || a.k < 16 || a.k > a.c || a.c > TC_MAX_C) return false;
    if (a.splits != 1 && a.splits != 2 && a.splits != 4) return false;
    if (a.splits > 1 && (a.chunk_pixels != 1 || (a.k / a.splits) % 16 != 0 || a.k % a.splits != 0)) return false;
    if (a.groups != 1 && a.groups != a.k) return false;
    const SmemLayout l = smem_layout(a.k, a.groups == 1 ? (1 << a.bits) : 0, ctx->max_smem_optin - 2048);
    return l.stages >= 2;
}

tc_status tc_launch_encode_wide(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const int budget = ctx->max_smem_optin - 2048;            // leaves room for the static shared variables
    const SmemLayout l = smem_layout(a.k, a.groups == 1 ? (1 << a.bits) : 0, budget);
    if (l.stages < 2) return TC_ERR_UNSUPPORTED;
    const bool per_channel = a.groups != 1, debug = a.dbg_coef || a.dbg_sym;
    const bool tma = a.basis_map != nullptr;
    const bool sym_only = a.sym_park != nullptr;
    void (*kernel)(EncodeArgs, int, const CUtensorMap) =
        sym_only ? (tma ? (debug ? encode_wide_kernel<false, true, true, true> : encode_wide_kernel<false, false, true, true>)
                        : (debug ? encode_wide_kernel<false, true, false, true> : encode_wide_kernel<false, false, false, true>))
        : tma ? (per_channel ? (debug ? encode_wide_kernel<true, true, true, false> : encode_wide_kernel<true, false, true, false>)
                           : (debug ? encode_wide_kernel<false, true, true, false> : encode_wide_kernel<false, false, true, false>))
            : (per_channel ? (debug ? encode_wide_kernel<true, true, false, false> : encode_wide_kernel<true, false, false, false>)
                           : (debug ? encode_wide_kernel<false, true, false, false> : encode_wide_kernel<false, false, false, false>));
    const size_t smem_bytes = (size_t)l.total + 1024;         // room to align the buffer to 1 KB
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
        return TC_ERR_CUDA;
    const long long n_units = sym_only ? a.n_tiles * ((a.k + kBlockCoef - 1) / kBlockCoef) : a.n_tiles;
    const unsigned int grid = (unsigned int)((n_units < ctx->sm_count) ? n_units : ctx->sm_count);
    EncodeArgs args = a;
    int budget_arg = budget;
    CUtensorMap map_arg;
    if (tma) map_arg = *a.basis_map;
    else memset(&map_arg, 0, sizeof(map_arg));
    void *params[] = {&args, &budget_arg, &map_arg};
    // cooperative launch: the grid must be co-resident, which is what makes the look-back safe
    const cudaError_t err = cudaLaunchCooperativeKernel((void *)kernel, dim3(grid), dim3(kThreads), params, smem_bytes, s);
    if (err != cudaSuccess) {
        if (getenv("TC_VERBOSE")) fprintf(stderr, "tc: wide encode launch failed: %s\n", cudaGetErrorString(err));
        cudaGetLastError();
        return TC_ERR_CUDA;
    }
    return TC_OK;
}
