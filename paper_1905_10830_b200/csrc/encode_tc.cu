// Fused tensor-core encode for bf16 tensors (Section 3: transform, quantiser, VLC).
//
// One persistent block per SM walks tiles of 128 consecutive pixels.  Warp roles:
//   warps 0-7, 8-15  two epilogue groups (alternating tiles).  Within a group warps 0-3 own the
//                    first half of the coefficients of the tile's 128 pixels and warps 4-7 the
//                    second half: TMEM -> registers, quantise, code lengths, bit offsets (scan +
//                    tile look-back), pack, 128-bit stores.  The symbols stay packed in
//                    registers between the length pass and the packing pass.
//   warps 21, 22     one store warp per epilogue group: resolves the tile's stream offset by
//                    look-back and copies the group's staging buffer out, while the group
//                    already works on its next tile
//   warps 16-19      loaders: cp.async NCHW -> shared memory in the MMA's MN-major layout
//   warp 20          one thread issues tcgen05.mma:  D[pixel][coef] = X_tile[pixel][c] * T[coef][c]
// The basis T (bf16, K x C) stays resident in shared memory; the X tile streams through a ring
// of 64-channel panels; the fp32 accumulators are double-buffered in tensor memory so that the
// epilogue of one tile overlaps the loads and MMAs of the next.
#include <cstdio>
#include <cstdlib>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace tcdev;
using namespace sm100;

constexpr int kPanelCh = 64;                      // channels per ring stage
constexpr int kStages = 4;
constexpr int kStageBytes = kPanelCh * TC_TILE_PIXELS * 2;   // 16 KB
constexpr int kLag = 2;                           // cp.async groups kept in flight per loader thread; the
                                                  // remaining ring stage absorbs the MMA's latency
constexpr int kStagingBytes = 15360;              // packed-bit staging per epilogue group (15 KB)
constexpr int kEpiWarps = 16;                     // 2 groups x (2 column halves x 4 lane quarters)
constexpr int kLoaderWarp0 = kEpiWarps, kMmaWarp = kEpiWarps + 4;
constexpr int kStoreWarp0 = kMmaWarp + 1;         // two store warps follow
constexpr int kThreads = (kEpiWarps + 7) * 32;
constexpr int kMaxHalfCols = 128;                 // coefficients per epilogue thread (K <= 256)
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kPairMaxBits = 4;                   // symbols of up to 4 bits are coded two at a time (256-entry tables)

struct SmemLayout {
    uint32_t basis, ring, staging, enc, len8, bias, xch, total;
};

__host__ __device__ inline SmemLayout smem_layout(int c, int k, int enc_entries)
{
    SmemLayout l;
    l.basis = 0;
    l.ring = (uint32_t)(((size_t)k * c * 2 + 1023) & ~(size_t)1023);
    l.staging = l.ring + kStages * kStageBytes;
    l.enc = l.staging + 2 * kStagingBytes;
    l.len8 = l.enc + (uint32_t)enc_entries * 8;          // code lengths as bytes (per-layer table)
    l.bias = (l.len8 + (enc_entries ? 256u : 0u) + 15u) & ~15u;
    l.xch = l.bias + (uint32_t)k * 4;                   // code lengths exchanged between the halves: [2 groups][2][128] u16
    l.total = l.xch + 2u * 2u * 128u * 2u;
    return l;
}

// Quantiser in fp32.  The level is rounded to the nearest integer (ties to even) by adding
// 1.5 * 2^23 -- the integer then sits in the low mantissa bits.  (A float -> int conversion
// instruction would do the same but issues at a quarter of the rate.)
constexpr float kMagic = 12582912.0f;
constexpr uint32_t kMagicBits = 0x4B400000u;

// Bit writer into the shared-memory staging buffer.  A word is stored (plain, predicated
// store) by the writer that supplies its last bit; bits that other writers own in that word
// are zero in the stored value.  What is left after the last full word -- a writer's tail --
// is merged afterwards with one shared-memory OR per writer (finish()), behind a barrier, so
// that it cannot be overwritten by the store of the word's last writer.  A put adds fewer
// than 32 bits (the pending count stays below 32 between puts).
struct SmemBitWriter {
    uint32_t addr;             // shared address of the word being filled
    uint32_t lo, hi;           // pending bits, right-aligned in hi:lo (bits above `pending` are stale)
    int pending;
    __device__ __forceinline__ void init(uint32_t base_addr, unsigned int bitpos)
    {
        addr = base_addr + (bitpos >> 5) * 4u;
        pending = (int)(bitpos & 31u);
        lo = hi = 0;
    }
    __device__ __forceinline__ void put(uint32_t code, int len)
    {
        // hi:lo <<= len; lo |= code; pending += len; if (pending >= 32) { store bits
        // [pending-32, pending) of hi:lo; addr += 4; pending -= 32; }  (the funnel shift takes
        // its amount modulo 32, so `pending` itself serves as pending - 32)
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b32 t, o;\n\t"
            "shf.l.wrap.b32 %1, %0, %1, %5;\n\t"
            "shl.b32 t, %0, %5;\n\t"
            "or.b32 %0, t, %4;\n\t"
            "add.s32 %2, %2, %5;\n\t"
            "setp.ge.s32 p, %2, 32;\n\t"
            "shf.r.wrap.b32 o, %0, %1, %2;\n\t"
            "@p st.shared.u32 [%3], o;\n\t"
            "@p add.s32 %3, %3, 4;\n\t"
            "@p add.s32 %2, %2, -32;\n\t}"
            : "+r"(lo), "+r"(hi), "+r"(pending), "+r"(addr)
            : "r"(code), "r"(len));
    }
    // call after a barrier that follows every writer's puts
    __device__ __forceinline__ void finish()
    {
        const uint32_t out = pending > 0 ? (lo << (32 - pending)) : 0u;
        if (out) asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(addr), "r"(out) : "memory");
    }
};

// Two coefficients at once.  The position on the quantiser's grid is computed as a fraction of
// its range, t = (y - lo) / (step (2^b - 1)), with a saturating multiply-add: the clamp to the
// first and last level costs nothing.  A second multiply-add (packed: two fp32 lanes per
// instruction, each rounded exactly as the scalar instruction rounds) scales t back to levels and
// adds the magic constant, which leaves the level, rounded to nearest even, in the mantissa.
__device__ __forceinline__ void quantise_bits2(uint32_t acc0, uint32_t acc1, float inv_range, float bias0, float bias1, float top,
                                               uint32_t &q0, uint32_t &q1)
{
    float t0, t1;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(t0) : "f"(__uint_as_float(acc0)), "f"(inv_range), "f"(bias0));
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(t1) : "f"(__uint_as_float(acc1)), "f"(inv_range), "f"(bias1));
    asm("{\n\t.reg .b64 v, s, m;\n\t"
        "mov.b64 v, {%2, %3};\n\t"
        "mov.b64 s, {%4, %4};\n\t"
        "mov.b64 m, {%5, %5};\n\t"
        "fma.rn.f32x2 v, v, s, m;\n\t"
        "mov.b64 {%0, %1}, v;\n\t}"
        : "=r"(q0), "=r"(q1) : "f"(t0), "f"(t1), "f"(top), "f"(kMagic));
}

// kPair (per-layer tables, b <= 4): the code tables are indexed by two neighbouring symbols at
// once (q0 | q1 << b, at most 256 entries), which halves the lookups of both passes.
// kHist (statistics, Section 3.1 "Variable length coding": the entropy needs the distribution of
// the symbols): every symbol is also counted, per coefficient channel, into a.hist.  The lanes of
// a warp hold one coefficient of 32 pixels; the symbol most of them hold (the zero level) is
// counted once per warp from a ballot, the others one atomic each.
template <bool kPerChannel, bool kDebug, bool kPair, bool kHist>
__global__ void __launch_bounds__(kThreads, 1) encode_tc_kernel(EncodeArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_full[kStages], s_empty[kStages], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ unsigned int s_warp_sums[2][4];
    __shared__ unsigned long long s_base[2];
    __shared__ int s_write_ok[2];
    __shared__ __align__(8) unsigned long long s_stg_full[2], s_stg_free[2];   // staging hand-over to the store warp
    __shared__ unsigned long long s_padded[2];
    __shared__ int s_store_cmd[2];             // 1: copy the staged tile out, 2: nothing to copy, 3: stop

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nsym = 1 << a.bits;
    constexpr bool enc_in_smem = !kPerChannel;
    const int enc_entries = enc_in_smem ? (kPair ? nsym * nsym : nsym) : 0;
    const SmemLayout L = smem_layout(a.c, a.k, enc_entries);
    unsigned char *s_basis = smem + L.basis;
    uint32_t *s_enc = reinterpret_cast<uint32_t *>(smem + L.enc);
    float *s_bias = reinterpret_cast<float *>(smem + L.bias);
    const uint32_t ring_addr = smem_u32(smem + L.ring);
    const uint32_t basis_addr = smem_u32(s_basis);
    const int n_panels = (a.c + kPanelCh - 1) / kPanelCh;

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&s_full[s]), 128); mbar_init(smem_u32(&s_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&s_tfull[b]), 1);
            mbar_init(smem_u32(&s_tempty[b]), 256);
            mbar_init(smem_u32(&s_stg_full[b]), 256);
            mbar_init(smem_u32(&s_stg_free[b]), 1);
        }
        mbar_fence_init();
    }
    if (warp == kMmaWarp) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    // basis -> K-major core-matrix layout: element (j, ch) at (j/8)*sbo + (ch/8)*128 + (j%8)*16 + (ch%8)*2
    {
        const uint32_t sbo = (uint32_t)(a.c / 8) * 128u;
        const int chunks_per_row = a.c / 8;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.basis_bf16);
        // (asynchronous copies: all of a thread's pieces are in flight at once)
        for (int i = tid; i < a.k * chunks_per_row; i += kThreads) {
            const int j = i / chunks_per_row, c8 = i - j * chunks_per_row;
            cp_async_16(basis_addr + (j >> 3) * sbo + c8 * 128 + (j & 7) * 16, src + i, 16u);
        }
        cp_async_commit();
        for (int i = tid; i < a.k; i += kThreads) s_bias[i] = a.enc_bias[i] / (float)(nsym - 1);   // as a fraction of the range
        if (enc_in_smem)
            for (int i = tid; i < enc_entries; i += kThreads) {
                // per-layer table: (1 << length, code) pairs, so that appending a code to a register is
                // one multiply-add, and the lengths once more as bytes.  In pair mode entry
                // q0 | q1 << b holds the two codes joined (q0's first), at most 24 bits.
                uint32_t len, code;
                if constexpr (kPair) {
                    const uint32_t e0 = a.enc[i & (nsym - 1)], e1 = a.enc[i >> a.bits];
                    len = (e0 & 0xffu) + (e1 & 0xffu);
                    code = ((e0 >> 8) << (e1 & 0xffu)) | (e1 >> 8);
                } else {
                    const uint32_t e = a.enc[i];
                    len = e & 0xffu;
                    code = e >> 8;
                }
                s_enc[2 * i] = 1u << len;
                s_enc[2 * i + 1] = code;
                (smem + L.len8)[i] = (unsigned char)len;
            }
    }
    cp_async_wait<0>();
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    const long long my_tiles = (a.n_tiles > blockIdx.x) ? (a.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp >= kLoaderWarp0 && warp < kMmaWarp) {
        // ================= loaders =================
        const int lw = warp - kLoaderWarp0, kk = lane & 7;
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
            if (it >= 2) { cp_async_wait<1>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 2) % kStages])); }
            if (it >= 1) { cp_async_wait<0>(); fence_proxy_async_smem(); mbar_arrive(smem_u32(&s_full[(it - 1) % kStages])); }
        } else {
            cp_async_wait<0>();
            tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else if (warp == kMmaWarp) {
        // ================= MMA issuer =================
        // The whole warp walks the loop and waits on the barriers; lane 0 issues, through instructions
        // that carry their own guard (a branch taken by one lane around every MMA costs about 90
        // cycles per instruction).
        {
            const uint32_t issuer = lane == 0 ? 1u : 0u;
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
                        mma_bf16_ss_guarded(d_tmem, adesc, bdesc, idesc, (kp | q) != 0 ? 1u : 0u, issuer);
                    }
                    mma_commit_guarded(smem_u32(&s_empty[s]), issuer);
                }
                if (alive) mma_commit_guarded(smem_u32(&s_tfull[acc]), issuer);
            }
            if (!alive && issuer) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else if (warp >= kStoreWarp0) {
        // ================= store warps =================
        const int grp = warp - kStoreWarp0;
        const uint32_t stg_addr = smem_u32(smem + L.staging + grp * kStagingBytes);
        long long n = 0;
        for (long long tl = grp; tl < my_tiles; tl += 2, ++n) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            if (!mbar_wait(smem_u32(&s_stg_full[grp]), (uint32_t)(n & 1))) { if (lane == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT); break; }
            const int cmd = s_store_cmd[grp];
            if (cmd == 3) break;
            if (cmd == 1) {
                const unsigned long long padded = s_padded[grp];
                bool ok;
                const unsigned long long base = lookback_resolve(a.tile_state, tile, padded, a.status, ok);
                const bool fits = base + padded <= a.capacity_bits;
                if (ok && !fits && lane == 0) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
                if (ok && fits) {
                    uint4 *dst = reinterpret_cast<uint4 *>(a.stream + (base >> 5));
                    for (unsigned int i = lane; i < (unsigned int)(padded >> 7); i += 32) {
                        uint4 v;
                        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(stg_addr + i * 16u));
                        dst[i] = v;
                    }
                }
                if (lane == 0) {
                    a.tile_off[tile] = base;
                    if (tile == a.n_tiles - 1) a.tile_off[a.n_tiles] = base + padded;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_stg_free[grp]));
        }
    } else {
        // ================= epilogue groups =================
        const int grp = warp >> 3;                 // 0 or 1
        const int wg = warp & 7;
        const int half = wg >> 2;                  // which half of the coefficients
        const int wq = wg & 3;                     // TMEM lane quarter
        const int m = wq * 32 + lane;              // pixel within the tile = TMEM lane
        const int tg = (tid & 255);                // thread within the group
        const int half_cols = ((a.k + 31) / 32) * 16;              // columns of half 0 (multiple of 16)
        const int col0 = half * half_cols;
        const int ncols = half ? a.k - half_cols : half_cols;      // multiple of 16, may be 0
        unsigned char *stg = smem + L.staging + grp * kStagingBytes;
        const uint32_t stg_addr = smem_u32(stg);
        const uint32_t enc_addr = smem_u32(s_enc);
        const uint32_t len8_rel = smem_u32(smem + L.len8) - kMagicBits;   // + (kMagicBits + q) = address of len8[q]
        const uint32_t pair_len_rel = smem_u32(smem + L.len8) - kMagicBits * (1u + (1u << a.bits));   // same for a pair sum
        unsigned short *xch = reinterpret_cast<unsigned short *>(smem + L.xch) + grp * 256;   // [2][128] lengths exchanged between the halves
        long long n_done = 0;                      // tiles this group has handed to its store warp
        const float inv_range = (float)(a.basis_scale / (a.step * (double)(nsym - 1)));   // the operand holds basis / basis_scale
        const float top = (float)(nsym - 1);
        const float coef_scale = (float)a.basis_scale;
        const int bar_id = 1 + grp;
        bool alive = true;

        auto resolve_base = [&](long long tile, unsigned long long padded) {
            if (wg == 0) {
                bool ok;
                const unsigned long long base = lookback_resolve(a.tile_state, tile, padded, a.status, ok);
                if (lane == 0) {
                    const bool fits = base + padded <= a.capacity_bits;
                    if (ok && !fits) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
                    s_base[grp] = base;
                    s_write_ok[grp] = (ok && fits) ? 1 : 0;
                }
            }
        };

        for (long long tl = grp; tl < my_tiles && alive; tl += 2) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            const long long p = tile * TC_TILE_PIXELS + m;
            const bool valid = p < a.pixels;
            if (!mbar_wait(smem_u32(&s_tfull[grp]), (uint32_t)((tl >> 1) & 1))) { alive = false; break; }
            tc_fence_after_sync();
            const uint32_t trow = tmem_base + grp * kAccCols + ((uint32_t)(wq * 32) << 16) + col0;

            // pass 1: quantise, keep the symbols (one byte each) in registers, add up code lengths
            uint32_t sym[kPair ? kMaxHalfCols / 8 : kMaxHalfCols / 4];   // one byte per symbol, or per pair of symbols
            uint32_t blk_bits[kMaxHalfCols / 64] = {};          // code bits of each block of 16 symbols, one byte each
            unsigned int my_bits = 0, bits_first = 0;          // bits_first: the first half of this thread's coefficients
            [[maybe_unused]] unsigned int n_clamped = 0;       // statistics mode: coefficients outside the quantiser's range
#pragma unroll
            for (int blk = 0; blk < kMaxHalfCols / 16; ++blk) {
                if (blk * 16 < ncols) {
                    if (blk * 32 == ncols) bits_first = my_bits;
                    const unsigned int bits_before = my_bits;
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(trow + blk * 16, r);
                    float4 bias4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) bias4[i] = *reinterpret_cast<const float4 *>(s_bias + col0 + blk * 16 + 4 * i);
                    const float *biasv = reinterpret_cast<const float *>(bias4);
                    tmem_ld_wait();
                    uint32_t qv[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) quantise_bits2(r[i], r[i + 1], inv_range, biasv[i], biasv[i + 1], top, qv[i], qv[i + 1]);
                    if constexpr (kHist) {
                        // every symbol other than the zero level is counted; the zero level's count is what
                        // is left of the pixels, which the caller works out
                        const uint32_t modal_bits = kMagicBits + (uint32_t)a.hist_modal;
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int j = col0 + blk * 16 + i;
                            if (valid && qv[i] != modal_bits) atomicAdd(a.hist + (size_t)j * nsym + (qv[i] & 0xffu), 1ull);
                            // outside the quantiser's range [lo, lo + (2^b - 1) step]
                            const float t = fmaf(__uint_as_float(r[i]), inv_range, biasv[i]);
                            n_clamped += (valid && (t < 0.f || t > 1.f)) ? 1u : 0u;
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int j = col0 + blk * 16 + i;
                        const uint32_t vb = qv[i];
                        if constexpr (kPerChannel) my_bits += __ldg(a.enc + j * nsym + (vb & 0xffu)) & 0xffu;
                        else if constexpr (!kPair) {
                            uint32_t l;
                            asm("ld.shared.u8 %0, [%1];" : "=r"(l) : "r"(vb + len8_rel));
                            my_bits += l;
                        }
                        if constexpr (kDebug) {
                            if (valid && a.dbg_coef) a.dbg_coef[p * a.k + j] = fmaf(__uint_as_float(r[i]), coef_scale, -a.tmu32[j]);
                            if (valid && a.dbg_sym) a.dbg_sym[p * a.k + j] = (uint8_t)(vb & 0xffu);
                        }
                        r[i] = vb;
                    }
                    if constexpr (kPair) {
                        // pair index in the low byte of vb0 + (vb1 << b) (the magic constants have a zero
                        // low byte); the same sum, rebased, addresses the pair-length table
#pragma unroll
                        for (int i = 0; i < 16; i += 2) {
                            r[i] = r[i] + (r[i + 1] << a.bits);
                            uint32_t l;
                            asm("ld.shared.u8 %0, [%1];" : "=r"(l) : "r"(r[i] + pair_len_rel));
                            my_bits += l;
                        }
#pragma unroll
                        for (int i = 0; i < 16; i += 8)      // low bytes of four pairs -> one register
                            sym[blk * 2 + i / 8] = __byte_perm(__byte_perm(r[i], r[i + 2], 0x0040), __byte_perm(r[i + 4], r[i + 6], 0x0040), 0x5410);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; i += 4)      // low bytes of four values -> one register
                            sym[blk * 4 + i / 4] = __byte_perm(__byte_perm(r[i], r[i + 1], 0x0040), __byte_perm(r[i + 2], r[i + 3], 0x0040), 0x5410);
                    }
                    blk_bits[blk >> 2] |= (my_bits - bits_before) << (8 * (blk & 3));      // at most 16 * 12 = 192
                }
            }
            // the accumulator buffer is free for the tile after next
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&s_tempty[grp]));
            if constexpr (kHist) {
                if (a.clamped) {
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) n_clamped += __shfl_xor_sync(0xffffffffu, n_clamped, d);
                    if (lane == 0 && n_clamped) atomicAdd(a.clamped, (unsigned long long)n_clamped);
                }
            }
            if (!valid) my_bits = 0;

            // bit offsets: pixel-major, first half before second half
            xch[half * 128 + m] = (unsigned short)my_bits;     // at most 128 * 12 bits
            named_bar_sync(bar_id, 256);
            const unsigned int other = xch[(half ^ 1) * 128 + m];
            const unsigned int pair = my_bits + other;
            unsigned int inc = pair;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += up;
            }
            if (lane == 31 && half == 0) s_warp_sums[grp][wq] = inc;
            named_bar_sync(bar_id, 256);
            unsigned int before = 0, tile_bits = 0;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const unsigned int sw = s_warp_sums[grp][w];
                if (w < wq) before += sw;
                tile_bits += sw;
            }
            const unsigned int pixel_off = before + inc - pair;
            const unsigned int my_off = pixel_off + (half ? other : 0u);
            // end of the chunk that starts at this pixel (chunks of several pixels): the offset of
            // the pixel chunk_pixels further on, which sits in this warp, or is a sum of warp totals
            unsigned int chunk_end = 0;
            if (a.chunk_pixels > 1) {
                const int cpx = a.chunk_pixels;
                if (cpx < 32) {
                    const unsigned int further = __shfl_down_sync(0xffffffffu, pixel_off, cpx);
                    chunk_end = (lane + cpx < 32) ? further : before + s_warp_sums[grp][wq];
                } else {
#pragma unroll
                    for (int w = 0; w < 4; ++w)
                        if (w < wq + (cpx >> 5)) chunk_end += s_warp_sums[grp][w];
                }
            }
            const unsigned long long padded = ((unsigned long long)tile_bits + 127ull) & ~127ull;
            if (tg == 0) lookback_publish(a.tile_state, tile, padded);
            const bool staged = padded <= (unsigned long long)kStagingBytes * 8ull;
            // the store warp must be done with the previous tile before staging is written again
            if (n_done > 0 && !mbar_wait(smem_u32(&s_stg_free[grp]), (uint32_t)((n_done - 1) & 1))) { alive = false; break; }

            if (staged) {
                // every word below tile_bits / 32 is stored by the writer of its last bit; the last
                // partial word and the padding up to the 128-bit boundary start as zero
                const unsigned int first_open = tile_bits >> 5, end_word = (unsigned int)(padded >> 5);
                if ((unsigned int)tg < end_word - first_open)
                    asm volatile("st.shared.u32 [%0], %1;" ::"r"(stg_addr + (first_open + tg) * 4u), "r"(0u) : "memory");
            } else {
                // rare: the tile does not fit the staging buffer -> resolve its position first and
                // pack straight into (zeroed) global memory
                resolve_base(tile, padded);
                named_bar_sync(bar_id, 256);
                if (s_write_ok[grp]) {
                    uint4 *z = reinterpret_cast<uint4 *>(a.stream + (s_base[grp] >> 5));
                    for (unsigned int i = tg; i < (unsigned int)(padded >> 7); i += 256) z[i] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            named_bar_sync(bar_id, 256);

            // pass 2: look up the codes of the kept symbols and pack; two symbols are joined in
            // registers and appended as one piece of at most 24 bits
            const bool do_pack = valid && (staged || s_write_ok[grp]);
            auto pack_tile = [&](auto &w) {
                if (!do_pack) return;
#pragma unroll
                for (int blk = 0; blk < kMaxHalfCols / 16; ++blk) {
                    if (blk * 16 < ncols) {
#pragma unroll
                        const int nbits = (int)((blk_bits[blk >> 2] >> (8 * (blk & 3))) & 0xffu);
                        if (!kPerChannel && nbits < 32) {
                            // the whole block fits one register: acc = acc * 2^len + code per symbol (or pair)
                            uint32_t acc = 0;
                            if constexpr (kPair) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const uint32_t q = (sym[blk * 2 + i / 4] >> (8 * (i & 3))) & 0xffu;
                                    uint32_t mul, code;
                                    asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(mul), "=r"(code) : "r"(enc_addr + q * 8u));
                                    acc = acc * mul + code;
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const uint32_t q = (sym[blk * 4 + i / 4] >> (8 * (i & 3))) & 0xffu;
                                    uint32_t mul, code;
                                    asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(mul), "=r"(code) : "r"(enc_addr + q * 8u));
                                    acc = acc * mul + code;
                                }
                            }
                            w.put(acc, nbits);
                        } else if constexpr (kPair) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) {         // pair by pair: at most 24 bits each
                                const uint32_t q = (sym[blk * 2 + i / 4] >> (8 * (i & 3))) & 0xffu;
                                uint32_t code, l;
                                asm("ld.shared.u32 %0, [%1];" : "=r"(code) : "r"(enc_addr + q * 8u + 4u));
                                asm("ld.shared.u8 %0, [%1];" : "=r"(l) : "r"(len8_rel + kMagicBits + q));
                                w.put(code, (int)l);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; i += 2) {
                                const uint32_t word = sym[blk * 4 + i / 4];
                                const uint32_t q0 = (word >> (8 * (i & 3))) & 0xffu, q1 = (word >> (8 * ((i + 1) & 3))) & 0xffu;
                                uint32_t c0, c1, l0, l1;
                                if constexpr (kPerChannel) {
                                    const int j = col0 + blk * 16 + i;
                                    const uint32_t e0 = __ldg(a.enc + j * nsym + q0), e1 = __ldg(a.enc + (j + 1) * nsym + q1);
                                    c0 = e0 >> 8; l0 = e0 & 0xffu; c1 = e1 >> 8; l1 = e1 & 0xffu;
                                } else {
                                    asm("ld.shared.u32 %0, [%1];" : "=r"(c0) : "r"(enc_addr + q0 * 8u + 4u));
                                    asm("ld.shared.u32 %0, [%1];" : "=r"(c1) : "r"(enc_addr + q1 * 8u + 4u));
                                    asm("ld.shared.u8 %0, [%1];" : "=r"(l0) : "r"(len8_rel + kMagicBits + q0));
                                    asm("ld.shared.u8 %0, [%1];" : "=r"(l1) : "r"(len8_rel + kMagicBits + q1));
                                }
                                w.put((c0 << l1) | c1, (int)(l0 + l1));
                            }
                        }
                    }
                }
            };
            if (staged) {
                SmemBitWriter ws;
                ws.init(stg_addr, my_off);
                pack_tile(ws);
                named_bar_sync(bar_id, 256);      // all full words stored
                if (do_pack) ws.finish();
                if (tg == 0) { s_padded[grp] = padded; s_store_cmd[grp] = 1; }
            } else {
                BitWriter wgl;
                wgl.init(a.stream, s_base[grp] + my_off);
                pack_tile(wgl);
                if (do_pack) wgl.finish();
                if (tg == 0) {
                    const unsigned long long base = s_base[grp];
                    a.tile_off[tile] = base;
                    if (tile == a.n_tiles - 1) a.tile_off[a.n_tiles] = base + padded;
                    s_store_cmd[grp] = 2;
                }
            }
            // hand the tile to the store warp (each thread's arrival releases its own writes)
            mbar_arrive(smem_u32(&s_stg_full[grp]));
            ++n_done;
            // chunk lengths: with four chunks per pixel each thread writes the two of its half
            // (one aligned word); otherwise the first half's thread of a pixel writes them
            if (valid && a.splits == 4)
                *reinterpret_cast<uint32_t *>(a.chunk_len + 4 * p + 2 * half) = bits_first | ((my_bits - bits_first) << 16);
            else if (valid && half == 0) {
                if (a.splits == 2)                        // one chunk per half: both lengths in one aligned word
                    *reinterpret_cast<uint32_t *>(a.chunk_len + 2 * p) = my_bits | (other << 16);
                else if (a.chunk_pixels == 1)
                    a.chunk_len[p] = (uint16_t)pair;
                else if ((p % a.chunk_pixels) == 0)
                    a.chunk_len[p / a.chunk_pixels] = (uint16_t)(chunk_end - pixel_off);
            }
        }
        if (!alive) {
            if (tg == 0) { tc_dev_set_status(a.status, TC_ERR_TIMEOUT); s_store_cmd[grp] = 3; }
            mbar_arrive(smem_u32(&s_stg_full[grp]));   // lets the store warp leave
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

// entries of the code table held in shared memory: none (per-channel tables stay in global
// memory), one per symbol, or one per pair of symbols
static int enc_table_entries(const EncodeArgs &a)
{
    if (a.groups != 1) return 0;
    return a.bits <= kPairMaxBits ? (1 << (2 * a.bits)) : (1 << a.bits);
}

bool tc_encode_tc_supported(const tc_ctx *ctx, const EncodeArgs &a)
{
    // K <= C leading components (PCA truncation): K is the N dimension of the MMA
    if (a.c % 16 != 0 || a.k % 16 != 0 || a.k < 16 || a.k > a.c || a.c > 256 || a.hw % 4 != 0) return false;
    // the loaders copy groups of four pixels with 8-byte cp.async: the tensor must start on an 8-byte boundary
    if (((uintptr_t)a.x & 7u) != 0) return false;
    // two chunks per pixel must coincide with the two halves the epilogue threads work on
    // (four chunks: each half splits once more in its middle)
    if (a.splits != 1 && !(a.splits == 2 && a.k % 32 == 0) && !(a.splits == 4 && a.k % 64 == 0 && a.chunk_pixels == 1)) return false;
    if (a.groups != 1 && a.groups != a.k) return false;
    const SmemLayout l = smem_layout(a.c, a.k, enc_table_entries(a));
    return (int)l.total + 512 <= ctx->max_smem_optin;       // leaves room for the static shared variables
}

tc_status tc_launch_encode_tc(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const SmemLayout l = smem_layout(a.c, a.k, enc_table_entries(a));
    const bool per_channel = a.groups != 1, debug = a.dbg_coef || a.dbg_sym, pair = !per_channel && a.bits <= kPairMaxBits;
    if (a.hist && (per_channel || debug)) return TC_ERR_UNSUPPORTED;      // statistics run with a per-layer table
    void (*kernel)(EncodeArgs) =
        a.hist      ? (pair ? encode_tc_kernel<false, false, true, true> : encode_tc_kernel<false, false, false, true>)
        : per_channel ? (debug ? encode_tc_kernel<true, true, false, false> : encode_tc_kernel<true, false, false, false>)
        : pair      ? (debug ? encode_tc_kernel<false, true, true, false> : encode_tc_kernel<false, false, true, false>)
                    : (debug ? encode_tc_kernel<false, true, false, false> : encode_tc_kernel<false, false, false, false>);
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.total) != cudaSuccess)
        return TC_ERR_CUDA;
    const unsigned int grid = (unsigned int)((a.n_tiles < ctx->sm_count) ? a.n_tiles : ctx->sm_count);
    EncodeArgs args = a;
    void *params[] = {&args};
    // cooperative launch: the grid must be co-resident, which is what makes the look-back safe
    const cudaError_t err = cudaLaunchCooperativeKernel((void *)kernel, dim3(grid), dim3(kThreads), params, l.total, s);
    if (err != cudaSuccess) {
        if (getenv("TC_VERBOSE")) fprintf(stderr, "tc: encode launch failed: %s\n", cudaGetErrorString(err));
        cudaGetLastError();
        return TC_ERR_CUDA;
    }
    return TC_OK;
}
