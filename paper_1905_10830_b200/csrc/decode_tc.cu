// Fused tensor-core decode for bf16 tensors (Section 3: VLD, inverse quantiser, inverse
// transform).
//
// One persistent block per SM; two tiles of 128 pixels are in flight at a time.  Warp roles:
//   warps 0-3, 4-7     two VLD groups (alternating tiles): one thread per chunk walks its part
//                      of the bit stream with a table-driven canonical Huffman decoder and
//                      writes the symbols, as exact bf16 integers, into the K-major A operand
//   warps 8-15         epilogue, all eight warps on every tile (two channel halves):
//                      TMEM -> registers, x_hat = step * acc + bias, round to bf16, NCHW stores
//   warps 16, 17       one thread each issues the tcgen05.mma of its group:
//                      D[pixel][c] = (Q[pixel][j] - center) * T[j][c]
// Each VLD group copies the bit-stream segment of its next tile into shared memory (cp.async,
// double-buffered) while it decodes the current one, so that the decoder's refills are
// shared-memory reads; a segment too long for the buffer is read from global memory instead.
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

constexpr int kPanelK = 32;                                   // coefficients per ring stage
constexpr int kStageBytes = kPanelK * TC_TILE_PIXELS * 2;     // 8 KB
constexpr int kThreads = 18 * 32;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kMaxStages = 8;                                 // per group
constexpr int kTransposeBytes = 32 * TC_TILE_PIXELS * 2;      // 32 channels x 128 pixels of bf16
// A chunk that starts inside a staged segment is read for at most chunk_pixels * K codes of 12
// bits, whatever the bits say; the slack after each buffer keeps those reads inside the block's
// shared memory even for a corrupt stream (the buffers lie back to back, the slack follows the
// last one).  Chunks longer than the slack allows are not staged.
constexpr int kStreamSlack = 1024;

struct SmemLayout {
    uint32_t basis, ring, lut, bias, sbuf, tbuf, total;
    int stages;                                               // ring stages per group
    uint32_t stream_buf;                                      // bytes per staged stream buffer (4 buffers), 0 = none
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
    l.tbuf = l.ring + 2u * (uint32_t)want * kStageBytes;          // two 8 KB transpose buffers (epilogue)
    l.sbuf = l.tbuf + 2u * kTransposeBytes;
    l.stream_buf = 0;
    // four stream buffers back to back (an overrun of one lands in the next), one slack area at the end
    for (uint32_t kb = 12; kb >= 3; --kb)
        if ((long long)l.sbuf + 4ll * kb * 1024 + kStreamSlack <= (long long)budget) { l.stream_buf = kb * 1024; break; }
    l.total = l.sbuf + (l.stream_buf ? 4u * l.stream_buf + kStreamSlack : 0u);
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

// The same reader over a segment staged in shared memory.  The word after the window is kept
// in a register, so that the shared-memory load of a refill is off the critical path, and the
// refill is predicated rather than branched.
struct SmemWindowReader {
    uint32_t next_addr;               // shared address of the word after `ahead`
    uint32_t hi, lo, ahead;
    int avail;

    __device__ __forceinline__ static uint32_t lds(uint32_t addr)
    {
        uint32_t v;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
        return v;
    }
    // `bitpos` is relative to the start of the staged segment at shared address `seg_addr`
    __device__ __forceinline__ void init(uint32_t seg_addr, uint32_t bitpos)
    {
        const uint32_t a0 = seg_addr + (bitpos >> 5) * 4u;
        const uint32_t w0 = lds(a0), w1 = lds(a0 + 4);
        ahead = lds(a0 + 8);
        next_addr = a0 + 12;
        const int sh = (int)(bitpos & 31u);
        hi = __funnelshift_l(w1, w0, sh);
        lo = w1 << sh;
        avail = 64 - sh;
    }
    __device__ __forceinline__ uint32_t peek(int nbits) const { return hi >> (32 - nbits); }
    // the shift takes its amount modulo 32: a table entry with the length in its low 5 bits
    // can be passed as it is
    __device__ __forceinline__ void skip_entry(uint32_t e)
    {
        hi = __funnelshift_l(lo, hi, e);
        lo = __funnelshift_l(0u, lo, e);
        avail -= (int)(e & 31u);
    }
    // nbits < 32
    __device__ __forceinline__ void skip_bits(int nbits)
    {
        hi = __funnelshift_l(lo, hi, nbits);
        lo <<= nbits;
        avail -= nbits;
    }
    __device__ __forceinline__ void refill()
    {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b32 s, t;\n\t"
            "setp.le.s32 p, %3, 32;\n\t"
            "sub.s32 s, 32, %3;\n\t"
            "shf.l.wrap.b32 t, %2, 0, s;\n\t"
            "@p or.b32 %0, %0, t;\n\t"
            "shl.b32 t, %2, s;\n\t"
            "@p or.b32 %1, %1, t;\n\t"
            "@p add.s32 %3, %3, 32;\n\t"
            "@p ld.shared.u32 %2, [%4];\n\t"
            "@p add.s32 %4, %4, 4;\n\t}"
            : "+r"(hi), "+r"(lo), "+r"(ahead), "+r"(avail), "+r"(next_addr));
    }
    // bits consumed since init(seg_addr, bitpos)
    __device__ __forceinline__ uint32_t consumed(uint32_t seg_addr, uint32_t bitpos) const
    {
        const uint32_t a0 = seg_addr + (bitpos >> 5) * 4u;
        return (next_addr - 4u - a0) * 8u - (bitpos & 31u) - (uint32_t)avail;
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
    constexpr int pair_size = 1 << TC_PAIR_LUT_BITS;
    const SmemLayout L = smem_layout(a.c, a.k, kPerChannel ? 0 : 2 * pair_size, a.chunk_pixels, a.smem_budget);
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
            mbar_init(smem_u32(&s_tempty[g]), 256);
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
            for (int i = tid; i < pair_size; i += kThreads) {
                // pair table entry: x = bf16(symbol0 - center) | bf16(symbol1 - center) << 16,
                //                   y = bits consumed | symbols decoded << 8 | length of the first code << 16
                const uint2 e = a.lut_pair[i];
                const float f0 = (float)((int)(e.x & 0xffu) - a.center), f1 = (float)((int)((e.x >> 8) & 0xffu) - a.center);
                s_lut[2 * i] = (__float_as_uint(f0) >> 16) | (__float_as_uint(f1) & 0xffff0000u);
                s_lut[2 * i + 1] = e.y;
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
        const uint32_t sbuf_bytes = L.stream_buf;
        const uint32_t sbuf_g = smem_u32(smem + L.sbuf) + (uint32_t)grp * 2u * sbuf_bytes;
        const int bar_id = 1 + grp;
        long long it = 0;                       // panels produced by this group so far
        bool alive = true;

        // offsets of a tile, validated; a tile that cannot be valid decodes nothing
        struct TileInfo { unsigned long long base, bits; bool ok, staged; unsigned int chunk_off; };
        auto tile_info = [&](long long tl) {
            TileInfo ti{0, 0, false, false, 0};
            if (tl >= my_tiles) return ti;
            const long long tile = blockIdx.x + tl * gridDim.x;
            const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
            ti.ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
            if (!ti.ok) return ti;
            ti.base = base;
            ti.bits = end - base;
            ti.staged = sbuf_bytes != 0 && ti.bits <= (unsigned long long)sbuf_bytes * 8ull &&
                        (cp * a.k * TC_MAX_CODE_LEN) / 8 + 16 <= kStreamSlack;
            const long long ch = tile * chunks_per_tile + t;
            if (t < chunks_per_tile && ch < a.n_chunks) ti.chunk_off = a.chunk_off[ch];
            return ti;
        };
        // start the copy of a tile's segment into stream buffer `which` (16 bytes per cp.async)
        auto stage_tile = [&](const TileInfo &ti, int which) {
            if (ti.ok && ti.staged) {
                const uint32_t dst = sbuf_g + (uint32_t)which * sbuf_bytes;
                const unsigned char *src = reinterpret_cast<const unsigned char *>(a.stream) + (ti.base >> 3);
                const uint32_t n16 = (uint32_t)(ti.bits >> 7);
                for (uint32_t i = t; i < n16; i += 128) cp_async_16(dst + i * 16u, src + (size_t)i * 16u, 16u);
            }
            cp_async_commit();
        };

        TileInfo cur = tile_info(grp), nxt = tile_info(grp + 2);
        stage_tile(cur, 0);
        int li = 0;
        for (long long tl = grp; tl < my_tiles && alive; tl += 2, ++li) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            stage_tile(nxt, (li + 1) & 1);           // its buffer was released by the barrier that ended tile li - 1
            cp_async_wait<1>();
            named_bar_sync(bar_id, 128);             // every thread's part of this tile's segment has landed
            const TileInfo after = tile_info(tl + 4); // offsets two tiles ahead: their latency hides behind the decode

            const long long ch = tile * chunks_per_tile + t;
            bool active = cur.ok && t < chunks_per_tile && ch < a.n_chunks;
            bool bad = !cur.ok;
            if (active && (unsigned long long)cur.chunk_off > cur.bits) { bad = true; active = false; }
            const int n_pix = active ? (int)min((long long)cp, a.pixels - (tile * TC_TILE_PIXELS + (long long)t * cp)) : 0;
            const uint32_t seg_addr = sbuf_g + (uint32_t)(li & 1) * sbuf_bytes;

            // walks this thread's chunk; `fill_panel(dst, k0, nk8)` decodes the next 8 * nk8 symbols
            // (coefficients k0 ...) into the operand row at shared address `dst`
            auto decode_chunk = [&](auto &&fill_panel) {
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
                            fill_panel(dst, k0, nk8);
                        }
                        if (pp == cp - 1) {
                            fence_proxy_async_smem();
                            mbar_arrive(smem_u32(&s_full[grp][s]));
                        }
                    }
                }
            };
            // symbol by symbol: eight symbols -> one 16-byte store
            auto by_pairs = [&](auto &&next_pair) {
                return [&, next_pair](uint32_t dst, int k0, int nk8) mutable {
                    for (int k8 = 0; k8 < nk8; ++k8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int i = 0; i < 8; i += 2) pk[i >> 1] = next_pair(k0 + k8 * 8 + i);
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + k8 * 2048), "r"(pk[0]),
                                     "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    }
                };
            };
            // table entry: bf16(symbol - center) << 16 | symbol << 8 | length; returns two bf16 values
            auto centre = [&](uint32_t e) { return __float_as_uint((float)((int)((e >> 8) & 0xffu) - a.center)); };

            if (cur.ok && cur.staged) {
                SmemWindowReader r;
                if (active) r.init(seg_addr, cur.chunk_off);
                else { r.hi = r.lo = r.ahead = 0; r.avail = 64; r.next_addr = seg_addr; }
                auto next_pair = [&](int j) -> uint32_t {
                    r.refill();
                    uint32_t e0, e1;
                    if constexpr (!kPerChannel) {
                        // both symbols from one lookup when their codes fit a 10-bit window
                        uint32_t v, meta;
                        asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v), "=r"(meta) : "r"(lut_addr + r.peek(TC_PAIR_LUT_BITS) * 8u));
                        if (((meta >> 8) & 3u) == 2u) {
                            r.skip_entry(meta);
                            return v;
                        }
                        // one symbol at a time: the first symbol of a pair entry, or, for the rare
                        // code longer than the window, the full table in global memory
                        auto one = [&](uint32_t vv, uint32_t mm) -> uint32_t {
                            if (((mm >> 8) & 3u) != 0u) {
                                r.skip_entry(mm >> 16);
                                return vv << 16;                      // bf16 bits in the upper half, as in lut32
                            }
                            const uint32_t e = __ldg(a.lut32 + r.peek(a.lut_bits));
                            r.skip_entry(e);
                            return centre(e);
                        };
                        const uint32_t h0 = one(v, meta);
                        asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v), "=r"(meta) : "r"(lut_addr + r.peek(TC_PAIR_LUT_BITS) * 8u));
                        const uint32_t h1 = one(v, meta);
                        return __byte_perm(h0, h1, 0x7632);
                    } else {
                        e0 = __ldg(a.lut32 + (size_t)j * lut_size + r.peek(a.lut_bits));
                        r.skip_entry(e0);
                        e1 = __ldg(a.lut32 + (size_t)(j + 1) * lut_size + r.peek(a.lut_bits));
                        r.skip_entry(e1);
                    }
                    return __byte_perm(centre(e0), centre(e1), 0x7632);
                };
                if (!kPerChannel && a.run_shift >= 0) {
                    // The shortest code is all zeros (canonical order), and at low rates it belongs to
                    // the symbol that nearly every coefficient of the trailing channels takes.  Eight
                    // such symbols in a row are 8 (or 16) zero bits: one test replaces eight lookups.
                    const uint32_t fill = a.run_fill;              // bf16(that symbol - center) twice
                    const int bits8 = 8 << a.run_shift;            // bits of eight shortest codes
                    decode_chunk([&](uint32_t dst, int k0, int nk8) {
                        for (int k8 = 0; k8 < nk8; ++k8) {
                            uint32_t pk[4];
                            r.refill();
                            if ((r.hi >> (32 - bits8)) == 0u) {
                                r.skip_bits(bits8);
                                pk[0] = pk[1] = pk[2] = pk[3] = fill;
                            } else {
#pragma unroll
                                for (int i = 0; i < 8; i += 2) pk[i >> 1] = next_pair(k0 + k8 * 8 + i);
                            }
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + k8 * 2048), "r"(pk[0]),
                                         "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                        }
                    });
                } else {
                    decode_chunk(by_pairs(next_pair));
                }
                if (active && (unsigned long long)cur.chunk_off + r.consumed(seg_addr, cur.chunk_off) > cur.bits) bad = true;
            } else {
                WindowReader r;
                unsigned long long used = cur.base + cur.chunk_off;
                if (active) r.init(a.stream, used, cur.base + cur.bits);
                else { r.words = a.stream; r.next = r.end = 0; r.hi = r.lo = 0; r.avail = 64; }
                decode_chunk(by_pairs([&](int j) -> uint32_t {
                    r.refill();
                    const size_t tbl = kPerChannel ? (size_t)j * lut_size : 0, tbl1 = kPerChannel ? (size_t)(j + 1) * lut_size : 0;
                    const uint32_t e0 = __ldg(a.lut32 + tbl + r.peek(a.lut_bits));
                    r.skip((int)(e0 & 0xffu));
                    const uint32_t e1 = __ldg(a.lut32 + tbl1 + r.peek(a.lut_bits));
                    r.skip((int)(e1 & 0xffu));
                    used += (e0 & 0xffu) + (e1 & 0xffu);
                    return __byte_perm(centre(e0), centre(e1), 0x7632);
                }));
                if (active && used > cur.base + cur.bits) bad = true;
            }
            it += n_panels;
            if (bad) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
            named_bar_sync(bar_id, 128);             // this tile's stream buffer may be refilled
            cur = nxt;
            nxt = after;
        }
        cp_async_wait<0>();
        if (!alive && t == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else if (warp < 16) {
        // ================= epilogue: all eight warps work on every tile =================
        // warps 8-11 store the first half of the channels, warps 12-15 the second half, so that an
        // accumulator is released after half the store time and the VLD group behind it stalls less
        const int half = (warp - 8) >> 2;
        const int wq = warp & 3;
        const int m = wq * 32 + lane;                       // pixel within the tile = TMEM lane
        const int half_cols = ((a.c + 31) / 32) * 16;
        const int col0 = half * half_cols;
        const int ncols = half ? a.c - half_cols : half_cols;   // multiple of 16
        const float step = (float)a.step;
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.xhat);
        // With H*W a multiple of 4 every aligned group of four pixels lies inside one image and is
        // 8-byte aligned: 32 channels x 128 pixels are transposed through shared memory and leave
        // as one 256-byte row per warp store.  Otherwise each lane stores its own 2-byte values.
        const bool vec = (a.hw & 3) == 0;
        const uint32_t tb_addr = smem_u32(smem + L.tbuf) + (uint32_t)half * kTransposeBytes;
        const int ebar = 3 + half;
        bool alive = true;
        for (long long tl = 0; tl < my_tiles && alive; ++tl) {
            const int grp = (int)(tl & 1);
            const long long tile = blockIdx.x + tl * gridDim.x;
            const long long p = tile * TC_TILE_PIXELS + m;
            const bool valid = p < a.pixels;
            const long long img = valid ? p / a.hw : 0;
            __nv_bfloat16 *dst = out + img * a.c * (long long)a.hw + (valid ? p - img * a.hw : 0) + (long long)col0 * a.hw;
            // the four pixels this lane stores in the transposed phase
            const long long p4 = tile * TC_TILE_PIXELS + 4 * lane;
            const bool valid4 = p4 < a.pixels;
            const long long img4 = valid4 ? p4 / a.hw : 0;
            __nv_bfloat16 *dst4 = out + img4 * a.c * (long long)a.hw + (valid4 ? p4 - img4 * a.hw : 0) + (long long)col0 * a.hw;
            if (!mbar_wait(smem_u32(&s_tfull[grp]), (uint32_t)((tl >> 1) & 1))) { alive = false; break; }
            tc_fence_after_sync();
            const uint32_t trow = tmem_base + grp * kAccCols + ((uint32_t)(wq * 32) << 16) + col0;
            for (int c0 = 0; c0 < ncols; c0 += 32) {
                const int nc = min(32, ncols - c0);            // 32 or 16
                uint32_t r[32];
                {
                    uint32_t r16[16];
                    tmem_ld_32x32b_x16(trow + c0, r16);
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = r16[i];
                    if (nc == 32) {
                        tmem_ld_32x32b_x16(trow + c0 + 16, r16);
#pragma unroll
                        for (int i = 0; i < 16; ++i) r[16 + i] = r16[i];
                    }
                }
                tmem_ld_wait();
                if (vec) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        if (i < nc) {
                            const float v0 = fmaf(__uint_as_float(r[i]), step, s_bias[col0 + c0 + i]);
                            const float v1 = fmaf(__uint_as_float(r[i + 1]), step, s_bias[col0 + c0 + i + 1]);
                            const __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                            const uint32_t hb = *reinterpret_cast<const uint32_t *>(&h);
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(tb_addr + i * 256 + m * 2), "h"((unsigned short)(hb & 0xffffu)) : "memory");
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(tb_addr + (i + 1) * 256 + m * 2), "h"((unsigned short)(hb >> 16)) : "memory");
                        }
                    }
                    named_bar_sync(ebar, 128);                 // the block is in shared memory
                    for (int ch = wq; ch < nc; ch += 4) {      // one channel row of 128 pixels per warp store
                        uint32_t lo2, hi2;
                        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(lo2), "=r"(hi2) : "r"(tb_addr + ch * 256 + lane * 8));
                        if (valid4) *reinterpret_cast<uint2 *>(dst4 + (long long)(c0 + ch) * a.hw) = make_uint2(lo2, hi2);
                    }
                    named_bar_sync(ebar, 128);                 // the buffer may be overwritten
                } else if (valid) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        if (i < nc) {
                            const float v0 = fmaf(__uint_as_float(r[i]), step, s_bias[col0 + c0 + i]);
                            const float v1 = fmaf(__uint_as_float(r[i + 1]), step, s_bias[col0 + c0 + i + 1]);
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
        if (!alive && lane == 0 && wq == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
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
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (2 << TC_PAIR_LUT_BITS) : 0, a.chunk_pixels,
                                     ctx->max_smem_optin - 512);
    return l.stages > 0;
}

tc_status tc_launch_decode_tc(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (2 << TC_PAIR_LUT_BITS) : 0, a.chunk_pixels,
                                     ctx->max_smem_optin - 512);
    if (l.stages == 0) return TC_ERR_UNSUPPORTED;
    void (*kernel)(DecodeArgs) = a.groups != 1 ? decode_tc_kernel<true> : decode_tc_kernel<false>;
    DecodeArgs args = a;
    args.smem_budget = ctx->max_smem_optin - 512;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.total) != cudaSuccess)
        return TC_ERR_CUDA;
    const unsigned int grid = (unsigned int)((a.n_tiles < ctx->sm_count) ? a.n_tiles : ctx->sm_count);
    kernel<<<grid, kThreads, l.total, s>>>(args);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
