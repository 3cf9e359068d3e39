// Fused tensor-core decode for bf16 tensors (Section 3: VLD, inverse quantiser, inverse
// transform).
//
// One persistent block per SM; two tiles of 128 pixels are in flight at a time.  Warp roles:
//   warps 0-7, 8-15    two VLD groups (alternating tiles): one thread per chunk walks its part
//                      of the bit stream with a table-driven canonical Huffman decoder and
//                      writes the symbols, as exact bf16 integers, into the K-major A operand.
//                      With two chunks per pixel (pixel_splits = 2) warps 0-3 of a group decode
//                      the first half of the coefficients and warps 4-7 the second half, each
//                      half feeding its own two-slot ring of 16-coefficient panels; otherwise
//                      only warps 0-3 of a group work.
//   warps 16-23        epilogue, all eight warps on every tile: TMEM -> registers,
//                      x_hat = step * acc + bias, round to bf16, NCHW stores.  The accumulator is
//                      held transposed (TMEM lane = channel, column = pixel): a thread owns one
//                      channel and gets 16 consecutive pixels per TMEM load; each warp turns its
//                      32 channels x 32 pixels through a private shared-memory block (16-byte
//                      writes, no block barrier) so that every channel row leaves as 64
//                      contiguous bytes.
//   warps 24, 25       one thread each issues the tcgen05.mma of its group, one per block of 128
//                      channels:  D[c][pixel] = T[j][c] * (Q[pixel][j] - center)
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

constexpr int kVldWarps = 16, kEpiWarp0 = 16, kMmaWarp0 = 24;
constexpr int kThreads = 26 * 32;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kMaxSlots = 8;                                  // ring slots per group
// A chunk that starts inside a staged segment is read for at most chunk_pixels * K codes of 12
// bits, whatever the bits say; the slack after each buffer keeps those reads inside the block's
// shared memory even for a corrupt stream (the buffers lie back to back, the slack follows the
// last one).  Chunks longer than the slack allows are not staged.
constexpr int kStreamSlack = 1024;
// Epilogue transpose block of one warp: 32 channel rows of 32 pixels (64 bytes) with 16 bytes
// of padding, which keeps both the 16-byte row writes and the 8-byte reads spread over the banks.
constexpr int kTrRowBytes = 80;
constexpr int kTrWarpBytes = 32 * kTrRowBytes;

struct SmemLayout {
    uint32_t basis, ring, lut, tbuf, sbuf, total;
    int slots;                                                // ring slots per group (0: does not fit)
    int panel_k;                                              // coefficients per ring slot
    uint32_t slot_bytes;
    uint32_t stream_buf;                                      // bytes per staged stream buffer (4 buffers), 0 = none
};

__host__ __device__ inline SmemLayout smem_layout(int c, int k, int lut_entries, int chunk_pixels, int splits, int budget)
{
    SmemLayout l;
    l.basis = 0;
    const int c_pad = ((c + 127) / 128) * 128;                // the MMA takes 128 channels at a time
    l.lut = (uint32_t)(((size_t)c_pad * k * 2 + 1023) & ~(size_t)1023);
    l.ring = (l.lut + (uint32_t)lut_entries * 4 + 1023) & ~1023u;
    // Two chunks per pixel: each half of the coefficients streams through its own two slots of
    // 16 coefficients.  One chunk per pixel: two slots of 32 coefficients.  A chunk of several
    // pixels is decoded pixel by pixel, so every panel of the tile has to stay resident until
    // the chunk's last pixel is done.
    l.panel_k = splits == 2 ? 16 : 32;
    l.slot_bytes = (uint32_t)l.panel_k * TC_TILE_PIXELS * 2;
    const int n_panels = (k + l.panel_k - 1) / l.panel_k;
    int want = splits == 2 ? 4 : (chunk_pixels > 1 ? n_panels : 2);
    if (want < 2) want = 2;
    l.slots = want;
    l.tbuf = l.ring + 2u * (uint32_t)want * l.slot_bytes;         // eight warp-private transpose blocks (epilogue)
    l.sbuf = l.tbuf + 8u * kTrWarpBytes;
    l.stream_buf = 0;
    // four stream buffers back to back (an overrun of one lands in the next), one slack area at the end
    for (uint32_t kb = 16; kb >= 3; --kb)
        if ((long long)l.sbuf + 4ll * kb * 1024 + kStreamSlack <= (long long)budget) { l.stream_buf = kb * 1024; break; }
    l.total = l.sbuf + (l.stream_buf ? 4u * l.stream_buf + kStreamSlack : 0u);
    if ((int)l.total > budget || want > kMaxSlots) l.slots = 0;
    return l;
}

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

// Branch-free reader for per-layer tables held in shared memory.  The window hi:lo holds the
// next 64 - c stream bits left-aligned, where c (the low bits of `used`) counts the bits taken
// since the last refill; a table entry carries its code length in bits 0-7, zeros in bits 8-15
// and the decoded value in bits 16-31, so that `used += entry` counts bits without a mask and
// the funnel shifts (which take their amount modulo 32) can be fed the entry as it is.
// refill() runs once per two symbols: codes are at most 12 bits, so that after it c < 32, the
// first symbol sees at least 33 valid bits and the second at least 21.
struct SmemSymbolReader {
    uint32_t next_addr;               // shared address of the word after `ahead`
    uint32_t hi, lo, ahead;
    uint32_t used;                    // low 8 bits: c

    __device__ __forceinline__ static uint32_t lds(uint32_t addr)
    {
        uint32_t v;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
        return v;
    }
    __device__ __forceinline__ void init(uint32_t seg_addr, uint32_t bitpos)
    {
        const uint32_t a0 = seg_addr + (bitpos >> 5) * 4u;
        const uint32_t w0 = lds(a0), w1 = lds(a0 + 4);
        ahead = lds(a0 + 8);
        next_addr = a0 + 12;
        const int sh = (int)(bitpos & 31u);
        hi = __funnelshift_l(w1, w0, sh);
        lo = w1 << sh;
        used = (uint32_t)sh;
    }
    __device__ __forceinline__ void idle(uint32_t seg_addr)
    {
        hi = lo = ahead = 0;
        used = 0;
        next_addr = seg_addr;
    }
    __device__ __forceinline__ uint32_t peek(int nbits) const { return hi >> (32 - nbits); }
    __device__ __forceinline__ void take(uint32_t entry)
    {
        hi = __funnelshift_l(lo, hi, entry);
        lo = __funnelshift_l(0u, lo, entry);
        used += entry;
    }
    __device__ __forceinline__ void refill()
    {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b32 t, u;\n\t"
            "and.b32 t, %3, 32;\n\t"
            "setp.ne.u32 p, t, 0;\n\t"
            "shf.l.wrap.b32 t, %2, 0, %3;\n\t"     // ahead >> (32 - (c - 32)); the shifts take c modulo 32
            "shf.l.wrap.b32 u, 0, %2, %3;\n\t"     // ahead << (c - 32)
            "@p or.b32 %0, %0, t;\n\t"
            "@p or.b32 %1, %1, u;\n\t"
            "@p add.u32 %3, %3, -32;\n\t"
            "@p ld.shared.u32 %2, [%4];\n\t"
            "@p add.u32 %4, %4, 4;\n\t}"
            : "+r"(hi), "+r"(lo), "+r"(ahead), "+r"(used), "+r"(next_addr));
    }
    // bits consumed since init(seg_addr, bitpos)
    __device__ __forceinline__ uint32_t consumed(uint32_t seg_addr, uint32_t bitpos) const
    {
        const uint32_t a0 = seg_addr + (bitpos >> 5) * 4u;
        return (next_addr - 12u - a0) * 8u + (used & 0xffu) - (bitpos & 31u);
    }
};

template <bool kPerChannel>
__global__ void __launch_bounds__(kThreads, 1) decode_tc_kernel(DecodeArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_full[2][kMaxSlots], s_empty[2][kMaxSlots], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    // [group][tile parity][half][warp]: chunk bits per warp, for the start positions.  Two copies: a warp
    // that is done with its tile early writes the next tile's sum while a slower warp may still be
    // reading this tile's; the group's barriers only order the write after next.
    __shared__ unsigned int s_wsum[2][2][2][4];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lut_size = 1 << a.lut_bits;
    const int S = a.splits;                      // chunks per pixel: 1 or 2
    const SmemLayout L = smem_layout(a.c, a.k, kPerChannel ? 0 : lut_size, a.chunk_pixels, S, a.smem_budget);
    const int slots = L.slots, panel_k = L.panel_k;
    const uint32_t slot_bytes = L.slot_bytes;
    unsigned char *s_basis = smem + L.basis;
    uint32_t *s_lut = reinterpret_cast<uint32_t *>(smem + L.lut);
    const uint32_t ring_addr = smem_u32(smem + L.ring);
    const uint32_t basis_addr = smem_u32(s_basis);
    const uint32_t lut_addr = smem_u32(s_lut);
    const int k_sub = a.k / S;                   // coefficients per chunk of one pixel
    const int n_panels = (k_sub + panel_k - 1) / panel_k;       // panels per half (S = 2) or per pixel

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int g = 0; g < 2; ++g) {
            for (int s = 0; s < kMaxSlots; ++s) { mbar_init(smem_u32(&s_full[g][s]), 128); mbar_init(smem_u32(&s_empty[g][s]), 1); }
            mbar_init(smem_u32(&s_tfull[g]), 1);
            mbar_init(smem_u32(&s_tempty[g]), 256);
        }
        mbar_fence_init();
    }
    if (warp == kMmaWarp0) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    {
        // transposed basis [c][j] -> K-major core matrices: (c/8)*sbo + (j/8)*128 + (c%8)*16 + (j%8)*2
        const uint32_t sbo = (uint32_t)(a.k / 8) * 128u;
        const int chunks_per_row = a.k / 8;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.basis_t_bf16);
        const int c_pad = ((a.c + 127) / 128) * 128;         // rows past C are zero: their outputs are never stored
        // (asynchronous copies: all of a thread's pieces are in flight at once; a copy of zero
        // source bytes fills its 16 bytes with zeros)
        for (int i = tid; i < c_pad * chunks_per_row; i += kThreads) {
            const int ch = i / chunks_per_row, j8 = i - ch * chunks_per_row;
            cp_async_16(basis_addr + (ch >> 3) * sbo + j8 * 128 + (ch & 7) * 16, ch < a.c ? src + i : src, ch < a.c ? 16u : 0u);
        }
        cp_async_commit();
        if (!kPerChannel)
            for (int i = tid; i < lut_size; i += kThreads) {
                // per-layer table: bf16(symbol - center) << 16 | code length
                const uint32_t e = a.lut32[i];
                const float f = (float)((int)((e >> 8) & 0xffu) - a.center);
                s_lut[i] = (__float_as_uint(f) & 0xffff0000u) | (e & 0xffu);
            }
    }
    cp_async_wait<0>();
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    const long long my_tiles = (a.n_tiles > blockIdx.x) ? (a.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp < kVldWarps) {
        // ================= VLD groups =================
        const int grp = warp >> 3;
        const int tg = tid & 255;                // thread within the group
        const int sub = S == 2 ? (tg >> 7) : 0;  // which half of the coefficients (warp-uniform)
        const int t = tg & 127;                  // S = 2: pixel within the tile; S = 1: chunk within the tile
        const int wq = t >> 5;
        const int cp = a.chunk_pixels;
        const int chunks_per_tile = S * TC_TILE_PIXELS / cp;
        const int n_thr = 128 * S;               // working threads of the group
        const bool working = tg < n_thr;
        const uint32_t ring_g = ring_addr + (uint32_t)grp * slots * slot_bytes;
        const uint32_t sbuf_bytes = L.stream_buf;
        const uint32_t sbuf_g = smem_u32(smem + L.sbuf) + (uint32_t)grp * 2u * sbuf_bytes;
        const int bar_id = 1 + grp;
        const int sub_slots = S == 2 ? 2 : slots; // ring slots of this thread's half
        // ring position of this thread's half at the start of a tile: slot and phase parity of
        // the next panel (kept incrementally: a division per panel would cost more than the decode)
        int slot0 = 0;
        uint32_t phase0 = 0;
        bool alive = true;

        // offsets of a tile, validated; a tile that cannot be valid decodes nothing.  `lens` holds
        // the chunk length(s) of this thread's pixel: both halves (S = 2) or the one chunk.
        // A segment of up to one stream buffer is copied while the tile before it is decoded; a
        // `big` one (up to two buffers) takes both buffers of the group and is copied when its own
        // turn comes; anything larger is read from global memory.
        struct TileInfo { unsigned long long base, bits; bool ok, staged, big; unsigned int lens; };
        auto tile_info = [&](long long tl) {
            TileInfo ti{0, 0, false, false, false, 0};
            if (tl >= my_tiles) return ti;
            const long long tile = blockIdx.x + tl * gridDim.x;
            const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
            ti.ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
            if (!ti.ok) return ti;
            ti.base = base;
            ti.bits = end - base;
            ti.staged = sbuf_bytes != 0 && ti.bits <= (unsigned long long)sbuf_bytes * 16ull &&
                        (cp * k_sub * TC_MAX_CODE_LEN) / 8 + 16 <= kStreamSlack;
            ti.big = ti.staged && ti.bits > (unsigned long long)sbuf_bytes * 8ull;
            if (S == 2) {
                const long long ch = tile * chunks_per_tile + 2 * t;     // even: both lengths in one aligned word
                if (ch < a.n_chunks) ti.lens = *reinterpret_cast<const unsigned int *>(a.chunk_len + ch);
            } else {
                const long long ch = tile * chunks_per_tile + t;
                if (t < chunks_per_tile && ch < a.n_chunks) ti.lens = a.chunk_len[ch];
            }
            return ti;
        };
        // start the copy of a tile's segment into stream buffer `which` (16 bytes per cp.async)
        auto stage_tile = [&](const TileInfo &ti, int which) {
            if (ti.ok && ti.staged) {
                const uint32_t dst = sbuf_g + (uint32_t)which * sbuf_bytes;
                const unsigned char *src = reinterpret_cast<const unsigned char *>(a.stream) + (ti.base >> 3);
                const uint32_t n16 = (uint32_t)(ti.bits >> 7);
                for (uint32_t i = tg; i < n16; i += n_thr) cp_async_16(dst + i * 16u, src + (size_t)i * 16u, 16u);
            }
            cp_async_commit();
        };

        // (with one chunk per pixel or fewer, warps 4-7 of a group have nothing to do)
        TileInfo cur{0, 0, false, false, false, 0}, nxt = cur;
        if (working) {
            cur = tile_info(grp);
            nxt = tile_info(grp + 2);
        }
        int li = 0;
        bool cur_copied = false;                     // the copy of `cur` was started one tile earlier
        for (long long tl = grp; tl < my_tiles && alive && working; tl += 2, ++li) {
            const long long tile = blockIdx.x + tl * gridDim.x;
            const int cur_buf = cur.big ? 0 : (li & 1);
            if (!cur_copied) stage_tile(cur, cur_buf);
            // the next tile's buffer was released by the barrier that ended tile li - 1; no copy
            // ahead while this tile or the next needs both buffers
            const bool ahead = !cur.big && !nxt.big;
            if (ahead) {
                stage_tile(nxt, (li + 1) & 1);
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            // start of every chunk = sum of the lengths before it in the tile (chunk order: pixel,
            // then half): scan over the pixels' totals; both halves of a group compute the same scan
            const unsigned int len0 = S == 2 ? (cur.lens & 0xffffu) : cur.lens, len1 = S == 2 ? (cur.lens >> 16) : 0u;
            const unsigned int tot = len0 + len1;
            unsigned int inc = tot;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += up;
            }
            if (lane == 31) s_wsum[grp][li & 1][sub][wq] = inc;
            named_bar_sync(bar_id, n_thr);           // every thread's part of this tile's segment has landed
            const TileInfo after = tile_info(tl + 4); // offsets two tiles ahead: their latency hides behind the decode
            unsigned int before = 0, tile_total = 0;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const unsigned int sw = s_wsum[grp][li & 1][sub][w];
                if (w < wq) before += sw;
                tile_total += sw;
            }
            const unsigned int chunk_start = before + inc - tot + (sub ? len0 : 0u);
            const unsigned int chunk_bits = sub ? len1 : len0;

            const long long ch = tile * chunks_per_tile + (S == 2 ? 2 * t + sub : t);
            bool active = cur.ok && (S == 2 || t < chunks_per_tile) && ch < a.n_chunks;
            bool bad = !cur.ok || (unsigned long long)tile_total > cur.bits;
            if (bad) active = false;
            const int n_pix = active ? (int)min((long long)cp, a.pixels - (tile * TC_TILE_PIXELS + (S == 2 ? (long long)t : (long long)t * cp))) : 0;
            const uint32_t seg_addr = sbuf_g + (uint32_t)cur_buf * sbuf_bytes;
            const int k_first = sub * k_sub, k_end = k_first + k_sub;

            // walks this thread's chunk; `fill_panel(dst, k0, nk8)` decodes the next 8 * nk8 symbols
            // (coefficients k0 ...) into the operand row at shared address `dst`
            auto decode_chunk = [&](auto &&fill_panel) {
                for (int pp = 0; pp < cp && alive; ++pp) {
                    const bool decode = pp < n_pix;
                    const int row = t * cp + pp;       // only meaningful while the chunk exists
                    int slot = slot0;
                    uint32_t phase = phase0;
                    for (int kp = 0; kp < n_panels; ++kp) {
                        const int s = sub * 2 + slot;
                        if (pp == 0 && !mbar_wait(smem_u32(&s_empty[grp][s]), phase ^ 1u, 200u)) { alive = false; break; }
                        if (++slot == sub_slots) { slot = 0; phase ^= 1u; }
                        if (decode) {
                            const int k0 = k_first + kp * panel_k;
                            const int nk8 = min(panel_k, k_end - k0) >> 3;
                            const uint32_t dst = ring_g + s * slot_bytes + (row >> 3) * 128 + (row & 7) * 16;
                            fill_panel(dst, k0, nk8);
                        }
                        // (the issuing thread makes the panel visible to the tensor core's proxy)
                        if (pp == cp - 1) mbar_arrive(smem_u32(&s_full[grp][s]));
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

            if (!kPerChannel && cur.ok && cur.staged) {
                // per-layer table in shared memory: one lookup per symbol and no branch, so that the
                // 32 lanes of a warp stay in step whatever their bits are
                SmemSymbolReader r;
                if (active) r.init(seg_addr, chunk_start);
                else r.idle(seg_addr);
                const int lb = a.lut_bits;
                decode_chunk([&](uint32_t dst, int k0, int nk8) {
                    for (int k8 = 0; k8 < nk8; ++k8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            r.refill();
                            const uint32_t e0 = SmemSymbolReader::lds(lut_addr + (r.peek(lb) << 2));
                            r.take(e0);
                            const uint32_t e1 = SmemSymbolReader::lds(lut_addr + (r.peek(lb) << 2));
                            r.take(e1);
                            pk[i] = __byte_perm(e0, e1, 0x7632);
                        }
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + k8 * 2048), "r"(pk[0]),
                                     "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    }
                });
                // a chunk must end exactly where its recorded length says
                if (active && r.consumed(seg_addr, chunk_start) != chunk_bits) bad = true;
            } else if (cur.ok && cur.staged) {
                // per-channel tables (global memory), stream from shared memory
                SmemWindowReader r;
                if (active) r.init(seg_addr, chunk_start);
                else { r.hi = r.lo = r.ahead = 0; r.avail = 64; r.next_addr = seg_addr; }
                decode_chunk(by_pairs([&](int j) -> uint32_t {
                    r.refill();
                    const uint32_t e0 = __ldg(a.lut32 + (size_t)j * lut_size + r.peek(a.lut_bits));
                    r.skip_entry(e0);
                    const uint32_t e1 = __ldg(a.lut32 + (size_t)(j + 1) * lut_size + r.peek(a.lut_bits));
                    r.skip_entry(e1);
                    return __byte_perm(centre(e0), centre(e1), 0x7632);
                }));
                if (active && r.consumed(seg_addr, chunk_start) != chunk_bits) bad = true;
            } else {
                WindowReader r;
                unsigned int used = 0;
                if (active) r.init(a.stream, cur.base + chunk_start, cur.base + cur.bits);
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
                if (active && used != chunk_bits) bad = true;
            }
            for (int kp = 0; kp < n_panels; ++kp)
                if (++slot0 == sub_slots) { slot0 = 0; phase0 ^= 1u; }
            if (bad) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
            named_bar_sync(bar_id, n_thr);           // this tile's stream buffer may be refilled
            cur = nxt;
            nxt = after;
            cur_copied = ahead;
        }
        cp_async_wait<0>();
        if (!alive && t == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else if (warp < kMmaWarp0) {
        // ================= epilogue: all eight warps work on every tile =================
        // A thread owns one channel (its TMEM lane) of one block of 128 channels.  With two
        // channel blocks warps 16-19 take the first and warps 20-23 the second; with one block
        // the two warp sets split the tile's pixels (TMEM columns) in halves.
        const int set = (warp - kEpiWarp0) >> 2;
        const int wq = warp & 3;                            // TMEM lane quarter of this warp
        const int n_blocks = (a.c + 127) / 128;
        const int blk = n_blocks == 2 ? set : 0;
        const int col_first = n_blocks == 2 ? 0 : 64 * set, col_count = n_blocks == 2 ? 128 : 64;
        const int ch = blk * 128 + wq * 32 + lane;
        const bool ch_ok = ch < a.c;
        const float step = (float)(a.step * a.basis_scale);        // the operand holds basis / basis_scale
        const float bias = ch_ok ? a.dec_bias[ch] : 0.f;
        const float floor_v = a.relu ? 0.f : __int_as_float((int)0xff800000u);        // the layer's non-linearity, when it follows the decoder
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.xhat);
        // With H*W a multiple of 4 every aligned group of four pixels lies inside one image and is
        // 8-byte aligned (given an 8-byte aligned tensor); otherwise pixels are stored one by one.
        const bool vec = (a.hw & 3) == 0 && ((uintptr_t)a.xhat & 7u) == 0;
        const long long img_stride = (long long)a.c * a.hw;
        const int ch_base = blk * 128 + wq * 32;            // first channel of this warp
        const int pgrp = lane & 7, r_sub = lane >> 3;
        const uint32_t tb = smem_u32(smem + L.tbuf) + (uint32_t)(warp - kEpiWarp0) * kTrWarpBytes;
        const uint32_t tb_wr = tb + (uint32_t)lane * kTrRowBytes;                   // this thread's channel row
        const uint32_t tb_rd = tb + (uint32_t)r_sub * kTrRowBytes + (uint32_t)pgrp * 8u;
        bool alive = true;
        for (long long tl = 0; tl < my_tiles && alive; ++tl) {
            const int grp = (int)(tl & 1);
            const long long tile = blockIdx.x + tl * gridDim.x;
            const long long p_first = tile * TC_TILE_PIXELS + col_first;
            const long long left = a.pixels - p_first;                       // pixels from this thread's first column on
            const int n_valid = (int)(left < (long long)col_count ? (left < 0 ? 0 : left) : (long long)col_count);
            // position of the first pixel; from there on it moves incrementally
            const long long img0 = left > 0 ? p_first / a.hw : 0;
            int s = left > 0 ? (int)(p_first - img0 * a.hw) : 0;
            __nv_bfloat16 *dst = out + img0 * img_stride + (long long)(ch_ok ? ch : 0) * a.hw + s;
            if (!mbar_wait(smem_u32(&s_tfull[grp]), (uint32_t)((tl >> 1) & 1), 1000u)) { alive = false; break; }
            tc_fence_after_sync();
            const uint32_t trow = tmem_base + grp * kAccCols + blk * 128 + ((uint32_t)(wq * 32) << 16) + col_first;
            if (vec) {
                // position of this lane's pixel group (4 pixels) in the first pass
                const long long pg = p_first + 4 * pgrp;
                long long img = pg < a.pixels ? pg / a.hw : 0;
                int sp = pg < a.pixels ? (int)(pg - img * a.hw) : 0;
                for (int c0 = 0; c0 < col_count; c0 += 32) {
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
                    // read phase: lane -> (row r_sub of every group of four channel rows, pixel group pgrp)
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
                for (int c0 = 0; c0 < col_count; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(trow + c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const __nv_bfloat16 h = __float2bfloat16_rn(fmaxf(fmaf(__uint_as_float(r[i]), step, bias), floor_v));
                        if (ch_ok && c0 + i < n_valid) *dst = h;
                        s += 1;
                        const bool wrap = s == a.hw;            // the next pixel starts the next image
                        dst += wrap ? 1 + img_stride - a.hw : 1;
                        s = wrap ? 0 : s;
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&s_tempty[grp]));
        }
        if (!alive && lane == 0 && wq == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else {
        // ================= MMA issuers (one per group) =================
        const int grp = warp - kMmaWarp0;
        if (lane == 0) {
            // A = transposed basis (128 channels per instruction), B = the decoded symbols of 128 pixels
            const uint32_t idesc = make_idesc_bf16(128, TC_TILE_PIXELS, /*A K-major*/ false, /*B K-major*/ false);
            const uint32_t a_sbo = (uint32_t)(a.k / 8) * 128u;
            const int n_blocks = (a.c + 127) / 128;
            const uint32_t ring_g = ring_addr + (uint32_t)grp * slots * slot_bytes;
            const int sub_slots = S == 2 ? 2 : slots;
            int slot = 0;                           // ring position (same for both halves) and its phase parity
            uint32_t phase = 0;
            bool alive = true;
            for (long long tl = grp; tl < my_tiles && alive; tl += 2) {
                if (!mbar_wait(smem_u32(&s_tempty[grp]), (uint32_t)(((tl >> 1) & 1) ^ 1), 500u)) { alive = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + grp * kAccCols;
                uint32_t accumulate = 0;
                for (int kp = 0; kp < n_panels && alive; ++kp) {
                    for (int sub = 0; sub < S; ++sub) {
                        const int s = sub * 2 + slot;
                        if (!mbar_wait(smem_u32(&s_full[grp][s]), phase, 200u)) { alive = false; break; }
                        // the panel was written with ordinary stores by threads that have arrived on the
                        // barrier: one proxy fence here, between that synchronisation and the MMA's
                        // operand reads, orders them for all 128 writers
                        fence_proxy_async_smem();
                        tc_fence_after_sync();
                        const int k0 = sub * k_sub + kp * panel_k;
                        const int nk16 = min(panel_k, (sub + 1) * k_sub - k0) >> 4;
                        for (int q = 0; q < nk16; ++q) {
                            const uint64_t bdesc = make_smem_desc(ring_g + s * slot_bytes + q * 4096, 2048, 128);
                            for (int blk = 0; blk < n_blocks; ++blk) {
                                const uint64_t adesc = make_smem_desc(basis_addr + blk * 16 * a_sbo + ((k0 + 16 * q) >> 3) * 128, 128, a_sbo);
                                mma_bf16_ss(d_tmem + blk * 128, adesc, bdesc, idesc, accumulate);
                            }
                            accumulate = 1u;
                        }
                        mma_commit(smem_u32(&s_empty[grp][s]));
                    }
                    if (++slot == sub_slots) { slot = 0; phase ^= 1u; }
                }
                if (alive) mma_commit(smem_u32(&s_tfull[grp]));
            }
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    }

    // ---- teardown ---------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

bool tc_decode_tc_supported(const tc_ctx *ctx, const DecodeArgs &a)
{
    // K <= C leading components (PCA truncation): K is the reduction dimension of the MMA
    if (a.c % 16 != 0 || a.k % 16 != 0 || a.k < 16 || a.k > a.c || a.c > 256) return false;
    if (a.splits != 1 && !(a.splits == 2 && a.chunk_pixels == 1 && a.k % 32 == 0)) return false;
    if (a.groups != 1 && a.groups != a.k) return false;
    if (a.lut_bits > TC_MAX_CODE_LEN) return false;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, a.chunk_pixels,
                                     a.splits, ctx->max_smem_optin - 512);
    return l.slots > 0;
}

// Bytes of a tile's stream segment this kernel can stage in shared memory (a segment of up to
// two stream buffers); longer segments are read from global memory, word by word.
size_t tc_decode_tc_staging_bytes(const tc_ctx *ctx, const DecodeArgs &a)
{
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, a.chunk_pixels,
                                     a.splits, ctx->max_smem_optin - 512);
    return l.slots > 0 ? 2u * (size_t)l.stream_buf : 0u;
}

tc_status tc_launch_decode_tc(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const SmemLayout l = smem_layout(a.c, a.k, a.groups == 1 ? (1 << a.lut_bits) : 0, a.chunk_pixels,
                                     a.splits, ctx->max_smem_optin - 512);
    if (l.slots == 0) return TC_ERR_UNSUPPORTED;
    void (*kernel)(DecodeArgs) = a.groups != 1 ? decode_tc_kernel<true> : decode_tc_kernel<false>;
    DecodeArgs args = a;
    args.smem_budget = ctx->max_smem_optin - 512;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.total) != cudaSuccess)
        return TC_ERR_CUDA;
    const unsigned int grid = (unsigned int)((a.n_tiles < ctx->sm_count) ? a.n_tiles : ctx->sm_count);
    kernel<<<grid, kThreads, l.total, s>>>(args);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
