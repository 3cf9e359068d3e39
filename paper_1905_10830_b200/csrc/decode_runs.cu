// Fused tensor-core decode for bf16 tensors with a per-layer code table (Section 3: VLD, inverse
// quantiser, inverse transform) whose work follows the information in the stream.
//
// After the PCA most coefficients of a pixel quantise to one symbol -- the level nearest zero --
// and the Huffman code gives that symbol the one-bit code 0 (Section 3.1, "Variable length
// coding"; Appendix E: the tail channels collapse to a single value).  A run of such symbols is
// a run of zero bits, so a decoder thread counts leading zeros and jumps over the whole run at
// once; only the other symbols cost a table lookup and a store.  The operand of the inverse
// projection is therefore filled first with the value of the modal symbol (16-byte stores) and
// the decoded symbols are then written into it one by one.
//
// One persistent block per SM.  Warp roles:
//   warps 0-7, 8-15    two VLD groups on alternating tiles of 128 pixels, each with its own operand
//                      buffer (all K coefficients of the tile, K-major).  One or two threads per
//                      pixel walk the pixel's chunks.
//   warps 16-23        epilogue, all eight warps on every work item: TMEM -> registers,
//                      x_hat = step * acc + bias, round to bf16, NCHW stores through warp-private
//                      transpose blocks (the accumulator is held transposed: lane = channel)
//   warps 24, 25       one thread each issues the tcgen05.mma of its accumulator's work items:
//                      D[c][pixel] = T[j][c] * (Q[pixel][j] - center)
// The transposed basis is the A operand and lives in TENSOR memory, not in shared memory: each
// block of 128 channels takes K / 2 columns (two bf16 per column), 256 columns at C = K = 256,
// loaded once per block with tcgen05.st.  That leaves shared memory to the symbols -- two whole
// tiles in flight, 128 KB at K = 256 -- and takes the basis off the MMA's shared-memory reads.
// The other 256 columns hold two accumulators of 128 columns: one tile of 128 pixels up to 128
// channels; with two channel blocks a work item is half a tile (2 x 64 columns), so that the
// epilogue of one item overlaps the MMAs of the next.
// The operand is handed back in panels of 32 coefficients: the MMA thread commits a barrier per
// panel, and a VLD thread of the group's next tile waits only for the panel it is about to touch.
//
// A tile whose stream is dense (more than kDenseBits128 / 128 bits per symbol) gains nothing
// from run skipping; its threads then decode symbol by symbol, eight symbols per 16-byte store.
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace tcdev;
using namespace sm100;

constexpr int kGroupWarps = 8, kEpiWarp0 = 2 * kGroupWarps, kMmaWarp = kEpiWarp0 + 8;
constexpr int kThreads = (kMmaWarp + 2) * 32;                  // two MMA warps, one per accumulator
constexpr int kTmemCols = 512;
constexpr int kAccBase = 256, kAccCols = 128;                 // two accumulators behind the basis columns
constexpr int kPanelK = 32;                                   // coefficients per hand-over panel
constexpr int kMaxPanels = 8;                                 // K <= 256
constexpr uint32_t kRunGuard = 0x800u;                        // bit 11 set: at most 20 zero bits are skipped per step (20 + 12 <= 32: one refill per step)
constexpr int kDenseBits128 = 224;                            // tiles above 1.75 bits per symbol are decoded symbol by symbol
// A chunk that starts inside a staged segment is read for at most (symbols of the chunk) x 12
// bits, whatever the bits say; the slack after the last buffer keeps those reads inside the
// block's shared memory even for a corrupt stream (the buffers lie back to back).
constexpr int kStreamSlack = 1024;
constexpr int kTrWarpBytes = 1024;                            // epilogue transpose block of one warp: 32 channel rows x 16 pixels
// Named barriers.  Hand-overs between warps that both run ordinary instructions use them instead
// of mbarriers: the waiting side is parked by the hardware, whereas a warp polling an mbarrier
// keeps issuing and takes issue slots from the warps that work.  (mbarriers remain where the
// tensor core signals: accumulator ready, operand panel consumed.)
constexpr int kBarGroup = 1;                                  // + group: the VLD threads of a group, once per tile
constexpr int kBarFull = 3;                                   // + group: operand complete, VLD threads -> MMA warp
constexpr int kBarAccFree = 5;                                // + accumulator: drained, epilogue warps -> MMA warp
constexpr int kBarEpi = 7;                                    // accumulator ready, polling epilogue warp -> the other seven

struct SmemLayout {
    uint32_t lut, opnd, tbuf, sbuf, total;
    uint32_t opnd_bytes;                                      // one operand buffer (one per VLD group)
    uint32_t stream_buf;                                      // bytes per staged stream buffer (two per group; 0: does not fit)
};

__host__ __device__ inline SmemLayout smem_layout(int k, int lut_entries, int budget)
{
    SmemLayout l;
    l.lut = 0;                                                // 32-bit entries: bf16(symbol - center) << 16 | length
    l.opnd = ((uint32_t)lut_entries * 4u + 1023u) & ~1023u;
    l.opnd_bytes = (uint32_t)k * TC_TILE_PIXELS * 2;
    l.tbuf = l.opnd + 2u * l.opnd_bytes;
    l.sbuf = l.tbuf + 8u * kTrWarpBytes;
    l.stream_buf = 0;
    l.total = 0;
    for (uint32_t kb = 16; kb >= 4; --kb)
        if ((long long)l.sbuf + 4ll * kb * 1024 + kStreamSlack <= (long long)budget) {
            l.stream_buf = kb * 1024;
            l.total = l.sbuf + 4u * l.stream_buf + kStreamSlack;
            break;
        }
    return l;
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u16(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

// MSB-first reader with a 64-bit window hi:lo (left-aligned) and one word of look-ahead.  `used`
// counts, in its low byte, the bits taken since the window was last moved on by a word; table
// entries (symbol << 8 | length) are added to it and fed to the funnel shifts as they are (the
// shifts take their amount modulo 32, lengths are at most 12).  refill() moves the window on by
// one word when 32 bits or more have been taken; a caller that takes at most 32 bits between two
// refills always sees at least 32 valid bits after one.
// kShared: the words lie in shared memory (a staged segment, with readable slack behind it);
// otherwise in global memory, where words at or past `end` read as zero.
template <bool kShared>
struct BitReader {
    uint32_t hi, lo, ahead, used;
    uint32_t next_addr;               // shared: address of the word after `ahead`
    const uint32_t *next, *end;       // global
    uint32_t origin;                  // shared: bit address (shared address * 8) init() was given; global: that position modulo 32
    uint32_t words;                   // global: words the window has moved on by

    __device__ __forceinline__ uint32_t fetch()
    {
        uint32_t w;
        if constexpr (kShared) { w = lds_u32(next_addr); next_addr += 4; }
        else { w = next < end ? __ldg(next) : 0u; ++next; }
        return w;
    }
    // kShared: `base_addr` is the shared address of the segment; else `base` / `end_word` delimit it
    __device__ __forceinline__ void init(uint32_t base_addr, const uint32_t *base, const uint32_t *end_word, uint32_t bitpos)
    {
        if constexpr (kShared) { next_addr = base_addr + (bitpos >> 5) * 4u; origin = next_addr * 8u + (bitpos & 31u); }
        else { next = base + (bitpos >> 5); end = end_word; origin = bitpos & 31u; }
        const uint32_t w0 = fetch(), w1 = fetch();
        ahead = fetch();
        const uint32_t sh = bitpos & 31u;
        hi = __funnelshift_l(w1, w0, sh);
        lo = w1 << sh;
        used = sh;
        words = 0;
    }
    __device__ __forceinline__ void idle()
    {
        hi = lo = ahead = used = origin = words = 0;
        next_addr = 0; next = end = nullptr;
    }
    // `entry`: a bit count below 32, or a table entry with the count in its low byte (what lies
    // above only reaches bits of `used` that nothing reads)
    __device__ __forceinline__ void take(uint32_t entry)
    {
        hi = __funnelshift_l(lo, hi, entry);
        lo = __funnelshift_l(0u, lo, entry);
        used += entry;
    }
    __device__ __forceinline__ void refill()
    {
        // with c = used - 32 bits of the next word's span already taken, the window gains `ahead`
        // behind its 64 - used valid bits: hi |= ahead >> (32 - c), lo |= ahead << c (the shifts take
        // their amount modulo 32)
        if constexpr (kShared) {
            asm volatile(
                "{\n\t.reg .pred p;\n\t.reg .b32 t, u;\n\t"
                "and.b32 t, %3, 32;\n\t"
                "setp.ne.u32 p, t, 0;\n\t"
                "shf.l.wrap.b32 t, %2, 0, %3;\n\t"
                "shf.l.wrap.b32 u, 0, %2, %3;\n\t"
                "@p or.b32 %0, %0, t;\n\t"
                "@p or.b32 %1, %1, u;\n\t"
                "@p add.u32 %3, %3, -32;\n\t"
                "@p ld.shared.u32 %2, [%4];\n\t"
                "@p add.u32 %4, %4, 4;\n\t}"
                : "+r"(hi), "+r"(lo), "+r"(ahead), "+r"(used), "+r"(next_addr));
        } else if (used & 32u) {
            hi |= __funnelshift_l(ahead, 0u, used);
            lo |= __funnelshift_l(0u, ahead, used);
            used -= 32u;
            ahead = fetch();
            ++words;
        }
    }
    // bits taken since init()
    __device__ __forceinline__ uint32_t consumed() const
    {
        if constexpr (kShared) return (next_addr - 12u) * 8u + (used & 0xffu) - origin;   // the window starts three words behind next_addr
        else return words * 32u + (used & 0xffu) - origin;
    }
};

template <bool kRelu>
__global__ void __launch_bounds__(kThreads, 1) decode_runs_kernel(DecodeArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_empty[2][kMaxPanels], s_tfull[2];
    __shared__ uint32_t s_tmem_base;
    // [group][tile parity][thread set][warp]: bits per warp, for the start positions.  Two copies: a warp
    // that is done with its tile early writes the next tile's sum while a slower warp may still
    // be reading this tile's; the group's barrier (one per tile) only orders the write after next.
    __shared__ unsigned int s_wsum[2][2][2][4];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lut_size = 1 << a.lut_bits;
    const SmemLayout L = smem_layout(a.k, lut_size, a.smem_budget);
    constexpr int nbuf = 2;
    const uint32_t lut_addr = smem_u32(smem + L.lut);
    const uint32_t opnd_addr = smem_u32(smem + L.opnd);
    const int n_blocks = (a.c + 127) / 128;                    // blocks of 128 channels
    const int items = n_blocks;                                // work items per tile: halves of 64 pixels with two channel blocks
    const int S = a.splits, cp = a.chunk_pixels;
    const int tpp = S >= 2 ? 2 : 1;                            // threads per pixel
    const int chunks_per_thread = S / tpp;                     // 1, or 2 with four chunks per pixel
    const int n_work = cp > 1 ? TC_TILE_PIXELS / cp : TC_TILE_PIXELS * tpp;   // threads of a group that own chunks
    const int n_thr = ((n_work + 31) / 32) * 32;               // whole warps take part in the group's barriers

    // ---- set-up ---------------------------------------------------------------------
    if (tid == 0) {
        for (int g = 0; g < 2; ++g) {
            for (int p = 0; p < kMaxPanels; ++p) mbar_init(smem_u32(&s_empty[g][p]), (uint32_t)items);   // one commit per item of the tile
            mbar_init(smem_u32(&s_tfull[g]), 1);
        }
        mbar_fence_init();
    }
    if (warp == kMmaWarp) { tmem_alloc(smem_u32(&s_tmem_base), kTmemCols); tmem_relinquish(); }
    {
        // per-layer table: bf16(symbol - center) << 16 | code length
        uint32_t *s_lut = reinterpret_cast<uint32_t *>(smem + L.lut);
        for (int i = tid; i < lut_size; i += kThreads) {
            const uint32_t e = a.lut32[i];
            const float f = (float)((int)((e >> 8) & 0xffu) - a.center);
            s_lut[i] = (__float_as_uint(f) & 0xffff0000u) | (e & 0xffu);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    if (warp >= kEpiWarp0 && warp < kMmaWarp) {
        // Transposed basis -> tensor memory: row c of block b (channel 128 b + c) goes to lane c,
        // its K coefficients, two per 32-bit column in memory order, to columns b K/2 ... of the A
        // operand.  A warp reaches the 32 lanes of its quarter; rows past C are zero (their outputs
        // are never stored).
        const int wq = warp & 3;
        const uint32_t *src = reinterpret_cast<const uint32_t *>(a.basis_t_bf16);
        for (int blk = (warp - kEpiWarp0) >> 2; blk < n_blocks; blk += 2) {
            const int ch = blk * 128 + wq * 32 + lane;
            const uint32_t *row = src + (size_t)(ch < a.c ? ch : 0) * (a.k / 2);
            const uint32_t trow = tmem_base + ((uint32_t)(wq * 32) << 16) + (uint32_t)(blk * (a.k / 2));
            for (int j = 0; j < a.k / 2; j += 16) {
                if (a.k / 2 - j >= 16) {
                    uint32_t r[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        const uint4 v = ch < a.c ? __ldg(reinterpret_cast<const uint4 *>(row + j + i)) : make_uint4(0u, 0u, 0u, 0u);
                        r[i] = v.x; r[i + 1] = v.y; r[i + 2] = v.z; r[i + 3] = v.w;
                    }
                    tmem_st_32x32b_x16(trow + j, r);
                } else {                                         // K % 32 == 16: eight columns left
                    uint32_t r[8];
#pragma unroll
                    for (int i = 0; i < 8; i += 4) {
                        const uint4 v = ch < a.c ? __ldg(reinterpret_cast<const uint4 *>(row + j + i)) : make_uint4(0u, 0u, 0u, 0u);
                        r[i] = v.x; r[i + 1] = v.y; r[i + 2] = v.z; r[i + 3] = v.w;
                    }
                    tmem_st_32x32b_x8(trow + j, r);
                }
            }
        }
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    const long long my_tiles = (a.n_tiles > blockIdx.x) ? (a.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp < kEpiWarp0) {
        // ================= VLD groups =================
        const int grp = warp >> 3;
        const int tg = tid & 255;                // thread within the group
        if (tg < n_thr) {
            const int set = cp > 1 ? 0 : tg >> 7;    // which thread of the pixel (warp-uniform)
            const int t = cp > 1 ? tg : (tg & 127);  // pixel within the tile, or chunk within the tile (cp > 1)
            const int wq = (t >> 5) & 3;
            const bool owner = tg < n_work;          // this thread has chunks to decode
            const int k_sub = a.k / S;               // coefficients per chunk of one pixel
            const int k_first = set * chunks_per_thread * k_sub;           // this thread's coefficients of a pixel
            const int k_last = cp > 1 ? a.k : k_first + chunks_per_thread * k_sub;
            const int p_first = k_first / kPanelK, p_last = (k_last + kPanelK - 1) / kPanelK;     // panels it touches
            const int chunks_per_tile = S * TC_TILE_PIXELS / cp;
            const uint32_t opnd_g = opnd_addr + (uint32_t)grp * L.opnd_bytes;
            const uint32_t sbuf_bytes = L.stream_buf;
            const uint32_t sbuf_g = smem_u32(smem + L.sbuf) + (uint32_t)grp * 2u * sbuf_bytes;
            const int bar_id = kBarGroup + grp;
            const int lb = a.lut_bits;
            const int dense_head = (a.dense_head + 7) & ~7;    // leading coefficients decoded symbol by symbol
            const uint32_t modal2 = (__float_as_uint((float)((a.modal < 0 ? a.center : a.modal) - a.center)) >> 16) * 0x00010001u;   // two bf16 copies of the modal symbol's value
            bool alive = true;

            // offsets of a tile, validated; a tile that cannot be valid decodes nothing.  `lens`
            // holds the chunk lengths of this thread's pixel (up to four), or of its chunk.
            struct TileInfo { unsigned long long base, bits; bool ok, staged; unsigned int l01, l23; };
            auto tile_info = [&](long long tl) {
                TileInfo ti{0, 0, false, false, 0, 0};
                if (tl >= my_tiles) return ti;
                const long long tile = blockIdx.x + tl * gridDim.x;
                const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
                ti.ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
                if (!ti.ok) return ti;
                ti.base = base;
                ti.bits = end - base;
                ti.staged = ti.bits <= (unsigned long long)sbuf_bytes * 8ull &&
                            (cp * (k_last - k_first) * TC_MAX_CODE_LEN) / 8 + 16 <= kStreamSlack;
                if (owner) {
                    const long long ch = tile * chunks_per_tile + (long long)t * (cp > 1 ? 1 : S);
                    if (cp > 1 || S == 1) { if (ch < a.n_chunks) ti.l01 = a.chunk_len[ch]; }
                    else if (ch < a.n_chunks) {      // S chunks of one pixel: an aligned word holds two lengths
                        ti.l01 = *reinterpret_cast<const unsigned int *>(a.chunk_len + ch);
                        if (S == 4) ti.l23 = *reinterpret_cast<const unsigned int *>(a.chunk_len + ch + 2);
                    }
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

            TileInfo cur = tile_info(grp), nxt = tile_info(grp + nbuf);
            stage_tile(cur, 0);
            int li = 0;
            // (a thread whose wait ran out keeps walking the tiles without decoding: the group's
            // barriers and the hand-over to the MMA thread need every thread's arrival)
            for (long long tl = grp; tl < my_tiles; tl += nbuf, ++li) {
                const long long tile = blockIdx.x + tl * gridDim.x;
                // start of every chunk = sum of the lengths before it in the tile (chunk order: pixel,
                // then part of the pixel): scan over the pixels' totals
                const unsigned int len0 = cur.l01 & 0xffffu, len1 = cur.l01 >> 16, len2 = cur.l23 & 0xffffu, len3 = cur.l23 >> 16;
                const unsigned int tot = len0 + len1 + len2 + len3;
                unsigned int inc = tot;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
                    if (lane >= d) inc += up;
                }
                if (lane == 31) s_wsum[grp][li & 1][set][wq] = inc;
                cp_async_wait<0>();
                // every thread's part of this tile's segment has landed, and every thread is done
                // with the tile before: its stream buffer may take the next tile's segment
                named_bar_sync(bar_id, n_thr);
                stage_tile(nxt, (li + 1) & 1);
                const TileInfo after = tile_info(tl + 2 * nbuf);   // offsets two tiles ahead: their latency hides behind the decode
                unsigned int before = 0, tile_total = 0;
                const int n_wq = (n_work / tpp + 31) / 32;          // warps of one thread set
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const unsigned int sw = w < n_wq ? s_wsum[grp][li & 1][set][w] : 0u;
                    if (w < wq) before += sw;
                    tile_total += sw;
                }
                // this thread's first chunk: after the pixels before it and the chunks of the pixel before its own
                unsigned int chunk_start = before + inc - tot;
                unsigned int my_len0 = len0, my_len1 = len1;
                if (cp == 1 && set == 1) {
                    if (S == 2) { chunk_start += len0; my_len0 = len1; }
                    else { chunk_start += len0 + len1; my_len0 = len2; my_len1 = len3; }
                }

                const long long ch = tile * chunks_per_tile + (long long)t * (cp > 1 ? 1 : S);
                bool active = cur.ok && owner && ch < a.n_chunks;
                bool bad = !cur.ok || (unsigned long long)tile_total > cur.bits;
                if (bad) active = false;
                const long long px0 = tile * TC_TILE_PIXELS + (long long)t * cp;
                const int n_pix = active ? (int)min((long long)cp, a.pixels - px0) : 0;
                const uint32_t seg_addr = sbuf_g + (uint32_t)(li & 1) * sbuf_bytes;
                // dense tiles are decoded symbol by symbol
                const bool runs = a.modal >= 0 &&
                                  cur.bits * 128ull <= (unsigned long long)kDenseBits128 * (unsigned long long)a.k * TC_TILE_PIXELS;
                const uint32_t wait_parity = (uint32_t)((li & 1) ^ 1);   // the buffer's hand-back by the tile before this one

                // Walks this thread's chunks.  Control flow is kept uniform across the warp: the lanes
                // of a warp step together (a lane that has finished its chunk idles until all have),
                // panels are waited for and filled by all lanes at once when any lane needs the next
                // one, and a wait that runs out is seen by every lane -- lanes that wander off on
                // their own would run the rest of the tile one after the other.
                auto decode_tile = [&](auto &r) {
                    uint32_t expect = 0;               // bits the chunks decoded so far should have taken
                    for (int pp = 0; pp < cp; ++pp) {
                        const bool decode = pp < n_pix;
                        const uint32_t row = (uint32_t)(t * cp + pp);
                        const uint32_t row_addr = opnd_g + (row >> 3) * 128u + (row & 7u) * 16u;
                        int ready = p_first;           // panels [p_first, ready) of the warp's rows are handed back and filled
                        // waits for panel p to be handed back by the MMAs of the tile before, then fills this
                        // thread's coefficients of it from coefficient `from` on with the modal symbol
                        auto prepare = [&](int p, int from) {
                            if (pp == 0 && alive) alive = mbar_wait(smem_u32(&s_empty[grp][p]), wait_parity, 200u);
                            if (owner) {
                                const int g0 = max(p * (kPanelK / 8), max(k_first, from) >> 3), g1 = min((p + 1) * (kPanelK / 8), k_last >> 3);
                                for (int g = g0; g < g1; ++g) sts_v4(row_addr + (uint32_t)g * 2048u, modal2, modal2, modal2, modal2);
                            }
                        };
                        for (int ci = 0; ci < (cp > 1 ? 1 : chunks_per_thread); ++ci) {
                            const int kf = cp > 1 ? 0 : k_first + ci * k_sub, ke = cp > 1 ? a.k : kf + k_sub;
                            // the leading coefficients (and every coefficient of a dense tile) symbol by symbol,
                            // eight symbols per 16-byte store; the rest run by run
                            const int kd = runs ? min(max(dense_head, kf), ke) : ke;
                            for (int k0 = kf; k0 < kd; k0 += 8) {
                                while (ready * kPanelK <= k0) prepare(ready++, kd);
                                uint32_t pk[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    r.refill();
                                    const uint32_t e0 = lds_u32(lut_addr + (r.hi >> (32 - lb)) * 4u);
                                    r.take(decode ? e0 : 0u);
                                    const uint32_t e1 = lds_u32(lut_addr + (r.hi >> (32 - lb)) * 4u);
                                    r.take(decode ? e1 : 0u);
                                    pk[i] = __byte_perm(e0, e1, 0x7632);
                                }
                                if (decode) sts_v4(row_addr + (uint32_t)(k0 >> 3) * 2048u, pk[0], pk[1], pk[2], pk[3]);
                            }
                            uint32_t pos = (uint32_t)kd, rem = decode ? (uint32_t)(ke - kd) : 0u;
                            uint32_t ready_end = (uint32_t)(ready * kPanelK);
                            while (__any_sync(0xffffffffu, rem != 0u)) {
                                r.refill();
                                // a run of the modal symbol is a run of zero bits: at most 20 per step
                                const uint32_t n = min((uint32_t)__clz((int)(r.hi | kRunGuard)), rem);
                                r.take(n);
                                pos += n;
                                rem -= n;
                                const bool sym = rem != 0u;            // a symbol follows the run
                                const uint32_t e = lds_u32(lut_addr + (r.hi >> (32 - lb)) * 4u);
                                r.take(sym ? e : 0u);
                                while (__any_sync(0xffffffffu, sym && pos >= ready_end)) { prepare(ready++, kd); ready_end += kPanelK; }
                                // coefficient pos of the row: core-matrix column pos / 8 (2048 bytes apart), 2 bytes per coefficient inside
                                if (sym) sts_u16(row_addr + pos * 2u + (pos >> 3) * 2032u, e >> 16);
                                pos += sym ? 1u : 0u;
                                rem -= sym ? 1u : 0u;
                            }
                            // a chunk of one pixel (or part of it) must end exactly where its length says
                            if (cp == 1) {
                                expect += ci == 0 ? my_len0 : my_len1;
                                if (active && r.consumed() != expect) bad = true;
                            }
                        }
                        while (ready < p_last) prepare(ready++, 0);
                    }
                    if (cp > 1 && active && r.consumed() != len0) bad = true;
                };
                if (cur.ok && cur.staged) {
                    BitReader<true> r;
                    if (active) r.init(seg_addr, nullptr, nullptr, chunk_start);
                    else r.idle();
                    decode_tile(r);
                } else {
                    BitReader<false> r;
                    if (active) {
                        const uint32_t *seg = a.stream + (cur.base >> 5);
                        r.init(0u, seg, seg + (cur.bits >> 5), chunk_start);
                    } else r.idle();
                    decode_tile(r);
                }
                // (the issuing thread makes the operand visible to the tensor core's proxy)
                named_bar_arrive(kBarFull + grp, n_thr + 32 * items);
                if (bad) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
                cur = nxt;
                nxt = after;
            }
            cp_async_wait<0>();
            if (!alive) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
        }
    } else if (warp < kMmaWarp) {
        // ================= epilogue: all eight warps work on every item =================
        // A thread owns one channel (its TMEM lane) of one block of 128 channels and 64 pixels of
        // the item.  With two channel blocks an item is half a tile: warps 16-19 take the first
        // block and warps 20-23 the second; with one block an item is a tile and the two warp sets
        // split its pixels (TMEM columns) in halves.
        const int set = (warp - kEpiWarp0) >> 2;
        const int wq = warp & 3;                            // TMEM lane quarter of this warp
        const int blk = n_blocks == 2 ? set : 0;
        const int col_first = n_blocks == 2 ? 0 : 64 * set;
        constexpr int col_count = 64;
        const int ch = blk * 128 + wq * 32 + lane;
        const bool ch_ok = ch < a.c;
        const float step = (float)(a.step * a.basis_scale);        // the operand holds basis / basis_scale
        const float bias = ch_ok ? a.dec_bias[ch] : 0.f;
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(a.xhat);
        // With H*W a multiple of 4 every aligned group of four pixels lies inside one image and is
        // 8-byte aligned (given an 8-byte aligned tensor); otherwise pixels are stored one by one.
        const bool vec = (a.hw & 3) == 0 && ((uintptr_t)a.xhat & 7u) == 0;
        const long long img_stride = (long long)a.c * a.hw;
        const int ch_base = blk * 128 + wq * 32;            // first channel of this warp
        // transpose block: row = channel (32 bytes = 16 pixels); the two 16-byte halves of a row are
        // swapped in rows 4-7, 12-15, ... so that neither the row writes nor the reads below collide
        const uint32_t tb = smem_u32(smem + L.tbuf) + (uint32_t)(warp - kEpiWarp0) * kTrWarpBytes;
        const uint32_t sw_wr = (uint32_t)((lane >> 2) & 1);
        const uint32_t tb_wr = tb + (uint32_t)lane * 32u;
        const int r_sub = lane >> 2, piece = lane & 3;      // read phase: channel row r_sub (+ 8, 16, 24), pixels 4 * piece ...
        const uint32_t tb_rd = tb + (uint32_t)r_sub * 32u + ((((uint32_t)piece >> 1) ^ ((uint32_t)(r_sub >> 2) & 1u)) << 4) + ((uint32_t)piece & 1u) * 8u;
        // two accumulator values -> two bf16: x_hat = step * acc + bias (one packed fused multiply-add)
        auto convert = [&](uint32_t x0, uint32_t x1) {
            float f0, f1;
            asm("{\n\t.reg .b64 v, s, b;\n\t"
                "mov.b64 v, {%2, %3};\n\t"
                "mov.b64 s, {%4, %4};\n\t"
                "mov.b64 b, {%5, %5};\n\t"
                "fma.rn.f32x2 v, v, s, b;\n\t"
                "mov.b64 {%0, %1}, v;\n\t}"
                : "=f"(f0), "=f"(f1) : "r"(x0), "r"(x1), "f"(step), "f"(bias));
            if constexpr (kRelu) { f0 = fmaxf(f0, 0.f); f1 = fmaxf(f1, 0.f); }   // the layer's non-linearity, when it follows the decoder
            const __nv_bfloat162 h = __floats2bfloat162_rn(f0, f1);
            return *reinterpret_cast<const uint32_t *>(&h);
        };
        // the four channel rows this lane stores in the read phase of a pass: offsets inside an image
        int row_off[4];
        bool row_ok[4];
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            row_ok[it] = ch_base + 8 * it + r_sub < a.c;
            row_off[it] = (ch_base + 8 * it + r_sub) * a.hw;
        }
        bool alive = true;
        const long long n_items = my_tiles * items;
        // (after a wait that ran out the warps keep walking the items: the MMA warp waits for their arrivals)
        for (long long it = 0; it < n_items; ++it) {
            const int acc = (int)(it & 1);
            const long long tl = items == 2 ? (it >> 1) : it;
            const int item = items == 2 ? (int)(it & 1) : 0;
            const long long tile = blockIdx.x + tl * gridDim.x;
            const long long p_first = tile * TC_TILE_PIXELS + item * 64 + col_first;
            const long long left = a.pixels - p_first;                       // pixels from this thread's first column on
            const int n_valid = (int)(left < (long long)col_count ? (left < 0 ? 0 : left) : (long long)col_count);
            // the first epilogue warp waits for the accumulator and lets the others in
            if (warp == kEpiWarp0) {
                if (alive) alive = mbar_wait(smem_u32(&s_tfull[acc]), (uint32_t)((it >> 1) & 1), 100u);
                tc_fence_before_sync();
            }
            named_bar_sync(kBarEpi, 256);
            tc_fence_after_sync();
            const uint32_t trow = tmem_base + kAccBase + acc * kAccCols + (n_blocks == 2 ? blk * 64 : 0) + ((uint32_t)(wq * 32) << 16) + col_first;
            if (vec) {
                // position of this lane's pixel group (4 pixels) in the first pass
                const long long pg = p_first + 4 * piece;
                long long img = pg < a.pixels ? pg / a.hw : 0;
                int sp = pg < a.pixels ? (int)(pg - img * a.hw) : 0;
                for (int c0 = 0; c0 < col_count; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(trow + c0, r);
                    tmem_ld_wait();
                    sts_v4(tb_wr + (sw_wr << 4), convert(r[0], r[1]), convert(r[2], r[3]), convert(r[4], r[5]), convert(r[6], r[7]));
                    sts_v4(tb_wr + ((sw_wr ^ 1u) << 4), convert(r[8], r[9]), convert(r[10], r[11]), convert(r[12], r[13]), convert(r[14], r[15]));
                    __syncwarp();
                    const bool px_ok = c0 + 4 * piece < n_valid;
                    __nv_bfloat16 *px_ptr = out + img * img_stride + sp;
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        uint32_t lo2, hi2;
                        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(lo2), "=r"(hi2) : "r"(tb_rd + it * 256));
                        if (px_ok && row_ok[it]) *reinterpret_cast<uint2 *>(px_ptr + row_off[it]) = make_uint2(lo2, hi2);
                    }
                    sp += 16;
                    while (sp >= a.hw) { sp -= a.hw; ++img; }
                    __syncwarp();                                   // the block may be overwritten
                }
            } else {
                // position of the first pixel; from there on it moves incrementally
                const long long img0 = left > 0 ? p_first / a.hw : 0;
                int s = left > 0 ? (int)(p_first - img0 * a.hw) : 0;
                __nv_bfloat16 *dst = out + img0 * img_stride + (long long)(ch_ok ? ch : 0) * a.hw + s;
                for (int c0 = 0; c0 < col_count; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(trow + c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float f = fmaf(__uint_as_float(r[i]), step, bias);
                        if constexpr (kRelu) f = fmaxf(f, 0.f);
                        if (ch_ok && c0 + i < n_valid) *dst = __float2bfloat16_rn(f);
                        s += 1;
                        const bool wrap = s == a.hw;            // the next pixel starts the next image
                        dst += wrap ? 1 + img_stride - a.hw : 1;
                        s = wrap ? 0 : s;
                    }
                }
            }
            tc_fence_before_sync();
            named_bar_arrive(kBarAccFree + acc, 256 + 32);
        }
        if (!alive && lane == 0) tc_dev_set_status(a.status, TC_ERR_TIMEOUT);
    } else {
        // ================= MMA issuers =================
        // Two warps, one per accumulator: with two channel blocks warp w issues item w (pixels 64 w ...)
        // of every tile, with one block the tiles alternate between the warps.  An MMA leaves its
        // issuing thread about every 64 cycles at best and an item is K / 16 of them per channel block,
        // so one warp alone would be the slowest stage of the kernel.  The whole warp walks the loop
        // and waits on the barriers; lane 0 issues, through instructions that carry their own guard
        // (no branch around an MMA).
        // A = transposed basis in tensor memory (128 channels per instruction), B = the decoded
        // symbols of the item's pixels (rows of the group's operand buffer).
        const int w = warp - kMmaWarp;
        const uint32_t issuer = lane == 0 ? 1u : 0u;
        const int np = items == 2 ? 64 : TC_TILE_PIXELS;          // pixels per work item
        const uint32_t idesc = make_idesc_bf16(128, np, /*A K-major*/ false, /*B K-major*/ false);
        const uint32_t a_blk1 = (uint32_t)(a.k / 2);               // columns between the two channel blocks of the basis
        const int n_k16 = a.k >> 4;
        const uint32_t d_tmem = tmem_base + kAccBase + w * kAccCols;
        for (long long tl = items == 2 ? 0 : w; tl < my_tiles; tl += items == 2 ? 1 : 2) {
            const int buf = (int)(tl & 1);
            const long long it = items == 2 ? 2 * tl + w : tl;       // index of the work item: item it uses accumulator it % 2 = w
            __syncwarp();
            named_bar_sync(kBarFull + buf, n_thr + 32 * items);       // the group's VLD threads have arrived
            // the operand was written with ordinary stores by threads that have arrived on the
            // barrier: one proxy fence here, between that synchronisation and the MMA's
            // operand reads, orders them for all writers
            fence_proxy_async_smem();
            const uint64_t b_base = make_smem_desc(opnd_addr + (uint32_t)buf * L.opnd_bytes, 2048, 128);
            const uint32_t b_hi = (uint32_t)(b_base >> 32);
            __syncwarp();
            if (it >= 2) named_bar_sync(kBarAccFree + w, 256 + 32);   // the epilogue has drained the accumulator
            tc_fence_after_sync();
            // rows 64 w ... of the buffer (two blocks): eight-row groups are 128 bytes apart; a step of 16
            // coefficients moves the start address on by two core-matrix columns of 2048 bytes
            uint32_t b_lo = (uint32_t)b_base + (items == 2 ? (uint32_t)w * (1024u >> 4) : 0u);
            uint32_t a_col = tmem_base;
            for (int q = 0; q < n_k16; ++q) {
                mma_bf16_ts_guarded(d_tmem, a_col, b_lo, b_hi, idesc, q ? 1u : 0u, issuer);
                if (n_blocks == 2) mma_bf16_ts_guarded(d_tmem + 64, a_col + a_blk1, b_lo, b_hi, idesc, q ? 1u : 0u, issuer);
                // a finished panel goes back to the VLD threads (when every item of the tile has read it)
                if ((q & 1) || q == n_k16 - 1) mma_commit_guarded(smem_u32(&s_empty[buf][q >> 1]), issuer);
                b_lo += 4096u >> 4;
                a_col += 8;
            }
            mma_commit_guarded(smem_u32(&s_tfull[w]), issuer);
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

bool tc_decode_runs_supported(const tc_ctx *ctx, const DecodeArgs &a)
{
    // K <= C leading components (PCA truncation): K is the reduction dimension of the MMA
    if (a.c % 16 != 0 || a.k % 16 != 0 || a.k < 16 || a.k > a.c || a.c > 256) return false;
    if (a.groups != 1) return false;                           // per-channel tables do not fit shared memory
    if (a.lut_bits > TC_MAX_CODE_LEN) return false;
    if (a.chunk_pixels > 1 ? a.splits != 1 : (a.splits != 1 && a.splits != 2 && a.splits != 4)) return false;
    if (a.splits > 1 && (a.k % a.splits != 0 || (a.k / a.splits) % 8 != 0)) return false;
    return smem_layout(a.k, 1 << a.lut_bits, ctx->max_smem_optin - 512).stream_buf > 0;
}

// Bytes of a tile's stream segment this kernel stages in shared memory; longer segments are read
// from global memory, word by word.
size_t tc_decode_runs_staging_bytes(const tc_ctx *ctx, const DecodeArgs &a)
{
    return smem_layout(a.k, 1 << a.lut_bits, ctx->max_smem_optin - 512).stream_buf;
}

tc_status tc_launch_decode_runs(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const SmemLayout l = smem_layout(a.k, 1 << a.lut_bits, ctx->max_smem_optin - 512);
    if (l.stream_buf == 0) return TC_ERR_UNSUPPORTED;
    void (*kernel)(DecodeArgs) = a.relu ? decode_runs_kernel<true> : decode_runs_kernel<false>;
    DecodeArgs args = a;
    args.smem_budget = ctx->max_smem_optin - 512;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l.total) != cudaSuccess)
        return TC_ERR_CUDA;
    const unsigned int grid = (unsigned int)((a.n_tiles < ctx->sm_count) ? a.n_tiles : ctx->sm_count);
    kernel<<<grid, kThreads, l.total, s>>>(args);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
