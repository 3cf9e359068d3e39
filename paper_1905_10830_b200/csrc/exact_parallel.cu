// Exact (fp64) projection and reconstruction with one thread per output value, for tensors of
// few pixels (the fp32 maps of one image: Section 4's ResNet-18 layers at batch 1).
//
// The exact encode / decode kernels give a pixel to a thread, which then walks C x K products
// alone: a 512 x 7 x 7 map keeps 49 threads busy for milliseconds.  Here every (pixel,
// coefficient) pair of the projection y_j = sum_c T[j][c] (x_c - mu_c) (Section 3, first
// equation) and every (pixel, channel) pair of the inverse x_hat_c = sum_j T[j][c] y_hat_j + mu_c
// is a thread of its own.  Each thread adds its products in the same order and with the same
// unfused double operations as the per-pixel kernels, so the results are bit-identical to theirs
// (and to the definition evaluated in fp64); the entropy coder then runs in the per-pixel kernels
// on the symbols these kernels leave in memory.
#include "device_utils.cuh"

namespace {

using namespace tcdev;

constexpr int kPx = 32;        // pixels per block (one warp row: loads along the pixels coalesce)
constexpr int kOut = 16;       // coefficients (encode) or channels (decode) per block

constexpr int kRed = 32;       // terms of the sums staged per step (channels in the projection, coefficients in the inverse)

template <typename TIn>
__global__ void __launch_bounds__(kPx * kOut) project_quantise_kernel(EncodeArgs a, uint8_t *sym)
{
    __shared__ uint8_t s_q[kPx][kOut];
    __shared__ float s_y[kPx][kOut + 1];
    // the operands of kRed terms of every sum of the block: centred pixels and basis entries
    __shared__ double s_d[kRed][kPx];
    __shared__ double s_t[kOut][kRed];
    const int tx = threadIdx.x, ty = threadIdx.y, t = ty * kPx + tx;
    const long long p = (long long)blockIdx.x * kPx + tx;
    const int j = blockIdx.y * kOut + ty;
    const bool valid = p < a.pixels && j < a.k;
    const int nsym = 1 << a.bits;
    const double top = (double)(nsym - 1);
    const TIn *xin = reinterpret_cast<const TIn *>(a.x);
    // staging roles: thread t fetches the centred pixel values (ch, px) = (t / 32, t % 32) and
    // (t / 32 + 16, t % 32) of a step, and the basis entry (coef, ch) = (t / 32, t % 32)
    const long long lp = (long long)blockIdx.x * kPx + tx;
    const bool lp_ok = lp < a.pixels;
    const long long limg = lp_ok ? lp / a.hw : 0;
    const TIn *xp = xin + limg * a.c * (long long)a.hw + (lp_ok ? lp - limg * a.hw : 0);
    const int lj = blockIdx.y * kOut + ty;
    auto fetch = [&](int c0, double &d0, double &d1, double &tv) {
        const int ca = c0 + ty, cb = c0 + ty + 16, ct = c0 + tx;
        d0 = (lp_ok && ca < a.c) ? __dsub_rn(load_as_double(xp + (long long)ca * a.hw), __ldg(a.mean64 + ca)) : 0.0;
        d1 = (lp_ok && cb < a.c) ? __dsub_rn(load_as_double(xp + (long long)cb * a.hw), __ldg(a.mean64 + cb)) : 0.0;
        tv = (lj < a.k && ct < a.c) ? __ldg(a.basis64 + (long long)lj * a.c + ct) : 0.0;
    };
    double acc = 0.0, d0, d1, tv;
    fetch(0, d0, d1, tv);
    for (int c0 = 0; c0 < a.c; c0 += kRed) {
        __syncthreads();                               // the previous step's operands have been used
        s_d[ty][tx] = d0;
        s_d[ty + 16][tx] = d1;
        s_t[ty][tx] = tv;
        __syncthreads();
        if (c0 + kRed < a.c) fetch(c0 + kRed, d0, d1, tv);       // in flight while this step is added up
        const int n = min(kRed, a.c - c0);
        // every sum takes its terms in channel order, one unfused multiply and add each
#pragma unroll 8
        for (int cc = 0; cc < n; ++cc) acc = __dadd_rn(acc, __dmul_rn(s_t[ty][cc], s_d[cc][tx]));
    }
    unsigned int clamped = 0;
    if (valid) {
        const double u = __ddiv_rn(__dsub_rn(acc, a.lo), a.step);
        double r = rint(u);
        if (u < 0.0 || u > top) clamped = 1;
        r = fmin(fmax(r, 0.0), top);
        s_q[tx][ty] = (uint8_t)(unsigned int)r;
        s_y[tx][ty] = (float)acc;
    }
    if (a.clamped) {
        const unsigned int n = __popc(__ballot_sync(0xffffffffu, clamped != 0));
        if (tx == 0 && n) atomicAdd(a.clamped, (unsigned long long)n);
    }
    __syncthreads();
    // a pixel's kOut symbols are contiguous in [P][K]: rows of the block leave in 16-byte pieces
    const int j0 = blockIdx.y * kOut;
    for (int i = t; i < kPx * kOut; i += kPx * kOut) {
        const int px = i / kOut, jj = i - px * kOut;
        const long long pp = (long long)blockIdx.x * kPx + px;
        if (pp < a.pixels && j0 + jj < a.k) {
            const uint8_t q = s_q[px][jj];
            sym[pp * a.k + j0 + jj] = q;
            if (a.dbg_sym) a.dbg_sym[pp * a.k + j0 + jj] = q;
            if (a.dbg_coef) a.dbg_coef[pp * a.k + j0 + jj] = s_y[px][jj];
        }
    }
}

template <typename TOut>
__global__ void __launch_bounds__(kPx * kOut) reconstruct_kernel(DecodeArgs a, const uint8_t *sym)
{
    // symbols of the block's pixels, coefficient-major ([K][kPx]: a warp reads 32 neighbouring bytes)
    extern __shared__ __align__(16) unsigned char s_sym[];
    __shared__ double s_t[kRed][kOut];                 // basis entries of kRed coefficients x the block's channels
    const int tx = threadIdx.x, ty = threadIdx.y, t = ty * kPx + tx;
    const long long p0 = (long long)blockIdx.x * kPx;
    const int n_px = (int)min((long long)kPx, a.pixels - p0);
    for (int i = t; i < n_px * a.k; i += kPx * kOut) {
        const int px = i / a.k, j = i - px * a.k;
        s_sym[j * kPx + px] = sym[p0 * a.k + i];
    }
    const long long p = p0 + tx;
    const int c = blockIdx.y * kOut + ty;
    // staging role: thread t fetches the basis entry (coef, ch) = (t / 16, t % 16) of a step
    const int lj = t / kOut, lc = blockIdx.y * kOut + (t % kOut);
    auto fetch = [&](int j0) { return (j0 + lj < a.k && lc < a.c) ? __ldg(a.basis64 + (long long)(j0 + lj) * a.c + lc) : 0.0; };
    double acc = 0.0, tv = fetch(0);
    for (int j0 = 0; j0 < a.k; j0 += kRed) {
        __syncthreads();                               // symbols staged (first step); the previous step's entries used
        s_t[lj][t % kOut] = tv;
        __syncthreads();
        if (j0 + kRed < a.k) tv = fetch(j0 + kRed);
        const int n = min(kRed, a.k - j0);
        if (tx < n_px) {
#pragma unroll 8
            for (int jj = 0; jj < n; ++jj) {
                const double yh = __dadd_rn(a.lo, __dmul_rn((double)s_sym[(j0 + jj) * kPx + tx], a.step));
                acc = __dadd_rn(acc, __dmul_rn(s_t[jj][ty], yh));
            }
        }
    }
    if (tx >= n_px || c >= a.c) return;
    double v = __dadd_rn(acc, __ldg(a.mean64 + c));
    if (a.relu && v < 0.0) v = 0.0;
    const long long img = p / a.hw;
    TOut *out = reinterpret_cast<TOut *>(a.xhat);
    store_rounded(out + img * a.c * (long long)a.hw + (long long)c * a.hw + (p - img * a.hw), v);
}

// Entropy coder on symbols that already sit in memory ([P][K] bytes), for tensors of few pixels:
// one block per tile of 128 pixels, `parts` threads per pixel, each coding a run of K / parts
// consecutive coefficients (a multiple of 16, so that a thread fetches its symbols in 16-byte
// pieces and a chunk -- one of 1, 2 or 4 runs of a pixel -- is a whole number of thread runs).
// Code lengths first (the lookups of a run are independent loads), then the bit offsets -- runs
// inside a pixel, pixels inside the tile, the tile inside the stream by look-back -- then every
// thread packs its run into the zeroed words of the tile.  Same stream, chunk lengths and tile
// offsets as the one-thread-per-pixel coder.
constexpr int kMaxParts = 8;

__global__ void __launch_bounds__(TC_TILE_PIXELS * kMaxParts) pack_symbols_kernel(EncodeArgs a, const uint8_t *sym, int parts)
{
    __shared__ long long s_tile;
    __shared__ unsigned int s_run_bits[TC_TILE_PIXELS * kMaxParts];
    __shared__ unsigned int s_warp_sums[4];
    __shared__ unsigned int s_pixel_off[TC_TILE_PIXELS + 1];
    __shared__ unsigned long long s_base;
    __shared__ int s_write_ok;
    const int t = threadIdx.x;
    const int nsym = 1 << a.bits;
    if (t == 0) s_tile = (long long)atomicAdd(a.ticket, 1u);
    __syncthreads();
    const long long tile = s_tile;
    const int px = t / parts, part = t - px * parts;          // the threads of a pixel are neighbours
    const long long p = tile * TC_TILE_PIXELS + px;
    const bool valid = p < a.pixels;
    const int run = a.k / parts, j0 = part * run;
    const uint8_t *src = sym + p * a.k + j0;

    unsigned int my_bits = 0;
    if (valid)
        for (int i = 0; i < run; i += 16) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src + i));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                const int j = j0 + i + b;
                const uint32_t q = (w[b >> 2] >> (8 * (b & 3))) & 0xffu;
                my_bits += __ldg(a.enc + (a.groups == 1 ? 0 : j) * nsym + q) & 0xffu;
            }
        }
    s_run_bits[t] = my_bits;
    __syncthreads();
    // pixel totals, scanned by the first 128 threads
    unsigned int tile_bits = 0;
    if (t < TC_TILE_PIXELS) {
        unsigned int pixel_bits = 0;
        for (int r = 0; r < parts; ++r) pixel_bits += s_run_bits[t * parts + r];
        const unsigned int off = group_exclusive_scan_128(pixel_bits, s_warp_sums, t, 1, tile_bits);
        s_pixel_off[t] = off;
        if (t == 0) s_pixel_off[TC_TILE_PIXELS] = tile_bits;
        const unsigned long long padded = ((unsigned long long)tile_bits + 127ull) & ~127ull;
        if (t < 32) {
            bool ok;
            const unsigned long long base = tile_lookback(a.tile_state, tile, padded, a.status, ok);
            if (t == 0) {
                const bool fits = base + padded <= a.capacity_bits;
                if (ok && !fits) tc_dev_set_status(a.status, TC_ERR_BUFFER_TOO_SMALL);
                s_base = base;
                s_write_ok = (ok && fits) ? 1 : 0;
                a.tile_off[tile] = base;
                if (tile == a.n_tiles - 1) a.tile_off[a.n_tiles] = base + padded;
            }
        }
    }
    __syncthreads();
    const unsigned long long base = s_base;
    tile_bits = s_pixel_off[TC_TILE_PIXELS];
    const unsigned long long padded = ((unsigned long long)tile_bits + 127ull) & ~127ull;
    unsigned int my_off = s_pixel_off[px];
    for (int r = 0; r < part; ++r) my_off += s_run_bits[px * parts + r];
    // chunk lengths: a chunk is chunk_pixels pixels, or one of `splits` runs of one pixel
    if (valid) {
        if (a.splits > 1) {
            const int per_chunk = parts / a.splits;
            if (part % per_chunk == 0) {
                unsigned int bits = 0;
                for (int r = 0; r < per_chunk; ++r) bits += s_run_bits[t + r];
                a.chunk_len[p * a.splits + part / per_chunk] = (uint16_t)bits;
            }
        } else if (part == 0 && (p % a.chunk_pixels) == 0) {
            const int last = min(px + a.chunk_pixels, TC_TILE_PIXELS);
            a.chunk_len[p / a.chunk_pixels] = (uint16_t)(s_pixel_off[last] - s_pixel_off[px]);
        }
    }
    if (!s_write_ok) return;
    {
        uint4 *dst = reinterpret_cast<uint4 *>(a.stream + (base >> 5));
        const unsigned int n16 = (unsigned int)(padded >> 7);
        for (unsigned int i = t; i < n16; i += blockDim.x) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    if (valid) {
        BitWriter w;
        w.init(a.stream, base + my_off);
        for (int i = 0; i < run; i += 16) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src + i));
            const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
            uint32_t e[16];
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                const int j = j0 + i + b;
                const uint32_t q = (wd[b >> 2] >> (8 * (b & 3))) & 0xffu;
                e[b] = __ldg(a.enc + (a.groups == 1 ? 0 : j) * nsym + q);
            }
#pragma unroll
            for (int b = 0; b < 16; ++b) w.put(e[b] >> 8, (int)(e[b] & 0xffu));
        }
        w.finish();
    }
}

// Entropy decoder that leaves the symbols in memory ([P][K] bytes), for tensors of few pixels:
// one block per tile, one thread per chunk (up to 512 per tile), so that every chunk of the tile is
// walked at the same time; the inverse transform then runs in reconstruct_kernel.  Same checks as
// the per-pixel decoder: tile offsets aligned, ordered and inside the stream, every chunk inside
// its tile and consumed to exactly its recorded length.
constexpr int kUnpackThreads = 512;

struct GlobalBitReader {
    const uint32_t *words;
    unsigned long long window;   // upcoming bits, left-aligned
    int avail;
    unsigned long long next_word, end_word;
    uint32_t ahead;              // the word behind the window, already loaded: a refill never waits for memory
    __device__ __forceinline__ uint32_t fetch()
    {
        const uint32_t v = (next_word < end_word) ? __ldg(words + next_word) : 0u;   // past the end: zeros, never a load
        ++next_word;
        return v;
    }
    __device__ __forceinline__ void init(const uint32_t *base, unsigned long long bitpos, unsigned long long end_bits)
    {
        words = base;
        next_word = bitpos >> 5;
        end_word = end_bits >> 5;
        const unsigned long long hi = fetch(), lo = fetch();
        ahead = fetch();
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
            window |= (unsigned long long)ahead << (32 - avail);
            avail += 32;
            ahead = fetch();
        }
    }
};

__global__ void __launch_bounds__(kUnpackThreads) unpack_symbols_kernel(DecodeArgs a, uint8_t *sym)
{
    __shared__ unsigned int s_warp_sums[kUnpackThreads / 32];
    extern __shared__ uint16_t s_lut[];                 // a per-layer table is staged (the launch sizes this to it, or to nothing)
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int lut_size = 1 << a.lut_bits;
    const bool lut_staged = a.groups == 1;
    if (lut_staged)
        for (int i = t; i < lut_size; i += kUnpackThreads) s_lut[i] = a.lut[i];
    const long long tile = blockIdx.x;
    const unsigned long long base = a.tile_off[tile], end = a.tile_off[tile + 1];
    const bool tile_ok = (base & 127ull) == 0 && (end & 127ull) == 0 && base <= end && end <= a.stream_bits;
    if (!tile_ok) {
        if (t == 0) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
        return;
    }
    const int chunks_per_tile = a.splits * TC_TILE_PIXELS / a.chunk_pixels;      // at most 512
    const long long ch = tile * chunks_per_tile + t;
    const bool mine = t < chunks_per_tile && ch < a.n_chunks;
    const unsigned int want = mine ? a.chunk_len[ch] : 0u;
    // where the chunk starts: the lengths of the tile's earlier chunks
    unsigned int inc = want;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += up;
    }
    if (lane == 31) s_warp_sums[warp] = inc;
    __syncthreads();
    unsigned int off = inc - want;
    for (int w = 0; w < warp; ++w) off += s_warp_sums[w];
    bool bad = false;
    if (mine) {
        bad = base + off + want > end;
        if (!bad) {
            GlobalBitReader r;
            r.init(a.stream, base + off, end);
            unsigned int used = 0;
            // the chunk's symbols: chunk_pixels whole pixels, or one of `splits` runs of one pixel
            const int run = a.k / a.splits;
            const int first_px = a.splits > 1 ? t / a.splits : t * a.chunk_pixels;
            const int j_first = a.splits > 1 ? (t % a.splits) * run : 0;
            for (int lp = first_px; lp < first_px + (a.splits > 1 ? 1 : a.chunk_pixels); ++lp) {
                const long long p = tile * TC_TILE_PIXELS + lp;
                if (p >= a.pixels) break;
                uint8_t *dst = sym + p * a.k;
                for (int j = j_first; j < j_first + run; ++j) {
                    const uint32_t e = lut_staged ? s_lut[r.peek(a.lut_bits)] : __ldg(a.lut + (size_t)j * lut_size + r.peek(a.lut_bits));
                    const int len = (int)(e & 0xffu);
                    dst[j] = (uint8_t)(e >> 8);
                    r.skip(len);
                    used += len;
                    if (len == 0) bad = true;
                }
            }
            if (used != want) bad = true;
        }
    }
    if (bad) tc_dev_set_status(a.status, TC_ERR_CORRUPT_STREAM);
}

}  // namespace

tc_status tc_launch_project_quantise(const EncodeArgs &a, int dtype, uint8_t *sym, cudaStream_t s)
{
    if (a.pixels <= 0) return TC_OK;
    const dim3 block(kPx, kOut), grid((unsigned int)((a.pixels + kPx - 1) / kPx), (unsigned int)((a.k + kOut - 1) / kOut));
    if (dtype == TC_F32) project_quantise_kernel<float><<<grid, block, 0, s>>>(a, sym);
    else project_quantise_kernel<__nv_bfloat16><<<grid, block, 0, s>>>(a, sym);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_reconstruct(const DecodeArgs &a, int dtype, const uint8_t *sym, cudaStream_t s)
{
    if (a.pixels <= 0) return TC_OK;
    const dim3 block(kPx, kOut), grid((unsigned int)((a.pixels + kPx - 1) / kPx), (unsigned int)((a.c + kOut - 1) / kOut));
    const size_t smem = (size_t)kPx * a.k;
    if (dtype == TC_F32) reconstruct_kernel<float><<<grid, block, smem, s>>>(a, sym);
    else reconstruct_kernel<__nv_bfloat16><<<grid, block, smem, s>>>(a, sym);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

// How many threads per pixel the parallel coder would use for K coefficients and `splits` chunks
// per pixel: the largest of 8, 4, 2, 1 that gives every thread a multiple of 16 coefficients and
// every chunk a whole number of threads (0: none, use the one-thread-per-pixel coder).
int tc_pack_symbols_parts(const EncodeArgs &a)
{
    if (((uintptr_t)a.stream & 15u) != 0) return 0;
    for (int parts = kMaxParts; parts >= 1; parts >>= 1)
        if (a.k % (16 * parts) == 0 && parts % a.splits == 0) return parts;
    return 0;
}

tc_status tc_launch_pack_symbols(const EncodeArgs &a, const uint8_t *sym, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    const int parts = tc_pack_symbols_parts(a);
    if (parts == 0 || ((uintptr_t)sym & 15u) != 0) return TC_ERR_UNSUPPORTED;
    pack_symbols_kernel<<<(unsigned int)a.n_tiles, TC_TILE_PIXELS * parts, 0, s>>>(a, sym, parts);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_launch_unpack_symbols(const DecodeArgs &a, uint8_t *sym, cudaStream_t s)
{
    if (a.n_tiles <= 0) return TC_OK;
    if (a.splits * TC_TILE_PIXELS / a.chunk_pixels > kUnpackThreads) return TC_ERR_UNSUPPORTED;
    const size_t smem = a.groups == 1 ? ((size_t)2 << a.lut_bits) : 0;
    unpack_symbols_kernel<<<(unsigned int)a.n_tiles, kUnpackThreads, smem, s>>>(a, sym);
    return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
