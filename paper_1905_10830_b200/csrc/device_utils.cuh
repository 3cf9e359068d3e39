// Device helpers shared by the codec kernels: block scan of bit lengths, the cross-tile
// look-back that turns tile sizes into stream offsets, and the MSB-first bit writer/reader.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "tc_internal.h"

namespace tcdev {

constexpr unsigned long long kFlagAggregate = 1ull << 62;
constexpr unsigned long long kFlagPrefix = 2ull << 62;
constexpr unsigned long long kValueMask = (1ull << 62) - 1;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // bounded look-back wait: 2 s

__device__ __forceinline__ unsigned long long ld_volatile_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_volatile_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ double load_as_double(const float *p) { return (double)__ldg(p); }
__device__ __forceinline__ double load_as_double(const __nv_bfloat16 *p)
{
    const unsigned short raw = __ldg(reinterpret_cast<const unsigned short *>(p));
    return (double)__uint_as_float((unsigned int)raw << 16);
}

// Round a double to the output type with a single rounding (ties to even).
__device__ __forceinline__ void store_rounded(float *p, double v) { *p = __double2float_rn(v); }
__device__ __forceinline__ void store_rounded(__nv_bfloat16 *p, double v)
{
    // double -> float with round-to-odd keeps enough information for the final RNE to bf16.
    float f = __double2float_rz(v);
    if ((double)f != v) f = __uint_as_float(__float_as_uint(f) | 1u);
    *p = __float2bfloat16_rn(f);
}

// Exclusive scan of one unsigned value per thread over a 128-thread group (4 warps).
// `warp_sums` is 4 words of shared memory; `bar_id`/`bar_threads` name the barrier to use
// (named barrier, so that other warps of the block are not involved).
__device__ __forceinline__ unsigned int group_exclusive_scan_128(unsigned int v, unsigned int *warp_sums,
                                                                int tid128, int bar_id, unsigned int &total)
{
    const int lane = tid128 & 31, warp = tid128 >> 5;
    unsigned int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned int up = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += up;
    }
    if (lane == 31) warp_sums[warp] = inc;
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    unsigned int before = 0, all = 0;
#pragma unroll
    for (int wv = 0; wv < 4; ++wv) {
        const unsigned int s = warp_sums[wv];
        if (wv < warp) before += s;
        all += s;
    }
    total = all;
    return before + inc - v;
}

// Decoupled look-back over per-tile sizes.  A tile first publishes its own padded size
// (lookback_publish, one thread), later one full warp resolves the sum of the sizes of all
// earlier tiles (lookback_resolve) and publishes the inclusive prefix.  Every earlier tile is
// owned by a block that is resident (tickets or a co-resident persistent grid), so the waits
// end; they are bounded all the same, and a wait that runs out clears `ok` and records a
// timeout in the status word.
__device__ __forceinline__ void lookback_publish(unsigned long long *state, long long tile, unsigned long long own)
{
    st_volatile_u64(state + tile, (tile == 0 ? kFlagPrefix : kFlagAggregate) | own);
}

__device__ __forceinline__ unsigned long long lookback_resolve(unsigned long long *state, long long tile,
                                                               unsigned long long own, unsigned int *status, bool &ok)
{
    const int lane = threadIdx.x & 31;
    ok = true;
    if (tile == 0) return 0;
    unsigned long long exclusive = 0;
    long long idx = tile - 1;
    const unsigned long long t0 = global_timer_ns();
    while (true) {
        const long long mine = idx - lane;
        unsigned long long s = kFlagPrefix;   // tiles before the first one: prefix 0
        if (mine >= 0) {
            s = ld_volatile_u64(state + mine);
            while ((s >> 62) == 0) {
                if (global_timer_ns() - t0 > kWaitLimitNs) break;
                __nanosleep(64);
                s = ld_volatile_u64(state + mine);
            }
        }
        const bool timed_out = (s >> 62) == 0;
        if (__any_sync(0xffffffffu, timed_out)) { ok = false; break; }
        const unsigned int prefix_lanes = __ballot_sync(0xffffffffu, (s >> 62) == 2);
        const int first_prefix = prefix_lanes ? (__ffs(prefix_lanes) - 1) : 32;
        unsigned long long contrib = (lane <= first_prefix) ? (s & kValueMask) : 0ull;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) contrib += __shfl_xor_sync(0xffffffffu, contrib, d);
        exclusive += contrib;
        if (prefix_lanes) break;
        idx -= 32;
    }
    if (!ok && lane == 0) tc_dev_set_status(status, TC_ERR_TIMEOUT);
    // publish the inclusive prefix even after a timeout so that later tiles are released
    if (lane == 0) st_volatile_u64(state + tile, kFlagPrefix | ((exclusive + own) & kValueMask));
    return exclusive;
}

__device__ __forceinline__ unsigned long long tile_lookback(unsigned long long *state, long long tile,
                                                            unsigned long long own, unsigned int *status, bool &ok)
{
    if ((threadIdx.x & 31) == 0) lookback_publish(state, tile, own);
    __syncwarp();
    return lookback_resolve(state, tile, own, status, ok);
}

// MSB-first bit writer into a zero-initialised word array.  The first and the last word a
// writer touches may be shared with its neighbours and are merged with atomicOr; words in
// between belong to this writer alone.
struct BitWriter {
    uint32_t *words;           // the (shared or global) word holding the writer's first bit
    unsigned long long acc;    // pending bits, right-aligned
    int pending;               // number of pending bits incl. the lead-in of the first word
    unsigned int word;         // index of the word being filled, relative to `words`
    bool first;

    __device__ __forceinline__ void init(uint32_t *base, unsigned long long bitpos)
    {
        words = base + (bitpos >> 5);
        word = 0;
        pending = (int)(bitpos & 31);
        acc = 0;
        first = true;
    }
    __device__ __forceinline__ void put(uint32_t code, int len)
    {
        acc = (acc << len) | code;
        pending += len;
        if (pending >= 32) {
            const uint32_t out = (uint32_t)(acc >> (pending - 32));
            if (first) { atomicOr(words + word, out); first = false; }
            else words[word] = out;
            ++word;
            pending -= 32;
            acc &= (1ull << pending) - 1ull;
        }
    }
    __device__ __forceinline__ void finish()
    {
        if (pending > 0) {
            const uint32_t out = (uint32_t)(acc << (32 - pending));
            if (out) atomicOr(words + word, out);
        }
    }
};

// MSB-first reader over 32-bit words with a 64-bit window held in two registers.  Words at or
// past `end` read as zero, so a corrupt offset can never cause an out-of-bounds load.
// kShared: the words lie in shared memory (a staged segment) instead of global memory.
template <bool kShared>
struct WindowReaderT {
    const uint32_t *words;
    unsigned long long next, end;     // word indices
    uint32_t hi, lo;                  // upcoming bits, left-aligned in hi:lo
    int avail;                        // valid bits in the window

    __device__ __forceinline__ uint32_t fetch()
    {
        uint32_t w = 0u;
        if (next < end) {
            if constexpr (kShared) w = words[next];
            else w = __ldg(words + next);
        }
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
using WindowReader = WindowReaderT<false>;

}  // namespace tcdev
