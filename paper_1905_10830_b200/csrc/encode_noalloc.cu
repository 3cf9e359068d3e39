// tc_encode_noalloc: tc_encode for callers that are not allowed to allocate device memory.
//
// tc_encode keeps the state of its cross-tile look-back (one 64-bit word per 128-pixel tile,
// plus a ticket counter) in a scratch arena that the context grows with cudaMalloc when a
// larger tensor arrives.  Some users of this library cannot accept that: a serving process
// that reserves its whole memory budget at start-up and treats any later cudaMalloc as a bug;
// a pipeline whose other streams must not be stalled by the device-wide synchronisation that
// cudaMalloc / cudaFree imply; a plug-in running under a host application that owns the
// allocator.  For them the same look-back state lives in a fixed array that is part of the
// library image, so the call touches no allocator at all.
#include <mutex>

#include "tc_internal.h"

namespace {

constexpr size_t kScratchBytes = kEncodeScratchHeader + (size_t)TC_NOALLOC_MAX_TILES * sizeof(unsigned long long);

// Lives in every device that loads the library, from load until the process exits (about 0.5 MB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address; the
// address the kernels need is asked for once per device, with that device current.
constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

tc_status scratch_address(int device, void **out)
{
    if (device < 0 || device >= kMaxDevices) return TC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[device]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return TC_ERR_CUDA;
        }
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    return TC_OK;
}

struct CurrentDevice {
    int prev = -1;
    bool ok = true;
    explicit CurrentDevice(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~CurrentDevice() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" tc_status tc_encode_noalloc(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const tc_tensor *x,
                                       const tc_encode_params *params, void *stream_out, size_t capacity,
                                       uint16_t *chunk_len, uint64_t *tile_off, void *cuda_stream)
{
    if (!ctx || !tile_off) return TC_ERR_INVALID_ARG;
    tc_stream_layout lay;
    tc_status st = tc_encode_bound(m, cb, x, params, &lay);      // argument checks, chunk size (host only)
    if (st != TC_OK) return st;
    if (lay.n_tiles > TC_NOALLOC_MAX_TILES) return TC_ERR_UNSUPPORTED;   // tensor too large for the fixed scratch
    const long long pixels = (long long)x->n * x->h * x->w;
    if (pixels > 0 && (!stream_out || !chunk_len)) return TC_ERR_INVALID_ARG;
    if (((uintptr_t)stream_out & 15u) != 0 || ((uintptr_t)chunk_len & 3u) != 0) return TC_ERR_INVALID_ARG;
    CurrentDevice guard(ctx->device);
    if (!guard.ok) return TC_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (lay.n_tiles == 0) {
        if (cudaMemsetAsync(tile_off, 0, sizeof(uint64_t), s) != cudaSuccess) { cudaGetLastError(); return TC_ERR_CUDA; }
        return TC_OK;
    }
    void *scratch = nullptr;
    if ((st = scratch_address(ctx->device, &scratch)) != TC_OK) return st;
    // The array still holds the previous call's tickets and tile states; the shared dispatch
    // clears, on the stream, everything this call will read, then picks the same kernels as
    // tc_encode (tensor-core kernels with the basis resident or streamed, fp32, fp64).
    return tc_encode_with_scratch(ctx, m, cb, x, lay.chunk_pixels, lay.pixel_splits, stream_out, capacity, chunk_len, tile_off,
                                  nullptr, scratch, /*no arena for symbols: the per-pixel exact kernels*/ nullptr, s);
}
