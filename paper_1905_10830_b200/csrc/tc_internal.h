// Internal declarations shared by the host API and the kernels of the codec library.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "tc.h"

constexpr int TC_TILE_PIXELS = 128;   // pixels per tile = threads per epilogue group
constexpr int TC_MAX_C = 1024;
constexpr int TC_MAX_CODE_LEN = 12;
constexpr int kMaxRoundtripChunks = 64;   // longest code the decode lookup table covers

// Device status word: first error wins.
__device__ __forceinline__ void tc_dev_set_status(unsigned int *status, unsigned int code)
{
    atomicCAS(status, 0u, code);
}

struct tc_ctx {
    int device = 0;
    int sm_count = 0;
    int max_smem_optin = 0;
    unsigned int *d_status = nullptr;     // device status word
    void *scratch = nullptr;              // look-back state, ticket counter
    size_t scratch_bytes = 0;
    void *host_arena = nullptr;           // device staging of tc_roundtrip_host (grown on demand)
    size_t host_arena_bytes = 0;
    // tc_roundtrip_host works through the batch in chunks, two in flight: copy-in and copy-out
    // streams beside the caller's, events that hand a chunk from one to the next, and a small
    // pinned array for the chunks' stream lengths (created at first use)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    unsigned long long *chunk_bits = nullptr;   // pinned HOST [kMaxRoundtripChunks]
    // tc_encode_many / tc_decode_many spread their items over these streams (created at first use)
    cudaStream_t many_streams[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t many_fork = nullptr, many_join[4] = {nullptr, nullptr, nullptr, nullptr};
    int force_exact = 0;                  // 1: route every tensor through the fp64 kernels; 2: skip the resident-basis kernels; 3: skip the run-skipping decoder
    int last_encode_path = 0;             // 0 = fp64 kernels, 1 = tensor-core kernels (resident basis), 2 = fp32 kernels, 3 = tensor-core kernels (streamed basis)
    int last_decode_path = 0;
    tc_codebook *stats_cb[9] = {};        // tc_stats: fixed-length code tables (one per bit width) for streams coded without a codebook
};

struct tc_model {
    int c = 0, k = 0, bits = 0, basis_dtype = 0;
    double lo = 0, step = 0;
    double basis_scale = 1.0;               // 8-bit basis: entries are integers times this; 1 otherwise
    int center = 0;                         // symbol whose level is nearest to y = 0
    // host copies; a model fitted on the device holds its basis there only, and `basis` is filled
    // from d_basis64 the first time the host needs it (export, folding)
    mutable std::vector<double> basis;      // [c][c], or empty
    std::vector<double> mean, eig;          // [c]
    int device = 0;
    // device copies
    double *d_basis64 = nullptr;            // [c][c] exact values of the (rounded) basis
    double *d_mean64 = nullptr;             // [c]
    __nv_bfloat16 *d_basis_bf16 = nullptr;  // [k][c]   bf16 basis, or the integers of an 8-bit basis (exact in bf16)
    __nv_bfloat16 *d_basis_t_bf16 = nullptr;// [c][k]   transpose, for the inverse projection
    float *d_enc_bias = nullptr;            // [k]  -(T mu + lo)_j / step
    float *d_dec_bias = nullptr;            // [c]  mu_c + (lo + center*step) * sum_j T[j][c]
    float *d_tmu32 = nullptr;               // [k]  (T mu)_j
    CUtensorMap basis_map;                  // d_basis_bf16 as a [k][c] tensor, boxes of 256 rows x 32 channels, 64-byte swizzle
    bool has_basis_map = false;
    CUtensorMap basis_t_map;                // d_basis_t_bf16 as a [c][k] tensor, boxes of 128 channel rows x 64 coefficients, 128-byte swizzle
    bool has_basis_t_map = false;
};

struct tc_codebook {
    int bits = 0, groups = 0, max_len = 0, lut_bits = 0;
    int modal = -1;                         // per-layer table: the symbol coded by the single bit 0 (-1: none)
    std::vector<uint8_t> lengths;           // host [groups][2^bits]
    int device = 0;
    uint32_t *d_enc = nullptr;              // [groups][2^bits]  (code << 8) | length
    uint16_t *d_lut = nullptr;              // [groups][2^lut_bits]  (symbol << 8) | length
    uint32_t *d_lut32 = nullptr;            // [groups][2^lut_bits]  bf16(symbol) << 16 | symbol << 8 | length
};

// ---- kernel argument blocks -------------------------------------------------------------

struct EncodeArgs {
    const void *x;
    int n, c, hw, k, bits, groups;
    long long pixels;
    long long n_tiles;
    int chunk_pixels;
    int splits;                 // chunks per pixel (1, 2 or 4; more than 1 only with chunk_pixels == 1)
    const double *basis64;      // [c][c]
    const double *mean64;       // [c]
    const __nv_bfloat16 *basis_bf16;   // [k][c]  (tensor-core path)
    const CUtensorMap *basis_map;      // HOST pointer to the model's tensor map of basis_bf16, or null
    const float *enc_bias;      // [k]  -(T mu + lo)_j / step
    const float *tmu32;         // [k]  (T mu)_j
    double lo, step;
    double basis_scale;         // basis_bf16 holds basis / basis_scale (8-bit basis: integers); 1 otherwise
    const uint32_t *enc;        // [groups][2^bits]
    uint32_t *stream;           // output words
    unsigned long long capacity_bits;
    uint16_t *chunk_len;        // bits of every chunk
    unsigned long long *tile_off;
    float *dbg_coef;            // nullable
    uint8_t *dbg_sym;           // nullable
    unsigned long long *tile_state;   // look-back state, zeroed before launch
    unsigned int *ticket;             // zeroed before launch
    unsigned int *status;
    unsigned long long *clamped;      // nullable: counts coefficients outside the range
    int emit;                         // 0: symbols only (statistics mode)
    const uint8_t *sym_in;            // exact kernels: non-null = the symbols [P][K] are given, skip the projection
    uint8_t *sym_park;                // streaming encoder: non-null = leave the symbols [P][K] here and stop (the entropy coder runs as a kernel of its own)
    unsigned long long *hist;         // tensor-core encoder, statistics: non-null = per-coefficient counts [K][2^bits] of every symbol but hist_modal are added here
    int hist_modal;                   // the symbol of the zero level, which most coefficients hold: statistics mode counts all the others
};

struct DecodeArgs {
    const uint32_t *stream;
    unsigned long long stream_bits;
    const uint16_t *chunk_len;          // bits of every chunk
    int splits;                         // chunks per pixel (1, 2 or 4)
    const unsigned long long *tile_off;
    const uint8_t *symbols;     // non-null: take symbols from here instead of the stream
    uint8_t *sym_out;           // exact kernels: non-null = write the decoded symbols [P][K] there and stop
    int n, c, hw, k, bits, groups;
    long long pixels;
    long long n_tiles, n_chunks;
    int chunk_pixels;
    int lut_bits;
    const uint16_t *lut;
    const uint32_t *lut32;              // tensor-core path
    const __nv_bfloat16 *basis_t_bf16;  // [c][k]
    const CUtensorMap *basis_t_map;     // HOST pointer to the model's tensor map of basis_t_bf16, or null
    const float *dec_bias;              // [c]
    int center;                         // subtracted from every symbol before the MMA
    int modal;                          // per-layer table: the symbol whose code is the single bit 0, or -1 if no code has one bit
    int mean_tile_bytes;                // caller's hint: mean size of a tile's stream segment, 0 = not known
    int dense_head;                     // run-skipping decoder: leading coefficients that are too often non-modal for run skipping to pay
    int relu;                           // x_hat = max(x_hat, 0) before it is rounded to the tensor type
    int smem_budget;                    // shared memory the tensor-core kernel may lay out (set by its launcher)
    int item_pixels;                    // streaming decoder: pixels per work item chosen by its launcher (0: the layout's default)
    const double *basis64;
    const double *mean64;
    double lo, step;
    double basis_scale;                 // basis_t_bf16 holds basis / basis_scale
    void *xhat;
    unsigned int *status;
};

// ---- encode dispatch shared by tc_encode and tc_encode_noalloc (tc_api.cu) --------------------
constexpr size_t kEncodeScratchHeader = 64;   // ticket counter, padded; the per-tile look-back words follow
tc_status tc_encode_with_scratch(tc_ctx *ctx, const tc_model *m, const tc_codebook *cb, const tc_tensor *x, int chunk_pixels,
                                 int splits, void *stream_out, size_t capacity, uint16_t *chunk_len, uint64_t *tile_off,
                                 const tc_debug_out *debug, void *scratch, uint8_t *sym_scratch, cudaStream_t s,
                                 unsigned long long *hist = nullptr, unsigned long long *clamped = nullptr, bool scratch_is_zero = false);
// tensors of fewer tiles than this many per SM take the one-thread-per-value exact kernels
constexpr int kExactParallelTilesPerSm = 2;

// ---- launchers (defined in the .cu files) ----------------------------------------------
tc_status tc_launch_encode_simt(const tc_ctx *ctx, const EncodeArgs &a, int dtype, cudaStream_t s);
tc_status tc_launch_decode_simt(const tc_ctx *ctx, const DecodeArgs &a, int dtype, cudaStream_t s);
tc_status tc_launch_encode_simt_fp32(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s);
tc_status tc_launch_decode_simt_fp32(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s);
tc_status tc_launch_project_quantise(const EncodeArgs &a, int dtype, uint8_t *sym, cudaStream_t s);
int tc_pack_symbols_parts(const EncodeArgs &a);
tc_status tc_launch_unpack_symbols(const DecodeArgs &a, uint8_t *sym, cudaStream_t s);
tc_status tc_launch_pack_symbols(const EncodeArgs &a, const uint8_t *sym, cudaStream_t s);
tc_status tc_launch_reconstruct(const DecodeArgs &a, int dtype, const uint8_t *sym, cudaStream_t s);
bool tc_encode_tc_supported(const tc_ctx *ctx, const EncodeArgs &a);
tc_status tc_launch_encode_tc(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s);
bool tc_decode_tc_supported(const tc_ctx *ctx, const DecodeArgs &a);
tc_status tc_launch_decode_tc(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s);
bool tc_decode_runs_supported(const tc_ctx *ctx, const DecodeArgs &a);
tc_status tc_launch_decode_runs(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s);
bool tc_encode_wide_supported(const tc_ctx *ctx, const EncodeArgs &a);
tc_status tc_launch_encode_wide(const tc_ctx *ctx, const EncodeArgs &a, cudaStream_t s);
bool tc_decode_wide_supported(const tc_ctx *ctx, const DecodeArgs &a);
tc_status tc_launch_decode_wide(const tc_ctx *ctx, const DecodeArgs &a, cudaStream_t s);
size_t tc_decode_tc_staging_bytes(const tc_ctx *ctx, const DecodeArgs &a);     // per tile
size_t tc_decode_runs_staging_bytes(const tc_ctx *ctx, const DecodeArgs &a);   // per tile
size_t tc_decode_wide_staging_bytes(const tc_ctx *ctx, const DecodeArgs &a);   // per tile

tc_status tc_launch_channel_sums(const void *x, int dtype, int n, int c, int hw, double *sums,
                                 cudaStream_t s);
tc_status tc_launch_covariance(const void *x, int dtype, int n, int c, int hw, const double *mean,
                               double *cov, cudaStream_t s);
tc_status tc_launch_range0(const void *x, int dtype, int n, int c, int hw, const double *mean,
                           const double *row0, double *block_minmax, int *n_blocks_out,
                           cudaStream_t s);
int tc_range0_max_blocks(long long pixels);
tc_status tc_launch_histogram(const uint8_t *sym, long long pixels, int k, int groups, int bits,
                              unsigned long long *hist, cudaStream_t s);
tc_status tc_launch_sqerr(const void *x, const void *xhat, int dtype, long long count,
                          double *sum_sq, unsigned long long *zeros, cudaStream_t s);

// ---- host algorithms (host_algos.cpp) ---------------------------------------------------
int tc_huffman_lengths_host(const uint64_t *counts, int nsym, int lmax, uint8_t *len);
void tc_canonical_codes_host(const uint8_t *len, int nsym, uint32_t *code);
int tc_eigh_host(double *a, int n, double *evals, double *evecs);

// ---- fit on the device (eigh_device.cu) ---------------------------------------------------
tc_status tc_launch_moments_to_cov(const double *sum, const double *outer, long long count, int c, double *mean, double *cov,
                                   cudaStream_t s);
tc_status tc_launch_scale_mirror(double *cov, int c, double denom, cudaStream_t s);
size_t tc_eigh_device_workspace_bytes(int c);
tc_status tc_eigh_device(const double *a, int c, double *evals, double *evecs, void *work, int *sweeps_out, cudaStream_t s);
tc_status tc_launch_round_basis(double *basis, int c, int dtype, double *scale_slot, cudaStream_t s);
tc_status tc_launch_model_consts(const double *basis, const double *mean, int c, int k, double lo, double step, double center,
                                 float *enc_bias, float *tmu32, float *dec_bias, cudaStream_t s);
tc_status tc_launch_basis_bf16(const double *basis, int c, int k, double basis_scale, bool int8, void *b, void *bt, cudaStream_t s);
