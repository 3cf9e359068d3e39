/*
 * tc.h -- C ABI of the B200 feature-map transform codec.
 *
 * The library encodes a dense NCHW activation tensor into a Huffman-coded bit stream and
 * decodes it back, following the transform-coding chain of the paper (Section 3):
 *
 *     x -> y = T (x - mu) -> Q_Delta -> VLC -> [memory] -> VLD -> Q_Delta^-1 -> T^T -> x_hat
 *
 * with 1 x 1 x C blocks (Section 3.1, "Linear transform"): every pixel's C-channel vector is
 * transformed on its own, so the transform is a dense (N*H*W) x C x C contraction.
 *
 * Conventions
 *   - Every pointer says whether it is HOST or DEVICE memory.  Device pointers must belong to
 *     the device the context was created on.  The caller owns every buffer it passes in; the
 *     library owns only the opaque handles it returns and a small scratch arena per context.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls that
 *     take one are asynchronous on it unless stated otherwise.
 *   - A context serves one stream at a time: its scratch arena (the cross-tile bookkeeping of
 *     tc_encode, the buffers of tc_stats and tc_roundtrip_host) and its status word are shared by
 *     all calls made on it, so two calls on the same context that could overlap on the GPU --
 *     different streams, no dependency between them -- corrupt each other's output.  Use one
 *     context per concurrent stream; models and codebooks may be shared between contexts of the
 *     same device.
 *   - Errors are return codes.  Argument errors are found on the host before any launch.
 *     Conditions only the device can see (corrupt stream, output capacity exceeded at run
 *     time, a bounded wait that ran out) are recorded in a per-context status word and
 *     reported by tc_get_status(); the kernels never read or write out of bounds because of
 *     them and never trap.
 *   - There is no CPU fallback: without a CUDA device tc_create() fails.
 *   - P = N*H*W pixels, pixel index p = (n*H + h)*W + w; K = number of coefficients kept
 *     (K <= C); V = P*C values; b = quantiser bit width.
 */
#ifndef TC_H_
#define TC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TC_OK = 0,
    TC_ERR_INVALID_ARG = 1,      /* null pointer, bad shape, mismatched model/codebook        */
    TC_ERR_UNSUPPORTED = 2,      /* b outside 1..8, C > 1024, code longer than 12 bits, ...   */
    TC_ERR_BUFFER_TOO_SMALL = 3, /* stream capacity exceeded (host check or device status)    */
    TC_ERR_CUDA = 4,             /* a CUDA runtime call failed                                */
    TC_ERR_CORRUPT_STREAM = 5,   /* decode found offsets or codes that cannot be valid        */
    TC_ERR_TIMEOUT = 6,          /* a bounded device-side wait ran out                        */
    TC_ERR_NOT_CONVERGED = 7     /* eigensolver did not converge                              */
} tc_status;

/* Element types.  TC_INT8 is not a tensor type: it only names the 8-bit basis of a model. */
typedef enum { TC_F32 = 0, TC_BF16 = 1, TC_INT8 = 2 } tc_dtype;

/* Dense NCHW tensor in DEVICE memory.  `data` must be aligned to its element size; bf16 tensors
 * that start on an 8-byte boundary (any allocation does; a view at an odd element offset may
 * not) and have H*W % 4 == 0 are moved four pixels at a time, others element by element. */
typedef struct {
    void *data;
    int32_t n, c, h, w;
    int32_t dtype; /* tc_dtype */
} tc_tensor;

typedef struct tc_ctx tc_ctx;
typedef struct tc_model tc_model;
typedef struct tc_codebook tc_codebook;

/* Context: binds a device, owns the scratch arena and the device status word. */
tc_status tc_create(tc_ctx **out, int device);
void tc_destroy(tc_ctx *ctx);
const char *tc_status_string(tc_status s);

/* Synchronises `cuda_stream`, returns the first device-side error recorded since the last
 * call (TC_OK if none) and clears it. */
tc_status tc_get_status(tc_ctx *ctx, void *cuda_stream);

/* Validation switch.  bf16 tensors normally take the tensor-core kernels (bf16 products, fp32
 * accumulation): up to 256 channels with rows of H*W % 4 == 0 elements the kernels that keep
 * the basis in shared memory, wider layers (up to 1024 channels) and other map sizes the
 * kernels that stream it; shapes neither takes (channel or coefficient counts that are not
 * multiples of 16) run on plain fp32 kernels with the same arithmetic.  fp32 tensors run on
 * kernels that evaluate the definition in fp64.  With `on` == 1 every tensor takes the fp64
 * kernels; with `on` == 2 bf16 tensors skip the resident-basis kernels, so that the streaming
 * kernels can be checked on the shapes both take; 0 restores the default. */
void tc_force_exact_path(tc_ctx *ctx, int on);
/* Which kernels the last tc_encode (decode == 0) or tc_decode (decode != 0) of this context
 * launched: 0 = fp64 kernels, 1 = tensor-core kernels with the basis resident in shared
 * memory, 2 = fp32 kernels, 3 = tensor-core kernels that stream the basis; -1 for a NULL
 * context. */
int tc_last_path(const tc_ctx *ctx, int decode);

/* ---------------------------------------------------------------------------------------
 * Model = per-layer transform and quantiser (Section 3; Section 3.1 "Linear transform" and
 * "Quantization"): mean mu[C]; basis T[C][C] whose row j is the j-th principal direction of
 * the calibration covariance (descending eigenvalue, orthonormal, T^-1 = T^T); the common
 * quantiser step Delta and lowest level lo, taken from the range of coefficient 0 (the
 * highest-variance channel) on the calibration maps: step = (hi - lo) / (2^b - 1).
 * ------------------------------------------------------------------------------------- */
typedef struct {
    int32_t bits;        /* b, 1..8                                                        */
    int32_t k;           /* coefficients kept, 1..C; 0 means C                             */
    int32_t basis_dtype; /* tc_dtype: the basis is rounded to this type at fit time and
                            the rounded matrix is the transform from then on.  TC_BF16 is
                            required for bf16 tensors, TC_F32 for fp32 tensors.  TC_INT8
                            (Section 3.1: the PCA matrix is stored in 8 bits) serves both:
                            one scale s = max|T| / 127 for the matrix, every entry becomes
                            s * n with n an integer in [-127, 127]; the decoder uses the
                            transpose of the same matrix.                                   */
    int32_t zero_level;  /* non-zero: the quantiser grid lo + q * step is shifted by at most half
                            a step so that y = 0 is one of its levels: lo = -step * n with
                            n = round(-lo_measured / step), ties to even.  The coefficients are
                            zero-mean and most of them tiny after the PCA; with zero on a level
                            a low-variance channel maps to a single value (Appendix E), with zero
                            between two levels it flips between both, which costs rate and
                            distortion.  0 keeps lo at the calibration minimum.                */
    int32_t eigensolver; /* TC_EIG_DEVICE (0): one-sided Jacobi on the device, no C x C matrix
                            crosses to the host during the fit.  TC_EIG_HOST (1): the
                            covariance is copied to the host and solved there (Householder
                            tridiagonalisation + implicit QR, tc_host_eigh).  Both return the
                            same decomposition up to rounding.                                  */
} tc_fit_params;
enum { TC_EIG_DEVICE = 0, TC_EIG_HOST = 1 };

/* Fit on calibration maps (`calib->n` maps).  Mean and covariance (1/(M-1), M = n*h*w pixel
 * vectors) are accumulated on the device in fp64, the eigendecomposition runs there too
 * (params->eigensolver), the basis is rounded and the range of coefficient 0 taken on the
 * device; the model keeps its basis on the device and copies it to the host only when
 * tc_model_export or a fold asks for it.  Synchronous: returns after the model is complete.  Errors: INVALID_ARG, UNSUPPORTED (C > 1024 or C % 8 != 0 ... see
 * tc_encode), NOT_CONVERGED, CUDA. */
tc_status tc_fit_pca(tc_ctx *ctx, const tc_tensor *calib, const tc_fit_params *params,
                     tc_model **out, void *cuda_stream);

/* Online fit (Section 3.1, "Linear transform": the covariance is estimated on calibration
 * data and "can be updated online").  The running state is the sample count M, the sum of the
 * pixel vectors s[C] and the sum of their outer products S[C][C], held in fp64 on the device.
 * A further batch only adds to the three, so the state can be carried across batches,
 * checkpointed, and merged with the states of other devices by adding them (one all-reduce of
 * count, s and S -- at most 8.4 MB at C = 1024).
 *   tc_fit_state_create  zeroed state for C channels.
 *   tc_fit_state_update  adds the N*H*W pixel vectors of `maps` (DEVICE tensor, fp32 or bf16,
 *                        C channels); asynchronous on `cuda_stream`.
 *   tc_fit_state_export  synchronises and copies the state to HOST arrays sum[C],
 *                        outer[C][C] (full symmetric matrix) and *count.
 *   tc_fit_state_import  replaces the state by HOST arrays (for example the sum over devices).
 *   tc_fit_state_finish  mean = s / M, covariance = (S - s s^T / M) / (M - 1), then as
 *                        tc_fit_pca: eigendecomposition (on the device unless
 *                        params->eigensolver says otherwise), basis rounded to
 *                        params->basis_dtype, quantiser range from coefficient 0 over
 *                        `range_maps` (DEVICE tensor; the basis is not known while the state
 *                        is being accumulated, so the caller names the maps the range is
 *                        measured on, for instance the last calibration batch).  Synchronous.
 * Errors: INVALID_ARG (shape mismatch, fewer than two samples, constant range maps),
 * UNSUPPORTED (C > 1024, bits outside 1..8), NOT_CONVERGED, CUDA. */
typedef struct tc_fit_state tc_fit_state;
tc_status tc_fit_state_create(tc_ctx *ctx, int32_t c, tc_fit_state **out);
void tc_fit_state_free(tc_fit_state *state);
tc_status tc_fit_state_update(tc_ctx *ctx, tc_fit_state *state, const tc_tensor *maps, void *cuda_stream);
tc_status tc_fit_state_export(tc_ctx *ctx, const tc_fit_state *state, int64_t *count, double *sum,
                              double *outer, void *cuda_stream);
tc_status tc_fit_state_import(tc_ctx *ctx, tc_fit_state *state, int64_t count, const double *sum,
                              const double *outer, void *cuda_stream);
tc_status tc_fit_state_finish(tc_ctx *ctx, const tc_fit_state *state, const tc_tensor *range_maps,
                              const tc_fit_params *params, tc_model **out, void *cuda_stream);

/* Plain HOST description of a model, for import/export (checkpointing, and the injection
 * point for externally computed models).  `basis` is [C][C] row-major, rows = directions;
 * entries must already be exactly representable in `basis_dtype` (import rejects others). */
typedef struct {
    int32_t c, k, bits, basis_dtype;
    double lo, step;
    double *basis; /* HOST [c*c] */
    double *mean;  /* HOST [c]   */
    double *eig;   /* HOST [c], may be NULL on import */
    double basis_scale; /* TC_INT8 basis: the scale s (every basis entry is an integer in
                           [-127, 127] times s, checked on import); otherwise ignored on
                           import and 1.0 on export */
} tc_model_desc;

tc_status tc_model_import(tc_ctx *ctx, const tc_model_desc *desc, tc_model **out);
/* Fills the scalar fields and, where the caller set the array pointers, the arrays. */
tc_status tc_model_export(const tc_model *model, tc_model_desc *desc);
void tc_model_free(tc_model *model);

/* Folding (Section 3.1, "Linear transform": with 1 x 1 x C blocks the PCA is a 1 x 1
 * convolution and can be folded, like the batch normalisation, into the convolution that
 * produces the feature map; the inverse transform folds into the convolution that reads it).
 * Offline helpers on HOST arrays, fp64, no device work.
 *
 * tc_fold_forward: the producing layer computes z_c = scale_c (sum_f W[c][f] u_f + bias_c) +
 * shift_c, f over the `fan` = C_in * kernel positions (`w` is [C][fan] row-major; scale/shift
 * are the batch normalisation as an affine map; bias, scale, shift may be NULL = 0, 1, 0), and
 * the encoder y = T (z - mu).  Out: w_folded [K][fan], bias_folded [K] with
 * y_j = sum_f w_folded[j][f] u_f + bias_folded[j].
 *
 * tc_fold_inverse: a next layer that reads x_hat = T^T y_hat + mu directly (no non-linearity
 * in between) computes v_o = sum_{c,t} w_next[o][c][t] x_hat_c(t) + bias_next[o], t over the
 * `taps` kernel positions (`w_next` is [c_out][C][taps]).  Out: w_folded [c_out][K][taps],
 * bias_folded [c_out] with v_o = sum_{j,t} w_folded[o][j][t] y_hat_j(t) + bias_folded[o]; the
 * constant is exact where every tap lies inside the map (zero padding breaks it at the border).
 * Errors: INVALID_ARG. */
tc_status tc_fold_forward(const tc_model *model, const double *w, const double *bias, const double *scale,
                          const double *shift, int64_t fan, double *w_folded, double *bias_folded);
tc_status tc_fold_inverse(const tc_model *model, const double *w_next, const double *bias_next, int32_t c_out,
                          int32_t taps, double *w_folded, double *bias_folded);

/* ---------------------------------------------------------------------------------------
 * Codebook = canonical Huffman code for the quantiser output (Section 3.1, "Variable
 * length coding").  `groups` is 1 (one table per layer) or K (one table per coefficient
 * channel).  Lengths come from counts + 1 (every symbol has a code) by Huffman's algorithm
 * with deterministic tie-breaking -- leaves sorted by (weight, symbol), a leaf before an
 * internal node of equal weight -- and, if the longest code would exceed `max_length`, by the
 * length-limited optimum (package-merge).  Codes are canonical: ordered by (length, symbol).
 * ------------------------------------------------------------------------------------- */
typedef struct {
    int32_t groups;     /* 1 or K                                  */
    int32_t max_length; /* b..12; 0 means 12                       */
} tc_codebook_params;

/* `hist` is [groups][2^b] counts, HOST memory if hist_on_device == 0 else DEVICE memory.
 * Synchronous. */
tc_status tc_build_codebook(tc_ctx *ctx, const tc_model *model, const uint64_t *hist,
                            int hist_on_device, const tc_codebook_params *params,
                            tc_codebook **out);
/* `lengths` is HOST [groups][2^bits]; must satisfy Kraft's equality per group and be <= 12. */
tc_status tc_codebook_import(tc_ctx *ctx, int32_t bits, int32_t groups, const uint8_t *lengths,
                             tc_codebook **out);
/* `lengths` may be NULL to query bits/groups only. */
tc_status tc_codebook_export(const tc_codebook *cb, int32_t *bits, int32_t *groups,
                             uint8_t *lengths);
void tc_codebook_free(tc_codebook *cb);

/* Host utility behind tc_build_codebook: code lengths for one alphabet of `nsym` symbols
 * from `counts` (weights counts + 1).  HOST pointers.  No device needed. */
tc_status tc_host_huffman_lengths(const uint64_t *counts, int32_t nsym, int32_t max_length,
                                  uint8_t *lengths);
/* The fit's device eigensolver on its own (Section 3.1, "Linear transform": the PCA matrix is
 * the eigenvector matrix of the calibration covariance): `a` is a symmetric n x n matrix in DEVICE memory
 * (fp64, row-major, left untouched), evals [n] and evecs [n][n] DEVICE arrays, with the same
 * conventions as tc_host_eigh.  One-sided Jacobi, one launch per round of n / 2 disjoint
 * column pairs; synchronises the stream once per sweep.  *sweeps (HOST, may be NULL) receives
 * the number of sweeps.  Errors: INVALID_ARG, NOT_CONVERGED (150 sweeps), CUDA. */
tc_status tc_device_eigh(tc_ctx *ctx, const double *a, int32_t n, double *evals, double *evecs, int32_t *sweeps,
                         void *cuda_stream);
/* Host eigensolver (TC_EIG_HOST): eigendecomposition of a symmetric n x n matrix `a`
 * (HOST, row-major, destroyed).  On return evals[] is descending and row j of `evecs`
 * ([n][n]) is the unit eigenvector of evals[j], signed so that its largest-magnitude entry
 * is positive.  No device needed. */
tc_status tc_host_eigh(double *a, int32_t n, double *evals, double *evecs);

/* ---------------------------------------------------------------------------------------
 * Bit stream (the paper leaves the layout open; Section 3.1 only says the stream is
 * accumulated in external memory).
 *   - Symbols are emitted pixel-major: p ascending, coefficient j ascending inside a pixel,
 *     each with the code of table j (groups == K) or table 0.
 *   - Code bits most-significant first; stream bit i is bit 31 - (i mod 32) of the
 *     little-endian 32-bit word i / 32.
 *   - A tile is 128 pixels.  Tile t starts at absolute bit tile_off[t], a multiple of 128,
 *     with zero padding before it; tile_off[n_tiles] is the padded end of the stream.
 *   - A chunk is the unit a decoder thread starts from: `chunk_pixels` consecutive pixels (a
 *     power of two, 1..128), or, with chunk_pixels == 1, one of `pixel_splits` equal runs of
 *     a pixel's K coefficients (pixel_splits 1, 2 or 4; K a multiple of 8 * pixel_splits).
 *     Chunks are numbered in stream order; chunk_len[i] is the length of chunk i in bits, and
 *     inside a tile the chunks follow one another without gaps, so a chunk starts at its
 *     tile's start plus the lengths of the tile's earlier chunks.  A chunk may not exceed
 *     65535 bits: chunk_pixels * K / pixel_splits * (longest code) must stay below that.
 *   - Defaults (chunk_pixels = pixel_splits = 0): the smallest chunk_pixels that gives a chunk at
 *     least 96 symbols; from 256 coefficients on two chunks per pixel (K a multiple of 32),
 *     from 512 on four (K a multiple of 64).  tc_encode_bound reports what will be used.
 * ------------------------------------------------------------------------------------- */
typedef struct {
    int32_t chunk_pixels; /* power of two in 1..128; 0 = library default for this shape   */
    int32_t pixel_splits; /* 1, 2 or 4 (needs chunk_pixels == 1); 0 = library default      */
    int32_t relu;         /* tc_decode / tc_roundtrip_host only: non-zero applies the layer's
                             non-linearity after the inverse transform (Section 3.1),
                             x_hat = max(T^T y_hat + mu, 0), before rounding to the tensor type */
    int32_t mean_tile_bytes; /* tc_decode only, a hint that changes speed, never results: the mean size
                             of a tile's stream segment in bytes (stream length / n_tiles), 0 = not
                             known.  It matters for per-channel code tables on layers of up to 256
                             channels: the decoder that keeps the basis in shared memory stages
                             segments of up to about 14 KB there and reads longer ones from global
                             memory word by word, the decoder that streams the basis stages up to
                             32 KB; told that the segments are long, tc_decode picks the second.
                             tc_decode never infers the rate from `stream_bytes` (which may be the
                             length of the stream or the capacity of its buffer).            */
} tc_encode_params;

typedef struct {
    int64_t n_tiles, n_chunks;
    size_t stream_bytes;    /* worst case: every symbol at the longest code + padding  */
    size_t chunk_len_bytes; /* n_chunks * 2                                            */
    size_t tile_off_bytes;  /* (n_tiles + 1) * 8                                       */
    int32_t chunk_pixels;   /* the values that will be used                            */
    int32_t pixel_splits;
} tc_stream_layout;

/* Worst-case buffer sizes for encoding `x`. Host only.  INVALID_ARG for a chunk shape the
 * format cannot hold (see above). */
tc_status tc_encode_bound(const tc_model *model, const tc_codebook *cb, const tc_tensor *x,
                          const tc_encode_params *params, tc_stream_layout *out);

/* Optional debug outputs of tc_encode (DEVICE): the projected coefficients and the symbols,
 * which the normal path never writes to memory.  Either pointer may be NULL. */
typedef struct {
    float *coefficients; /* [P][K] fp32: y = T (x - mu) */
    uint8_t *symbols;    /* [P][K]                      */
} tc_debug_out;

/* Encode (Section 3: transform, quantiser, VLC).  One pass: stage, project, quantise, look up
 * codes, scan bit offsets, pack and store.
 *   stream_out  DEVICE, 16-byte aligned, `capacity` bytes; any capacity is accepted -- if
 *               the coded tensor does not fit, nothing is written past it and the status
 *               word records TC_ERR_BUFFER_TOO_SMALL.  tc_encode_bound() never fails.
 *   chunk_len   DEVICE uint16[n_chunks], 4-byte aligned;  tile_off  DEVICE uint64[n_tiles + 1]
 *               (tile_off[n_tiles] = total stream length in bits).
 * Errors: INVALID_ARG, UNSUPPORTED (C > 1024, dtype /
 * basis_dtype mismatch), CUDA. */
tc_status tc_encode(tc_ctx *ctx, const tc_model *model, const tc_codebook *cb,
                    const tc_tensor *x, const tc_encode_params *params, void *stream_out,
                    size_t capacity, uint16_t *chunk_len, uint64_t *tile_off,
                    const tc_debug_out *debug, void *cuda_stream);

/* tc_encode without any allocation.  (The paper has no counterpart: this entry point exists
 * for the sake of how the library is deployed, not of the method.)
 *
 * tc_encode keeps its cross-tile bookkeeping in a scratch arena that the context enlarges with
 * cudaMalloc when a bigger tensor arrives.  Callers that may not allocate -- a server that
 * fixes its memory budget at start-up, a pipeline that cannot afford the device-wide stall of
 * cudaMalloc / cudaFree next to its other streams, a plug-in whose host owns the allocator --
 * use this variant instead: the bookkeeping lives in a fixed array inside the library image
 * (about 0.5 MB on every GPU that loads the library, held until the process exits), and the
 * call runs no cudaMalloc, cudaFree or other allocating routine.
 *   - Same arguments, outputs, asynchrony and errors as tc_encode, minus the debug outputs.
 *   - Tensors of more than TC_NOALLOC_MAX_TILES tiles of 128 pixels (N*H*W > 8 388 608
 *     pixels) are refused with TC_ERR_UNSUPPORTED; nothing is launched.
 *   - The first call on a device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device, from every context, share the one array (it is cleared on the
 *     stream at the start of each call).  Two calls that can overlap on the GPU -- different
 *     streams, no dependency -- race on it and corrupt each other's streams: serialise them. */
#define TC_NOALLOC_MAX_TILES 65536
tc_status tc_encode_noalloc(tc_ctx *ctx, const tc_model *model, const tc_codebook *cb,
                            const tc_tensor *x, const tc_encode_params *params, void *stream_out,
                            size_t capacity, uint16_t *chunk_len, uint64_t *tile_off,
                            void *cuda_stream);

/* Decode (Section 3: VLD, inverse quantiser, inverse transform; params->relu adds the ReLU that
 * follows the decoder in Section 3.1, off by default).
 *   stream       DEVICE, 16-byte aligned, `stream_bytes` readable bytes
 *   x_hat        caller-allocated tensor of the shape and dtype that was encoded
 * Offsets and lengths are validated on the device (tile offsets against `stream_bytes`, the
 * chunk lengths of a tile against the tile's size, and every chunk must decode to exactly
 * its recorded length); a stream that fails sets TC_ERR_CORRUPT_STREAM in the status word and
 * leaves the affected tile's output unspecified (but in bounds). */
tc_status tc_decode(tc_ctx *ctx, const tc_model *model, const tc_codebook *cb, const void *stream,
                    size_t stream_bytes, const uint16_t *chunk_len, const uint64_t *tile_off,
                    const tc_encode_params *params, const tc_tensor *x_hat, void *cuda_stream);

/* Several tensors per call (Section 3.1: every layer has its own encoder and decoder -- its own
 * PCA matrix, range and code table -- and an inference pass codes them all).  A network's
 * layers at a small batch are each too small to fill the GPU, and a call per layer pays the
 * launch and set-up time of its kernels one after the other.  These entry points take the
 * whole list: the items are checked first (nothing is launched if one is invalid), the
 * bookkeeping of all of them is cleared at once, and their kernels are spread, largest first,
 * over four streams of the context so that small layers run beside one another; `cuda_stream`
 * waits for all of them, so later work on it sees every output.  The results are those of
 * tc_encode / tc_decode called per item (same arguments, same errors; the first error is
 * returned after all items that could be launched have been).  Output buffers of different
 * items must not overlap.  tc_last_path reports the route of the item launched last. */
typedef struct {
    const tc_model *model;
    const tc_codebook *codebook;
    const tc_tensor *x;
    const tc_encode_params *params; /* may be NULL */
    void *stream_out;               /* DEVICE, 16-byte aligned, `capacity` bytes */
    size_t capacity;
    uint16_t *chunk_len;            /* DEVICE uint16[n_chunks], 4-byte aligned   */
    uint64_t *tile_off;             /* DEVICE uint64[n_tiles + 1]                */
} tc_encode_item;
typedef struct {
    const tc_model *model;
    const tc_codebook *codebook;
    const void *stream;             /* DEVICE, 16-byte aligned */
    size_t stream_bytes;
    const uint16_t *chunk_len;
    const uint64_t *tile_off;
    const tc_encode_params *params; /* may be NULL */
    const tc_tensor *x_hat;
} tc_decode_item;
tc_status tc_encode_many(tc_ctx *ctx, const tc_encode_item *items, int32_t n_items, void *cuda_stream);
tc_status tc_decode_many(tc_ctx *ctx, const tc_decode_item *items, int32_t n_items, void *cuda_stream);

/* Whole chain on HOST tensors (Section 3: encoder, memory, decoder): copies `x_host` (dense
 * NCHW, `dtype`, pinned memory recommended) to the device, encodes, decodes and copies the
 * reconstruction to `x_hat_host`, then synchronises `cuda_stream`.  Larger batches are worked
 * through in chunks of whole tiles (about 24 MB of images each, at most 64 chunks), two in
 * flight: the kernels run on `cuda_stream` while the next chunk is copied in and the previous
 * one is copied out on two streams the context creates at the first call, so that both
 * directions of the host link are busy at once; the result and the stream length are those of
 * one pass over the whole tensor.  The device buffers (two slots of tensor, reconstruction,
 * worst-case stream, lengths and offsets) live in a context-owned arena that grows with
 * cudaMalloc when a larger chunk arrives.  `stream_bits` (HOST, may be NULL) receives the
 * length of the coded stream.  Returns the first host- or device-side error. */
tc_status tc_roundtrip_host(tc_ctx *ctx, const tc_model *model, const tc_codebook *cb,
                            const void *x_host, void *x_hat_host, int32_t n, int32_t c, int32_t h,
                            int32_t w, int32_t dtype, const tc_encode_params *params,
                            uint64_t *stream_bits, void *cuda_stream);

/* ---------------------------------------------------------------------------------------
 * Statistics (Section 3: rate and MSE distortion D = |x - x_hat|^2 / n; Section 3.1: entropy
 * H = -sum p log2 p as the theoretical rate; Appendix G: eigenvalue energy ratio).
 * Synchronous.  `hist` (DEVICE, uint64 [groups][2^b], may be NULL) receives the symbol
 * counts of `x` -- the input of tc_build_codebook.
 * ------------------------------------------------------------------------------------- */
typedef struct {
    int32_t groups;        /* in: 1 or K -- granularity of `hist`                          */
    uint64_t *hist;        /* in: DEVICE [groups][2^b] or NULL; overwritten                */
    double entropy;        /* out: bits/value, mean over groups of the group entropies     */
    double mean_length;    /* out: Huffman bits/value with `cb` (0 if cb == NULL)          */
    double mse;            /* out: mean squared error of the round trip (stored dtype)     */
    double clamped_fraction; /* out: fraction of coefficients outside the quantiser range  */
    double zero_fraction;  /* out: fraction of input values equal to zero                  */
    double energy_ratio_90;/* out: fraction of eigenvalues holding 90 % of the energy      */
} tc_stats_out;

tc_status tc_stats(tc_ctx *ctx, const tc_model *model, const tc_codebook *cb, const tc_tensor *x,
                   tc_stats_out *out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TC_H_ */
