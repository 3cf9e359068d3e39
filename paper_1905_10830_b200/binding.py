"""ctypes binding of libtc_b200.so.  Function names match the C ABI (include/tc.h)."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libtc_b200.so")

TC_F32, TC_BF16, TC_INT8 = 0, 1, 2       # TC_INT8 only names the 8-bit basis of a model
TC_EIG_DEVICE, TC_EIG_HOST = 0, 1
_STATUS = ["ok", "invalid argument", "unsupported configuration", "output buffer too small",
           "CUDA error", "corrupt stream", "device-side wait timed out",
           "eigensolver did not converge"]


class TcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = _STATUS[code] if 0 <= code < len(_STATUS) else f"status {code}"
        super().__init__(f"{where}: {name}")


class _Tensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("n", C.c_int32), ("c", C.c_int32), ("h", C.c_int32),
                ("w", C.c_int32), ("dtype", C.c_int32)]


class _FitParams(C.Structure):
    _fields_ = [("bits", C.c_int32), ("k", C.c_int32), ("basis_dtype", C.c_int32), ("zero_level", C.c_int32),
                ("eigensolver", C.c_int32)]


class _ModelDesc(C.Structure):
    _fields_ = [("c", C.c_int32), ("k", C.c_int32), ("bits", C.c_int32), ("basis_dtype", C.c_int32),
                ("lo", C.c_double), ("step", C.c_double), ("basis", C.c_void_p),
                ("mean", C.c_void_p), ("eig", C.c_void_p), ("basis_scale", C.c_double)]


class _CodebookParams(C.Structure):
    _fields_ = [("groups", C.c_int32), ("max_length", C.c_int32)]


class _EncodeParams(C.Structure):
    _fields_ = [("chunk_pixels", C.c_int32), ("pixel_splits", C.c_int32), ("relu", C.c_int32), ("mean_tile_bytes", C.c_int32)]


class _StreamLayout(C.Structure):
    _fields_ = [("n_tiles", C.c_int64), ("n_chunks", C.c_int64), ("stream_bytes", C.c_size_t),
                ("chunk_len_bytes", C.c_size_t), ("tile_off_bytes", C.c_size_t),
                ("chunk_pixels", C.c_int32), ("pixel_splits", C.c_int32)]


class _DebugOut(C.Structure):
    _fields_ = [("coefficients", C.c_void_p), ("symbols", C.c_void_p)]


class _StatsOut(C.Structure):
    _fields_ = [("groups", C.c_int32), ("hist", C.c_void_p), ("entropy", C.c_double),
                ("mean_length", C.c_double), ("mse", C.c_double), ("clamped_fraction", C.c_double),
                ("zero_fraction", C.c_double), ("energy_ratio_90", C.c_double)]


EXPORTS = ["tc_create", "tc_destroy", "tc_status_string", "tc_get_status", "tc_force_exact_path", "tc_last_path", "tc_fit_pca",
           "tc_model_import", "tc_model_export", "tc_model_free", "tc_build_codebook",
           "tc_codebook_import", "tc_codebook_export", "tc_codebook_free",
           "tc_host_huffman_lengths", "tc_host_eigh", "tc_device_eigh", "tc_encode_bound", "tc_encode", "tc_encode_noalloc", "tc_decode", "tc_encode_many", "tc_decode_many", "tc_roundtrip_host",
           "tc_stats", "tc_fit_state_create", "tc_fit_state_free", "tc_fit_state_update", "tc_fit_state_export",
           "tc_fit_state_import", "tc_fit_state_finish", "tc_fold_forward", "tc_fold_inverse"]

_lib = None


def library_path() -> str:
    return _LIB_PATH


def load_library() -> C.CDLL:
    """Load the CUDA library.  There is no fallback: a missing build is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_1905_10830_b200.build` "
                              "(there is no CPU fallback)")
        lib = C.CDLL(_LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        P = C.POINTER
        lib.tc_create.argtypes = [P(vp), C.c_int]
        lib.tc_destroy.argtypes = [vp]
        lib.tc_destroy.restype = None
        lib.tc_status_string.argtypes = [C.c_int]
        lib.tc_status_string.restype = C.c_char_p
        lib.tc_get_status.argtypes = [vp, vp]
        lib.tc_force_exact_path.argtypes = [vp, C.c_int]
        lib.tc_force_exact_path.restype = None
        lib.tc_last_path.argtypes = [vp, C.c_int]
        lib.tc_fit_pca.argtypes = [vp, P(_Tensor), P(_FitParams), P(vp), vp]
        lib.tc_model_import.argtypes = [vp, P(_ModelDesc), P(vp)]
        lib.tc_model_export.argtypes = [vp, P(_ModelDesc)]
        lib.tc_model_free.argtypes = [vp]
        lib.tc_model_free.restype = None
        lib.tc_build_codebook.argtypes = [vp, vp, vp, C.c_int, P(_CodebookParams), P(vp)]
        lib.tc_codebook_import.argtypes = [vp, i32, i32, vp, P(vp)]
        lib.tc_codebook_export.argtypes = [vp, P(i32), P(i32), vp]
        lib.tc_codebook_free.argtypes = [vp]
        lib.tc_codebook_free.restype = None
        lib.tc_host_huffman_lengths.argtypes = [vp, i32, i32, vp]
        lib.tc_host_eigh.argtypes = [vp, i32, vp, vp]
        lib.tc_encode_many.argtypes = [vp, vp, i32, vp]
        lib.tc_decode_many.argtypes = [vp, vp, i32, vp]
        lib.tc_device_eigh.argtypes = [vp, vp, i32, vp, vp, P(i32), vp]
        lib.tc_encode_bound.argtypes = [vp, vp, P(_Tensor), P(_EncodeParams), P(_StreamLayout)]
        lib.tc_encode.argtypes = [vp, vp, vp, P(_Tensor), P(_EncodeParams), vp, C.c_size_t, vp, vp,
                                  P(_DebugOut), vp]
        lib.tc_encode_noalloc.argtypes = [vp, vp, vp, P(_Tensor), P(_EncodeParams), vp, C.c_size_t, vp, vp, vp]
        lib.tc_decode.argtypes = [vp, vp, vp, vp, C.c_size_t, vp, vp, P(_EncodeParams), P(_Tensor), vp]
        lib.tc_roundtrip_host.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, P(_EncodeParams), P(C.c_uint64), vp]
        lib.tc_stats.argtypes = [vp, vp, vp, P(_Tensor), P(_StatsOut), vp]
        lib.tc_fit_state_create.argtypes = [vp, i32, P(vp)]
        lib.tc_fit_state_free.argtypes = [vp]
        lib.tc_fit_state_free.restype = None
        lib.tc_fit_state_update.argtypes = [vp, vp, P(_Tensor), vp]
        lib.tc_fit_state_export.argtypes = [vp, vp, P(C.c_int64), vp, vp, vp]
        lib.tc_fit_state_import.argtypes = [vp, vp, C.c_int64, vp, vp, vp]
        lib.tc_fit_state_finish.argtypes = [vp, vp, P(_Tensor), P(_FitParams), P(vp), vp]
        lib.tc_fold_forward.argtypes = [vp, vp, vp, vp, vp, C.c_int64, vp, vp]
        lib.tc_fold_inverse.argtypes = [vp, vp, vp, i32, i32, vp, vp]
        _lib = lib
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise TcError(code, where)


def _tensor(x: torch.Tensor) -> _Tensor:
    if not x.is_cuda or not x.is_contiguous() or x.dim() != 4:
        raise ValueError("expected a contiguous 4-d CUDA tensor (NCHW)")
    if x.dtype == torch.float32:
        dt = TC_F32
    elif x.dtype == torch.bfloat16:
        dt = TC_BF16
    else:
        raise ValueError("dtype must be float32 or bfloat16")
    n, c, h, w = x.shape
    return _Tensor(x.data_ptr(), n, c, h, w, dt)


def _stream_ptr(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


class _Handle:
    _free = None

    def __init__(self, ptr: int):
        self.ptr = C.c_void_p(ptr)

    def close(self):
        if self.ptr:
            getattr(load_library(), self._free)(self.ptr)
            self.ptr = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Context(_Handle):
    _free = "tc_destroy"

    def __init__(self, ptr: int, device: int):
        super().__init__(ptr)
        self.device = device


class Model(_Handle):
    _free = "tc_model_free"


class Codebook(_Handle):
    _free = "tc_codebook_free"


class FitState(_Handle):
    _free = "tc_fit_state_free"


@dataclass
class StreamLayout:
    n_tiles: int
    n_chunks: int
    stream_bytes: int
    chunk_len_bytes: int
    tile_off_bytes: int
    chunk_pixels: int
    pixel_splits: int


@dataclass
class EncodedStream:
    """Device buffers written by tc_encode."""
    words: torch.Tensor        # uint8 buffer holding the little-endian 32-bit stream words
    chunk_len: torch.Tensor    # int16 (bit pattern of uint16) [n_chunks, rounded up to even]
    tile_off: torch.Tensor     # int64 (bit pattern of uint64) [n_tiles + 1]
    layout: StreamLayout
    coefficients: torch.Tensor | None = None
    symbols: torch.Tensor | None = None

    def total_bits(self) -> int:
        return int(self.tile_off[-1].item())


@dataclass
class Stats:
    entropy: float
    mean_length: float
    mse: float
    clamped_fraction: float
    zero_fraction: float
    energy_ratio_90: float
    hist: torch.Tensor | None


def tc_create(device: int = 0) -> Context:
    out = C.c_void_p()
    _check(load_library().tc_create(C.byref(out), device), "tc_create")
    return Context(out.value, device)


def tc_force_exact_path(ctx: Context, on) -> None:
    """0 / False: default routes; 1 / True: fp64 kernels for everything; 2: bf16 tensors skip the
    resident-basis tensor-core kernels (validation of the streaming kernels)."""
    load_library().tc_force_exact_path(ctx.ptr, int(on))


def tc_last_path(ctx: Context, decode: bool = False) -> int:
    return load_library().tc_last_path(ctx.ptr, int(decode))


def tc_get_status(ctx: Context) -> int:
    return load_library().tc_get_status(ctx.ptr, _stream_ptr(ctx.device))


def tc_fit_pca(ctx: Context, calib: torch.Tensor, bits: int, k: int = 0, basis_dtype: int | None = None,
               zero_level: bool = True, eigensolver: int = TC_EIG_DEVICE) -> Model:
    """`zero_level` (on by default here; tc_fit_params.zero_level in the C ABI) shifts the quantiser
    grid so that y = 0 is one of its levels."""
    t = _tensor(calib)
    params = _FitParams(bits, k, t.dtype if basis_dtype is None else basis_dtype, int(zero_level), eigensolver)
    out = C.c_void_p()
    _check(load_library().tc_fit_pca(ctx.ptr, C.byref(t), C.byref(params), C.byref(out),
                                     _stream_ptr(ctx.device)), "tc_fit_pca")
    return Model(out.value)


def tc_fit_state_create(ctx: Context, c: int) -> FitState:
    out = C.c_void_p()
    _check(load_library().tc_fit_state_create(ctx.ptr, c, C.byref(out)), "tc_fit_state_create")
    st = FitState(out.value)
    st.c = c
    return st


def tc_fit_state_update(ctx: Context, state: FitState, maps: torch.Tensor) -> None:
    t = _tensor(maps)
    _check(load_library().tc_fit_state_update(ctx.ptr, state.ptr, C.byref(t), _stream_ptr(ctx.device)), "tc_fit_state_update")


def tc_fit_state_export(ctx: Context, state: FitState):
    """(count, sum[C], outer[C][C]) as host arrays."""
    c = state.c
    count = C.c_int64()
    s1 = np.zeros(c)
    s2 = np.zeros((c, c))
    _check(load_library().tc_fit_state_export(ctx.ptr, state.ptr, C.byref(count), s1.ctypes.data, s2.ctypes.data,
                                              _stream_ptr(ctx.device)), "tc_fit_state_export")
    return count.value, s1, s2


def tc_fit_state_import(ctx: Context, state: FitState, count: int, s1: np.ndarray, s2: np.ndarray) -> None:
    s1 = np.ascontiguousarray(s1, dtype=np.float64)
    s2 = np.ascontiguousarray(s2, dtype=np.float64)
    if s1.shape != (state.c,) or s2.shape != (state.c, state.c):
        raise ValueError("state arrays do not match the channel count")
    _check(load_library().tc_fit_state_import(ctx.ptr, state.ptr, int(count), s1.ctypes.data, s2.ctypes.data,
                                              _stream_ptr(ctx.device)), "tc_fit_state_import")


def tc_fit_state_finish(ctx: Context, state: FitState, range_maps: torch.Tensor, bits: int, k: int = 0,
                        basis_dtype: int | None = None, zero_level: bool = True, eigensolver: int = TC_EIG_DEVICE) -> Model:
    t = _tensor(range_maps)
    params = _FitParams(bits, k, t.dtype if basis_dtype is None else basis_dtype, int(zero_level), eigensolver)
    out = C.c_void_p()
    _check(load_library().tc_fit_state_finish(ctx.ptr, state.ptr, C.byref(t), C.byref(params), C.byref(out),
                                              _stream_ptr(ctx.device)), "tc_fit_state_finish")
    return Model(out.value)


def tc_fold_forward(model: Model, k: int, w: np.ndarray, bias=None, scale=None, shift=None):
    """Folded weights [K][fan] and bias [K] of the producing convolution (`w` is [C][fan])."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    c, fan = w.shape
    opt = [None if v is None else np.ascontiguousarray(v, dtype=np.float64) for v in (bias, scale, shift)]
    wf = np.zeros((k, fan))
    bf = np.zeros(k)
    _check(load_library().tc_fold_forward(model.ptr, w.ctypes.data, *[None if v is None else v.ctypes.data for v in opt],
                                          fan, wf.ctypes.data, bf.ctypes.data), "tc_fold_forward")
    return wf, bf


def tc_fold_inverse(model: Model, k: int, w_next: np.ndarray, bias_next=None):
    """Folded weights [Cout][K][taps] and bias [Cout] of the consuming convolution (`w_next` is [Cout][C][taps])."""
    w_next = np.ascontiguousarray(w_next, dtype=np.float64)
    cout, c, taps = w_next.shape
    b = None if bias_next is None else np.ascontiguousarray(bias_next, dtype=np.float64)
    wi = np.zeros((cout, k, taps))
    bi = np.zeros(cout)
    _check(load_library().tc_fold_inverse(model.ptr, w_next.ctypes.data, None if b is None else b.ctypes.data, cout, taps,
                                          wi.ctypes.data, bi.ctypes.data), "tc_fold_inverse")
    return wi, bi


def tc_model_import(ctx: Context, *, basis: np.ndarray, mean: np.ndarray, lo: float, step: float, bits: int,
                    basis_dtype: int, k: int | None = None, eig: np.ndarray | None = None,
                    basis_scale: float = 1.0) -> Model:
    basis = np.ascontiguousarray(basis, dtype=np.float64)
    mean = np.ascontiguousarray(mean, dtype=np.float64)
    c = basis.shape[0]
    eig_arr = None if eig is None else np.ascontiguousarray(eig, dtype=np.float64)
    d = _ModelDesc(c, c if k is None else k, bits, basis_dtype, lo, step, basis.ctypes.data, mean.ctypes.data,
                   None if eig_arr is None else eig_arr.ctypes.data, basis_scale)
    out = C.c_void_p()
    _check(load_library().tc_model_import(ctx.ptr, C.byref(d), C.byref(out)), "tc_model_import")
    return Model(out.value)


def tc_model_export(model: Model) -> dict:
    d = _ModelDesc()
    _check(load_library().tc_model_export(model.ptr, C.byref(d)), "tc_model_export")
    basis = np.zeros((d.c, d.c))
    mean = np.zeros(d.c)
    eig = np.zeros(d.c)
    d.basis, d.mean, d.eig = basis.ctypes.data, mean.ctypes.data, eig.ctypes.data
    _check(load_library().tc_model_export(model.ptr, C.byref(d)), "tc_model_export")
    return dict(c=d.c, k=d.k, bits=d.bits, basis_dtype=d.basis_dtype, lo=d.lo, step=d.step, basis=basis,
                mean=mean, eig=eig, basis_scale=d.basis_scale)


def tc_build_codebook(ctx: Context, model: Model, hist, *, groups: int = 1, max_length: int = 0) -> Codebook:
    params = _CodebookParams(groups, max_length)
    out = C.c_void_p()
    if isinstance(hist, torch.Tensor) and hist.is_cuda:
        if hist.dtype != torch.int64 or not hist.is_contiguous():
            raise ValueError("device histogram must be contiguous int64 (uint64 bit pattern)")
        ptr, on_dev = hist.data_ptr(), 1
        keep = hist
    else:
        keep = np.ascontiguousarray(hist.cpu().numpy() if isinstance(hist, torch.Tensor) else hist, dtype=np.uint64)
        ptr, on_dev = keep.ctypes.data, 0
    _check(load_library().tc_build_codebook(ctx.ptr, model.ptr, ptr, on_dev, C.byref(params), C.byref(out)),
           "tc_build_codebook")
    del keep
    return Codebook(out.value)


def tc_codebook_import(ctx: Context, lengths: np.ndarray, bits: int) -> Codebook:
    lengths = np.ascontiguousarray(lengths, dtype=np.uint8)
    if lengths.ndim == 1:
        lengths = lengths[None, :]
    out = C.c_void_p()
    _check(load_library().tc_codebook_import(ctx.ptr, bits, lengths.shape[0], lengths.ctypes.data, C.byref(out)),
           "tc_codebook_import")
    return Codebook(out.value)


def tc_codebook_export(cb: Codebook) -> np.ndarray:
    bits, groups = C.c_int32(), C.c_int32()
    _check(load_library().tc_codebook_export(cb.ptr, C.byref(bits), C.byref(groups), None), "tc_codebook_export")
    out = np.zeros((groups.value, 1 << bits.value), dtype=np.uint8)
    _check(load_library().tc_codebook_export(cb.ptr, C.byref(bits), C.byref(groups), out.ctypes.data),
           "tc_codebook_export")
    return out


def tc_host_huffman_lengths(counts: np.ndarray, max_length: int = 12) -> np.ndarray:
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    out = np.zeros(counts.shape[0], dtype=np.uint8)
    _check(load_library().tc_host_huffman_lengths(counts.ctypes.data, counts.shape[0], max_length, out.ctypes.data),
           "tc_host_huffman_lengths")
    return out


def tc_device_eigh(ctx: Context, a: torch.Tensor):
    """Eigenvalues (descending), eigenvectors (rows) and the number of Jacobi sweeps for a symmetric
    float64 CUDA matrix."""
    if a.dtype != torch.float64 or not a.is_cuda or a.dim() != 2 or a.shape[0] != a.shape[1]:
        raise ValueError("tc_device_eigh wants a square float64 CUDA tensor")
    a = a.contiguous()
    n = a.shape[0]
    evals = torch.empty(n, dtype=torch.float64, device=a.device)
    evecs = torch.empty((n, n), dtype=torch.float64, device=a.device)
    sweeps = C.c_int32(0)
    _check(load_library().tc_device_eigh(ctx.ptr, a.data_ptr(), n, evals.data_ptr(), evecs.data_ptr(), C.byref(sweeps),
                                         _stream_ptr(ctx.device)), "tc_device_eigh")
    return evals, evecs, sweeps.value


def tc_host_eigh(a: np.ndarray):
    a = np.array(a, dtype=np.float64, order="C")
    n = a.shape[0]
    evals = np.zeros(n)
    evecs = np.zeros((n, n))
    _check(load_library().tc_host_eigh(a.ctypes.data, n, evals.ctypes.data, evecs.ctypes.data), "tc_host_eigh")
    return evals, evecs


def tc_encode_bound(model: Model, cb: Codebook, x: torch.Tensor, chunk_pixels: int = 0,
                    pixel_splits: int = 0) -> StreamLayout:
    t = _tensor(x)
    p = _EncodeParams(chunk_pixels, pixel_splits)
    lay = _StreamLayout()
    _check(load_library().tc_encode_bound(model.ptr, cb.ptr, C.byref(t), C.byref(p), C.byref(lay)), "tc_encode_bound")
    return StreamLayout(lay.n_tiles, lay.n_chunks, lay.stream_bytes, lay.chunk_len_bytes, lay.tile_off_bytes,
                        lay.chunk_pixels, lay.pixel_splits)


def tc_encode(ctx: Context, model: Model, cb: Codebook, x: torch.Tensor, *, chunk_pixels: int = 0,
              pixel_splits: int = 0, out: EncodedStream | None = None, capacity: int | None = None, debug: bool = False,
              k: int | None = None) -> EncodedStream:
    """Encode `x`.  Buffers are allocated with torch (worst-case size) unless `out` is given."""
    t = _tensor(x)
    lay = tc_encode_bound(model, cb, x, chunk_pixels, pixel_splits)
    dev = x.device
    if out is None:
        nbytes = lay.stream_bytes if capacity is None else capacity
        out = EncodedStream(torch.empty(max(nbytes, 16), dtype=torch.uint8, device=dev),
                            torch.empty(max(lay.n_chunks + (lay.n_chunks & 1), 2), dtype=torch.int16, device=dev),
                            torch.empty(lay.n_tiles + 1, dtype=torch.int64, device=dev), lay)
    dbg = None
    if debug:
        pixels = t.n * t.h * t.w
        kk = t.c if k is None else k
        out.coefficients = torch.empty(pixels, kk, dtype=torch.float32, device=dev)
        out.symbols = torch.empty(pixels, kk, dtype=torch.uint8, device=dev)
        dbg = _DebugOut(out.coefficients.data_ptr(), out.symbols.data_ptr())
    p = _EncodeParams(lay.chunk_pixels, lay.pixel_splits)
    cap = out.words.numel() if capacity is None else min(capacity, out.words.numel())
    _check(load_library().tc_encode(ctx.ptr, model.ptr, cb.ptr, C.byref(t), C.byref(p), out.words.data_ptr(), cap,
                                    out.chunk_len.data_ptr(), out.tile_off.data_ptr(),
                                    C.byref(dbg) if dbg is not None else None, _stream_ptr(ctx.device)), "tc_encode")
    return out


def tc_encode_noalloc(ctx: Context, model: Model, cb: Codebook, x: torch.Tensor, out: EncodedStream, *,
                      chunk_pixels: int = 0, pixel_splits: int = 0) -> EncodedStream:
    """Encode `x` into buffers the caller already owns, through the entry point that never
    allocates device memory (see tc_encode_noalloc in include/tc.h).  `out` must come from an
    earlier tc_encode of the same shape or be sized with tc_encode_bound."""
    t = _tensor(x)
    p = _EncodeParams(chunk_pixels, pixel_splits)
    _check(load_library().tc_encode_noalloc(ctx.ptr, model.ptr, cb.ptr, C.byref(t), C.byref(p), out.words.data_ptr(),
                                            out.words.numel(), out.chunk_len.data_ptr(), out.tile_off.data_ptr(),
                                            _stream_ptr(ctx.device)), "tc_encode_noalloc")
    return out


def tc_decode(ctx: Context, model: Model, cb: Codebook, enc: EncodedStream, shape, dtype, *,
              out: torch.Tensor | None = None, stream_bytes: int | None = None, relu: bool = False,
              mean_tile_bytes: int | None = None) -> torch.Tensor:
    """Decode `enc`; `relu` applies the layer's non-linearity after the inverse transform;
    `mean_tile_bytes` is the rate hint of tc_encode_params (derived from `stream_bytes` when only
    that is given)."""
    if out is None:
        out = torch.empty(shape, dtype=dtype, device=enc.words.device)
    t = _tensor(out)
    # a caller that knows the stream's length also knows the mean tile size: pass it on as the rate hint
    if mean_tile_bytes is not None:
        hint = mean_tile_bytes
    else:
        hint = 0 if stream_bytes is None else min(2**31 - 1, stream_bytes // max(1, enc.layout.n_tiles))
    p = _EncodeParams(enc.layout.chunk_pixels, enc.layout.pixel_splits, int(relu), int(hint))
    nbytes = enc.words.numel() if stream_bytes is None else stream_bytes
    _check(load_library().tc_decode(ctx.ptr, model.ptr, cb.ptr, enc.words.data_ptr(), nbytes,
                                    enc.chunk_len.data_ptr(), enc.tile_off.data_ptr(), C.byref(p), C.byref(t),
                                    _stream_ptr(ctx.device)), "tc_decode")
    return out


class _EncodeItem(C.Structure):
    _fields_ = [("model", C.c_void_p), ("codebook", C.c_void_p), ("x", C.c_void_p), ("params", C.c_void_p),
                ("stream_out", C.c_void_p), ("capacity", C.c_size_t), ("chunk_len", C.c_void_p), ("tile_off", C.c_void_p)]


class _DecodeItem(C.Structure):
    _fields_ = [("model", C.c_void_p), ("codebook", C.c_void_p), ("stream", C.c_void_p), ("stream_bytes", C.c_size_t),
                ("chunk_len", C.c_void_p), ("tile_off", C.c_void_p), ("params", C.c_void_p), ("x_hat", C.c_void_p)]


def tc_encode_many(ctx: Context, layers, *, outs=None):
    """Encode several tensors in one call: `layers` is a list of (model, codebook, x).  Returns the
    list of EncodedStream; `outs` reuses the buffers of an earlier call."""
    n = len(layers)
    tensors, params, items = [], [], (_EncodeItem * max(n, 1))()
    result = []
    for i, (model, cb, x) in enumerate(layers):
        t = _tensor(x)
        lay = tc_encode_bound(model, cb, x, 0, 0)
        if outs is not None:
            out = outs[i]
        else:
            out = EncodedStream(torch.empty(max(lay.stream_bytes, 16), dtype=torch.uint8, device=x.device),
                                torch.empty(max(lay.n_chunks + (lay.n_chunks & 1), 2), dtype=torch.int16, device=x.device),
                                torch.empty(lay.n_tiles + 1, dtype=torch.int64, device=x.device), lay)
        p = _EncodeParams(lay.chunk_pixels, lay.pixel_splits)
        tensors.append(t); params.append(p); result.append(out)
        items[i] = _EncodeItem(model.ptr, cb.ptr, C.addressof(t), C.addressof(p), out.words.data_ptr(), out.words.numel(),
                               out.chunk_len.data_ptr(), out.tile_off.data_ptr())
    _check(load_library().tc_encode_many(ctx.ptr, items, n, _stream_ptr(ctx.device)), "tc_encode_many")
    return result


def tc_decode_many(ctx: Context, layers, *, outs=None, relu: bool = False):
    """Decode several tensors in one call: `layers` is a list of (model, codebook, enc, shape, dtype)."""
    n = len(layers)
    tensors, params, items = [], [], (_DecodeItem * max(n, 1))()
    result = []
    for i, (model, cb, enc, shape, dtype) in enumerate(layers):
        out = outs[i] if outs is not None else torch.empty(shape, dtype=dtype, device=enc.words.device)
        t = _tensor(out)
        p = _EncodeParams(enc.layout.chunk_pixels, enc.layout.pixel_splits, int(relu), 0)
        tensors.append(t); params.append(p); result.append(out)
        items[i] = _DecodeItem(model.ptr, cb.ptr, enc.words.data_ptr(), enc.words.numel(), enc.chunk_len.data_ptr(),
                               enc.tile_off.data_ptr(), C.addressof(p), C.addressof(t))
    _check(load_library().tc_decode_many(ctx.ptr, items, n, _stream_ptr(ctx.device)), "tc_decode_many")
    return result


def tc_roundtrip_host(ctx: Context, model: Model, cb: Codebook, x_host: torch.Tensor, out_host: torch.Tensor, *,
                      chunk_pixels: int = 0, pixel_splits: int = 0) -> int:
    """Encode + decode a HOST tensor (dense NCHW, ideally pinned) into `out_host`; returns the
    coded length in bits.  The copies and both kernels run inside the C call."""
    if x_host.is_cuda or out_host.is_cuda or not x_host.is_contiguous() or not out_host.is_contiguous():
        raise ValueError("expected contiguous host tensors")
    if x_host.shape != out_host.shape or x_host.dtype != out_host.dtype:
        raise ValueError("input and output must have the same shape and dtype")
    n, c, h, w = x_host.shape
    dt = TC_F32 if x_host.dtype == torch.float32 else TC_BF16
    p = _EncodeParams(chunk_pixels, pixel_splits)
    bits = C.c_uint64(0)
    _check(load_library().tc_roundtrip_host(ctx.ptr, model.ptr, cb.ptr, x_host.data_ptr(), out_host.data_ptr(), n, c, h, w,
                                            dt, C.byref(p), C.byref(bits), _stream_ptr(ctx.device)), "tc_roundtrip_host")
    return bits.value


def tc_stats(ctx: Context, model: Model, cb: Codebook | None, x: torch.Tensor, *, groups: int = 1,
             want_hist: bool = True) -> Stats:
    t = _tensor(x)
    exp = tc_model_export(model)
    hist = None
    if want_hist:
        hist = torch.zeros(groups, 1 << exp["bits"], dtype=torch.int64, device=x.device)
    s = _StatsOut(groups, hist.data_ptr() if hist is not None else None, 0, 0, 0, 0, 0, 0)
    _check(load_library().tc_stats(ctx.ptr, model.ptr, cb.ptr if cb is not None else None, C.byref(t), C.byref(s),
                                   _stream_ptr(ctx.device)), "tc_stats")
    return Stats(s.entropy, s.mean_length, s.mse, s.clamped_fraction, s.zero_fraction, s.energy_ratio_90, hist)
