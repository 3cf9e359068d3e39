"""ctypes front end of the CPU oracle (oracle/tc_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg use
it; the CUDA package never imports it.  The wrappers only marshal numpy arrays; every step of
the method is in the C file, which cites the paper passage each function follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tc_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libtc_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, no fast-math) and return the library path."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        d, i64, i32, vp = C.c_double, C.c_int64, C.c_int, C.c_void_p
        sig = {
            "orc_round_bf16": (d, [d]),
            "orc_mean_cov": (None, [vp, i64, i32, i64, vp, vp]),
            "orc_eigh_jacobi": (i32, [vp, i32, vp, vp]),
            "orc_fit_pca": (i32, [vp, i64, i32, i64, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
            "orc_project": (None, [vp, i64, i32, i64, vp, vp, i32, vp]),
            "orc_quantize": (None, [vp, i64, d, d, i32, vp, vp]),
            "orc_histogram": (None, [vp, i64, i32, i32, i32, vp]),
            "orc_huffman_lengths": (i32, [vp, i32, i32, vp]),
            "orc_huffman_lengths_raw": (i32, [vp, i32, i32, i32, vp]),
            "orc_canonical_codes": (None, [vp, i32, vp]),
            "orc_encode": (i64, [vp, i64, i32, i32, i32, vp, i64, i64, vp, i64, vp, vp]),
            "orc_decode_symbols": (i32, [vp, i64, vp, vp, i64, i32, i32, i32, vp, i64, i64, vp]),
            "orc_reconstruct": (None, [vp, i64, i32, i64, i32, vp, vp, d, d, i32, i32, vp]),
            "orc_moments_update": (None, [vp, i64, i32, i64, vp, vp, vp]),
            "orc_moments_mean_cov": (None, [i64, vp, vp, i32, vp, vp]),
            "orc_fit_pca_moments": (i32, [i64, vp, vp, vp, i64, i32, i64, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
            "orc_fold_forward": (None, [vp, vp, i32, i32, vp, vp, vp, vp, i64, vp, vp]),
            "orc_fold_inverse": (None, [vp, vp, i32, i32, vp, vp, i32, i32, vp, vp]),
            "orc_entropy": (d, [vp, i32]),
            "orc_mean_length": (d, [vp, vp, i32]),
            "orc_mse": (d, [vp, vp, i64]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(_lib, name)
            fn.restype, fn.argtypes = res, args
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _f32(x) -> np.ndarray:
    """NCHW tensor (numpy or torch, fp32 or bf16) -> contiguous float32 numpy array (exact)."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 4
    return x


@dataclass
class Model:
    """Per-layer transform and quantiser: y = basis (x - mean); levels lo + q*step."""
    c: int
    k: int
    bits: int
    mean: np.ndarray      # [C] float64
    basis: np.ndarray     # [C][C] float64, row j = j-th principal direction (first k rows used)
    eig: np.ndarray       # [C] float64, descending
    lo: float
    step: float
    basis_round: str = "f64"   # "f64", "bf16", "f32" or "int8": how the basis was rounded at fit time
    basis_scale: float = 1.0   # "int8": every basis entry is an integer in [-127, 127] times this
    cal_lo: float | None = None   # range of coefficient 0 on the calibration maps, as measured
    cal_hi: float | None = None
    zero_level: bool = False   # the grid was shifted so that y = 0 is a level (zero_level_lo)


@dataclass
class Stream:
    words: np.ndarray          # uint32, padded stream
    chunk_len: np.ndarray      # uint16 [n_chunks], bits of every chunk
    tile_off: np.ndarray       # uint64 [n_tiles + 1], absolute bits, multiples of 128
    total_bits: int
    pixels: int
    k: int
    chunk_pixels: int          # pixels per chunk (1 when pixel_splits > 1)
    pixel_splits: int          # chunks per pixel
    tile_pixels: int

    @property
    def chunk_symbols(self) -> int:
        return self.chunk_pixels * self.k // self.pixel_splits

    def chunk_starts(self) -> np.ndarray:
        """Absolute start bit of every chunk (tile start plus the lengths before it)."""
        cpt = self.tile_pixels * self.k // self.chunk_symbols
        out = np.zeros(self.chunk_len.shape[0], dtype=np.uint64)
        for t in range(self.tile_off.shape[0] - 1):
            ln = self.chunk_len[t * cpt:(t + 1) * cpt].astype(np.uint64)
            out[t * cpt:t * cpt + ln.shape[0]] = self.tile_off[t] + np.concatenate(([0], np.cumsum(ln)[:-1])).astype(np.uint64)
        return out


def round_bf16(v: float) -> float:
    return lib().orc_round_bf16(float(v))


def mean_cov(x):
    x = _f32(x)
    n, c, h, w = x.shape
    mean = np.zeros(c)
    cov = np.zeros((c, c))
    lib().orc_mean_cov(_p(x), n, c, h * w, _p(mean), _p(cov))
    return mean, cov


def eigh_jacobi(a: np.ndarray):
    a = np.array(a, dtype=np.float64, order="C")
    n = a.shape[0]
    ev = np.zeros(n)
    vt = np.zeros((n, n))
    sweeps = lib().orc_eigh_jacobi(_p(a), n, _p(ev), _p(vt))
    return ev, vt, sweeps


JACOBI_MAX_C = 128


def zero_level_lo(lo: float, step: float) -> float:
    """Lowest level of the quantiser grid shifted so that y = 0 is one of its levels.

    Section 3.1 ("Quantization") takes the dynamic range from the highest-variance coefficient and
    leaves the position of the levels open.  The coefficients are zero-mean (the mean is
    subtracted before the projection) and, after the PCA, most of them are tiny: Appendix E
    observes that all values of a low-variance channel map to a single value.  That only happens
    when zero is a reconstruction level; with zero half-way between two levels such a channel
    flips between its two neighbours.  So the grid lo + q*step keeps the step the range gives
    and moves by at most half a step: round(-lo / step) levels (ties to even) lie below zero."""
    return float(-step * np.rint(-lo / step))


def _finish_model(c, k, bits, mean, basis, eig, lo, step, basis_round, scale, zero_level) -> "Model":
    hi = lo + step * ((1 << bits) - 1)
    return Model(c, k, bits, mean, basis, eig, zero_level_lo(lo, step) if zero_level else lo, step,
                 basis_round, scale, lo, hi, zero_level)


def fit_pca(x, bits: int, *, k: int | None = None, basis_bf16: bool = False,
            basis_round: str | None = None, eigensolver: str = "auto", zero_level: bool = False) -> Model:
    """Fit mean, basis and quantiser range on calibration maps.  `zero_level` shifts the quantiser
    grid so that y = 0 is a level (zero_level_lo).

    basis_round: "f64" (keep), "bf16", "f32" or "int8" (8-bit matrix with one scale).  eigensolver: "jacobi" (the in-file solver),
    "lapack" (numpy.linalg.eigh, a library primitive used as one step) or "auto" = Jacobi up
    to JACOBI_MAX_C channels, LAPACK beyond (Jacobi needs minutes there).
    """
    x = _f32(x)
    n, c, h, w = x.shape
    if basis_round is None:
        basis_round = "bf16" if basis_bf16 else "f64"
    mode = {"f64": 0, "bf16": 1, "f32": 2, "int8": 3}[basis_round]
    if eigensolver == "auto":
        eigensolver = "jacobi" if c <= JACOBI_MAX_C else "lapack"
    pre_ev = pre_vt = None
    if eigensolver == "lapack":
        _, cov = mean_cov(x)
        ev, vec = np.linalg.eigh(cov)
        pre_ev = np.ascontiguousarray(ev)
        pre_vt = np.ascontiguousarray(vec.T)
    mean = np.zeros(c)
    basis = np.zeros((c, c))
    eig = np.zeros(c)
    lo = C.c_double()
    step = C.c_double()
    scale = C.c_double()
    rc = lib().orc_fit_pca(_p(x), n, c, h * w, bits, mode,
                           _p(pre_ev) if pre_ev is not None else None,
                           _p(pre_vt) if pre_vt is not None else None,
                           _p(mean), _p(basis), _p(eig), C.byref(lo), C.byref(step), C.byref(scale))
    if rc != 0:
        raise RuntimeError("oracle eigensolver did not converge")
    return _finish_model(c, c if k is None else k, bits, mean, basis, eig, lo.value, step.value,
                         basis_round, scale.value, zero_level)


def with_bits(m: Model, bits: int) -> Model:
    """The same transform with the calibration range divided into 2^bits - 1 steps."""
    lo = m.lo if m.cal_lo is None else m.cal_lo
    hi = m.lo + m.step * ((1 << m.bits) - 1) if m.cal_hi is None else m.cal_hi
    return _finish_model(m.c, m.k, bits, m.mean, m.basis, m.eig, lo, (hi - lo) / ((1 << bits) - 1),
                         m.basis_round, m.basis_scale, m.zero_level)


def project(model: Model, x) -> np.ndarray:
    """[P][K] coefficients, P = N*H*W in pixel order p = n*HW + s."""
    x = _f32(x)
    n, c, h, w = x.shape
    y = np.zeros((n * h * w, model.k))
    lib().orc_project(_p(x), n, c, h * w, _p(model.mean), _p(model.basis), model.k, _p(y))
    return y


def quantize(model: Model, y: np.ndarray, *, with_units: bool = False):
    y = np.ascontiguousarray(y, dtype=np.float64)
    q = np.zeros(y.shape, dtype=np.uint8)
    units = np.zeros(y.shape) if with_units else None
    lib().orc_quantize(_p(y), y.size, model.lo, model.step, model.bits, _p(q),
                       _p(units) if with_units else None)
    return (q, units) if with_units else q


def histogram(q: np.ndarray, bits: int, per_channel: bool) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    pixels, k = q.shape
    groups = k if per_channel else 1
    hist = np.zeros((groups, 1 << bits), dtype=np.uint64)
    lib().orc_histogram(_p(q), pixels, k, groups, bits, _p(hist))
    return hist


def huffman_lengths(hist: np.ndarray, lmax: int = 12) -> np.ndarray:
    """Code lengths [groups][2^bits] from counts [groups][2^bits] (weights = count + 1)."""
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    if hist.ndim == 1:
        hist = hist[None, :]
    out = np.zeros(hist.shape, dtype=np.uint8)
    for g in range(hist.shape[0]):
        row = np.ascontiguousarray(hist[g])
        ln = np.zeros(hist.shape[1], dtype=np.uint8)
        if lib().orc_huffman_lengths(_p(row), hist.shape[1], lmax, _p(ln)) != 0:
            raise ValueError("bad alphabet size / length limit")
        out[g] = ln
    return out


def huffman_lengths_raw(weights, lmax: int = 31, force_limited: bool = False) -> np.ndarray:
    w = np.ascontiguousarray(weights, dtype=np.uint64)
    ln = np.zeros(w.shape[0], dtype=np.uint8)
    if lib().orc_huffman_lengths_raw(_p(w), w.shape[0], lmax, int(force_limited), _p(ln)) != 0:
        raise ValueError("bad alphabet size / length limit")
    return ln


def canonical_codes(lengths: np.ndarray) -> np.ndarray:
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    code = np.zeros(ln.shape[0], dtype=np.uint32)
    lib().orc_canonical_codes(_p(ln), ln.shape[0], _p(code))
    return code


def encode(q: np.ndarray, lengths: np.ndarray, bits: int, *, chunk_pixels: int = 1,
           pixel_splits: int = 1, tile_pixels: int = 128) -> Stream:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    pixels, k = q.shape
    lengths = np.ascontiguousarray(lengths, dtype=np.uint8)
    if lengths.ndim == 1:
        lengths = lengths[None, :]
    groups = lengths.shape[0]
    if pixel_splits > 1 and chunk_pixels != 1:
        raise ValueError("a pixel is split only when a chunk is one pixel")
    if (chunk_pixels * k) % pixel_splits or (tile_pixels * k) % (chunk_pixels * k // pixel_splits):
        raise ValueError("tiles must hold a whole number of chunks")
    chunk_symbols = chunk_pixels * k // pixel_splits
    n_tiles = -(-pixels // tile_pixels) if pixels else 0
    n_chunks = -(-(pixels * k) // chunk_symbols)
    cap_bits = pixels * k * int(lengths.max()) + 128 * (n_tiles + 1)
    cap_words = cap_bits // 32 + 4
    words = np.zeros(cap_words, dtype=np.uint32)
    chunk_len = np.zeros(max(n_chunks, 1), dtype=np.uint16)
    tile_off = np.zeros(n_tiles + 1, dtype=np.uint64)
    total = lib().orc_encode(_p(q), pixels, k, groups, bits, _p(lengths), chunk_symbols,
                             tile_pixels, _p(words), cap_words, _p(chunk_len), _p(tile_off))
    if total == -2:
        raise ValueError("a chunk is longer than 65535 bits")
    if total < 0:
        raise RuntimeError("oracle stream capacity too small")
    return Stream(words[: total // 32].copy(), chunk_len[:n_chunks].copy(), tile_off, int(total),
                  pixels, k, chunk_pixels, pixel_splits, tile_pixels)


def decode_symbols(s: Stream, lengths: np.ndarray, bits: int) -> np.ndarray:
    lengths = np.ascontiguousarray(lengths, dtype=np.uint8)
    if lengths.ndim == 1:
        lengths = lengths[None, :]
    q = np.zeros((s.pixels, s.k), dtype=np.uint8)
    words = np.ascontiguousarray(s.words, dtype=np.uint32)
    chunk_len = np.ascontiguousarray(s.chunk_len, dtype=np.uint16)
    tile_off = np.ascontiguousarray(s.tile_off, dtype=np.uint64)
    rc = lib().orc_decode_symbols(_p(words), words.shape[0], _p(chunk_len), _p(tile_off),
                                  s.pixels, s.k, lengths.shape[0], bits, _p(lengths),
                                  s.chunk_symbols, s.tile_pixels, _p(q))
    if rc != 0:
        raise ValueError("corrupt stream")
    return q


def reconstruct(model: Model, q: np.ndarray, shape, *, out_bf16: bool, relu: bool = False) -> np.ndarray:
    """x_hat (NCHW float32 array holding fp32 or bf16-rounded values) from symbols [P][K];
    `relu` applies the layer's non-linearity after the inverse transform."""
    n, c, h, w = shape
    q = np.ascontiguousarray(q, dtype=np.uint8)
    xhat = np.zeros((n, c, h, w), dtype=np.float32)
    lib().orc_reconstruct(_p(q), n, c, h * w, model.k, _p(model.mean), _p(model.basis),
                          model.lo, model.step, int(out_bf16), int(relu), _p(xhat))
    return xhat


class Moments:
    """Running state of the online estimate: count, sum of pixel vectors, sum of outer products."""

    def __init__(self, c: int):
        self.c = c
        self.count = 0
        self.sum = np.zeros(c)
        self.outer = np.zeros((c, c))

    def update(self, x) -> "Moments":
        x = _f32(x)
        n, c, h, w = x.shape
        cnt = C.c_int64(self.count)
        lib().orc_moments_update(_p(x), n, c, h * w, C.byref(cnt), _p(self.sum), _p(self.outer))
        self.count = cnt.value
        return self

    def merge(self, other: "Moments") -> "Moments":
        self.count += other.count
        self.sum += other.sum
        self.outer += other.outer
        return self

    def mean_cov(self):
        mean = np.zeros(self.c)
        cov = np.zeros((self.c, self.c))
        lib().orc_moments_mean_cov(self.count, _p(self.sum), _p(self.outer), self.c, _p(mean), _p(cov))
        return mean, cov


def fit_pca_moments(state: Moments, x_range, bits: int, *, k: int | None = None, basis_round: str = "f64",
                    eigensolver: str = "auto", zero_level: bool = False) -> Model:
    """fit_pca with mean and covariance from a running state; the range of coefficient 0 is
    measured on `x_range`."""
    x = _f32(x_range)
    n, c, h, w = x.shape
    mode = {"f64": 0, "bf16": 1, "f32": 2, "int8": 3}[basis_round]
    if eigensolver == "auto":
        eigensolver = "jacobi" if c <= JACOBI_MAX_C else "lapack"
    pre_ev = pre_vt = None
    if eigensolver == "lapack":
        _, cov = state.mean_cov()
        ev, vec = np.linalg.eigh(cov)
        pre_ev = np.ascontiguousarray(ev)
        pre_vt = np.ascontiguousarray(vec.T)
    mean = np.zeros(c)
    basis = np.zeros((c, c))
    eig = np.zeros(c)
    lo, step, scale = C.c_double(), C.c_double(), C.c_double()
    rc = lib().orc_fit_pca_moments(state.count, _p(state.sum), _p(state.outer), _p(x), n, c, h * w, bits, mode,
                                   _p(pre_ev) if pre_ev is not None else None,
                                   _p(pre_vt) if pre_vt is not None else None,
                                   _p(mean), _p(basis), _p(eig), C.byref(lo), C.byref(step), C.byref(scale))
    if rc != 0:
        raise RuntimeError("oracle eigensolver did not converge")
    return _finish_model(c, c if k is None else k, bits, mean, basis, eig, lo.value, step.value, basis_round,
                         scale.value, zero_level)


def fold_forward(model: Model, w: np.ndarray, bias: np.ndarray, scale: np.ndarray, shift: np.ndarray):
    """Producer-side folding: conv weights w[C][fan], bias[C], batch-norm affine (scale, shift)
    -> weights [K][fan] and bias [K] of the convolution that outputs the coefficients y."""
    w = np.ascontiguousarray(w, dtype=np.float64).reshape(model.c, -1)
    fan = w.shape[1]
    bias, scale, shift = (np.ascontiguousarray(v, dtype=np.float64) for v in (bias, scale, shift))
    wf = np.zeros((model.k, fan))
    bf = np.zeros(model.k)
    lib().orc_fold_forward(_p(model.basis), _p(model.mean), model.c, model.k, _p(w), _p(bias), _p(scale), _p(shift),
                           fan, _p(wf), _p(bf))
    return wf, bf


def fold_inverse(model: Model, wn: np.ndarray, bias: np.ndarray):
    """Consumer-side folding: next-layer weights wn[Cout][C][taps], bias[Cout] -> weights
    [Cout][K][taps] and bias [Cout] of the convolution that consumes the dequantised y_hat."""
    wn = np.ascontiguousarray(wn, dtype=np.float64)
    cout, c, taps = wn.shape
    bias = np.ascontiguousarray(bias, dtype=np.float64)
    wi = np.zeros((cout, model.k, taps))
    bi = np.zeros(cout)
    lib().orc_fold_inverse(_p(model.basis), _p(model.mean), c, model.k, _p(wn), _p(bias), cout, taps, _p(wi), _p(bi))
    return wi, bi


def entropy(hist_row: np.ndarray) -> float:
    h = np.ascontiguousarray(hist_row, dtype=np.uint64)
    return lib().orc_entropy(_p(h), h.shape[0])


def mean_length(hist_row: np.ndarray, lengths_row: np.ndarray) -> float:
    h = np.ascontiguousarray(hist_row, dtype=np.uint64)
    ln = np.ascontiguousarray(lengths_row, dtype=np.uint8)
    return lib().orc_mean_length(_p(h), _p(ln), h.shape[0])


def mse(x, xhat) -> float:
    a = _f32(x).ravel()
    b = np.ascontiguousarray(xhat, dtype=np.float32).ravel()
    return lib().orc_mse(_p(a), _p(b), a.shape[0])
