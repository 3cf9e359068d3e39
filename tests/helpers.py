"""Shared set-up for the parity tests: build the oracle's model and codebook on the CPU and
import them into the CUDA library, so that both sides use identical T, mu, lo, step and code
lengths on identical input bytes."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from synth import featuremaps as fm


def basis_round_for(dtype) -> str:
    return "bf16" if dtype == torch.bfloat16 else "f32"


def oracle_side(spec: fm.LayerSpec, bits: int, n_cal: int, n_test: int, dtype, per_channel: bool,
                lmax: int = 12, model: oracle.Model | None = None, k: int | None = None,
                basis_round: str | None = None, zero_level: bool = True):
    """Returns dict(model, lengths, cal, x, y, q, units) computed by the oracle on CPU maps."""
    params = fm.layer_params(spec)
    cal = fm.make_maps(params, n_cal, calib=True, dtype=dtype)
    x = fm.make_maps(params, n_test, dtype=dtype)
    if model is None:
        model = oracle.fit_pca(cal, bits, basis_round=basis_round or basis_round_for(dtype), k=k, zero_level=zero_level)
    elif model.bits != bits:
        model = oracle.with_bits(model, bits)
    q_cal = oracle.quantize(model, oracle.project(model, cal))
    lengths = oracle.huffman_lengths(oracle.histogram(q_cal, bits, per_channel), lmax)
    y = oracle.project(model, x)
    q, units = oracle.quantize(model, y, with_units=True)
    return dict(model=model, lengths=lengths, cal=cal, x=x, y=y, q=q, units=units, q_cal=q_cal)


def import_model(tc, ctx, m: oracle.Model, dtype):
    if m.basis_round == "int8":
        basis_dtype = tc.binding.TC_INT8
    else:
        basis_dtype = tc.binding.TC_BF16 if dtype == torch.bfloat16 else tc.binding.TC_F32
    return tc.tc_model_import(ctx, basis=m.basis, mean=m.mean, lo=m.lo, step=m.step, bits=m.bits,
                              basis_dtype=basis_dtype, k=m.k, eig=m.eig, basis_scale=m.basis_scale)


def stream_words(enc) -> np.ndarray:
    total = enc.total_bits()
    return enc.words[: total // 8].cpu().numpy().view(np.uint32)


def chunk_len(enc) -> np.ndarray:
    return enc.chunk_len[: enc.layout.n_chunks].cpu().numpy().view(np.uint16)


def tile_off(enc) -> np.ndarray:
    return enc.tile_off.cpu().numpy().view(np.uint64)


def expected_output_flips(m: oracle.Model, q: np.ndarray, *, out_bf16: bool = True) -> float:
    """Expected number of reconstructed values that an fp32 tensor-core decoder rounds to the
    neighbouring output value, for symbols `q` ([P][K]).

    The decoder computes v = fl32(step * acc + bias_c) with acc = sum_j T[j][c] (q_j - center)
    accumulated in fp32, one rounding per tensor-core step of 16 coefficients (products of a bf16
    and a small integer are exact), then rounds v once to the output type; the oracle rounds the
    exact value once.  The two differ only where an output rounding boundary lies between the
    exact value and v.  A rounding to fp32 errs by at most h = 2^-24 |x|, uniformly; n such errors
    add like a random walk to a mean magnitude of 0.46 sqrt(sum h_i^2), so with s_i the partial
    sums after each step
        E|delta| = 0.46 * 2^-24 * sqrt(sum_i (step s_i)^2 + v^2).
    Output rounding boundaries are one output ulp u apart, so a value flips with probability
    E|delta| / u.  Outputs near zero (a bias cancelled by the sum) have a small ulp and carry most
    of the expectation; it grows with the bit width because more coefficients are non-zero and
    the cancelled terms grow."""
    k = m.k
    t = np.asarray(m.basis[:k], dtype=np.float64)
    top = (1 << m.bits) - 1
    center = min(top, max(0.0, float(np.rint(-m.lo / m.step))))
    d = q.astype(np.float64) - center
    bias = m.mean + (m.lo + center * m.step) * t.sum(axis=0)
    run = np.zeros((q.shape[0], t.shape[1]))
    sum_sq = np.zeros_like(run)
    for j0 in range(0, k, 16):
        run = run + m.step * (d[:, j0:j0 + 16] @ t[j0:j0 + 16])
        sum_sq += run * run
    v = run + bias
    mant = 7 if out_bf16 else 23
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(v), 2.0 ** -126))) - mant)
    delta = 0.46 * 2.0 ** -24 * np.sqrt(sum_sq + v * v)
    return float(np.minimum(1.0, delta / ulp).sum())


def flip_allowance(expected: float) -> int:
    """Upper bound on the observed count given the model's expectation: twice the expectation
    (an accumulator that truncates instead of rounding doubles every error) plus 4.5 standard
    deviations of a Poisson count of that mean, plus one."""
    lam = 2.0 * expected
    return int(np.ceil(lam + 4.5 * np.sqrt(lam) + 1.0))


def count_output_flips(got: np.ndarray, want: np.ndarray, channel_axis: int = 1) -> int:
    """Reconstructed values that differ from the oracle's, counted once per (channel, oracle value):
    pixels whose symbols agree (at a low bit width: all at the zero level) share one exact value per
    channel, and if that value sits on an output rounding boundary they all land on the neighbouring
    number together -- one event of the model above, however many pixels show it."""
    diff = got != want
    if not diff.any():
        return 0
    idx = np.nonzero(diff)
    pairs = np.stack([idx[channel_axis].astype(np.float64), want[diff].astype(np.float64)], axis=1)
    return int(np.unique(pairs, axis=0).shape[0])
