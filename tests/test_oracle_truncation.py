"""Pins for the oracle's K < C path (PCA truncation: only the K leading components are coded;
Section 4, ablation, and Fig. 4 right).

With T orthonormal, x - mu = sum_j y_j t_j, and the decoder rebuilds sum_{j<K} yhat_j t_j + mu.
The error therefore splits into two orthogonal parts: the dropped components, whose mean energy
on the calibration set is exactly the sum of the dropped eigenvalues of the sample covariance,
and the quantisation error of the K kept ones, at most (step / 2)^2 each.  A wrong loop bound,
a transposed basis or a dropped term in the truncated path breaks these identities.
"""
import numpy as np
import pytest
import torch

import oracle
from synth import featuremaps as fm


def _gaussian_maps(c=16, n=40, ratio=0.8, seed=4242):
    params = fm.layer_params(fm.LayerSpec(c, 8, 8, ratio, None, seed))
    return fm.make_plain_gaussian(params, n).float()


def _flat(x):
    n, c, h, w = x.shape
    return np.asarray(x, dtype=np.float64).transpose(0, 2, 3, 1).reshape(-1, c)


@pytest.mark.parametrize("k", [16, 12, 8, 4, 1])
def test_error_is_dropped_eigenvalues_plus_bounded_quantisation_noise(k):
    x = _gaussian_maps()
    c = x.shape[1]
    m = oracle.fit_pca(x, 8, k=k)
    assert m.k == k
    y = oracle.project(m, x)
    assert y.shape == (x.shape[0] * 64, k)
    q = oracle.quantize(m, y)
    xhat = oracle.reconstruct(m, q, x.shape, out_bf16=False)
    err = _flat(x) - _flat(xhat)
    pixels = err.shape[0]
    total = float((err * err).sum() / pixels)                 # mean squared error per pixel, all channels
    dropped = float(m.eig[k:].sum()) * (pixels - 1) / pixels   # covariance is normalised by M - 1
    assert total >= dropped - 1e-6 * (1 + dropped)
    assert total <= dropped + k * (m.step / 2) ** 2 + 1e-6 * (1 + dropped)
    if k >= 4:
        # uniform quantisation noise: step^2 / 12 per kept coefficient (a few clamped tail values aside)
        noise = total - dropped
        assert 0.6 * k * m.step ** 2 / 12 <= noise <= 1.4 * k * m.step ** 2 / 12


def test_reconstruction_stays_in_the_span_of_the_kept_rows():
    x = _gaussian_maps()
    m = oracle.fit_pca(x, 6, k=5)
    q = oracle.quantize(m, oracle.project(m, x))
    xhat = _flat(oracle.reconstruct(m, q, x.shape, out_bf16=False)) - m.mean[None, :]
    dropped_rows = m.basis[5:]                                   # [C - K][C]
    assert np.abs(xhat @ dropped_rows.T).max() <= 1e-5 * np.abs(xhat).max()
    # and the kept coordinates are the quantiser's levels
    levels = xhat @ m.basis[:5].T
    assert np.allclose(levels, m.lo + q.astype(np.float64) * m.step, atol=1e-5)


def test_truncated_projection_is_the_leading_columns_of_the_full_one():
    x = _gaussian_maps(c=12, n=6)
    full = oracle.fit_pca(x, 5)
    for k in (1, 7, 12):
        part = oracle.fit_pca(x, 5, k=k)
        assert np.array_equal(part.basis, full.basis) and part.lo == full.lo and part.step == full.step
        assert np.array_equal(oracle.project(part, x), oracle.project(full, x)[:, :k])
    assert oracle.fit_pca(x, 5, k=12).k == full.k == 12


def test_distortion_falls_and_rate_rises_with_k():
    x = _gaussian_maps(c=16, n=24, ratio=0.7)
    prev_mse, prev_bits = None, None
    for k in (2, 4, 8, 16):
        m = oracle.fit_pca(x, 5, k=k)
        q = oracle.quantize(m, oracle.project(m, x))
        ln = oracle.huffman_lengths(oracle.histogram(q, 5, False), 12)
        s = oracle.encode(q, ln, 5, chunk_pixels=1, tile_pixels=128)
        assert np.array_equal(oracle.decode_symbols(s, ln, 5), q)
        mse = oracle.mse(x, oracle.reconstruct(m, q, x.shape, out_bf16=False))
        bits = s.total_bits / x.numel()          # per value of the tensor, not per coded coefficient
        if prev_mse is not None:
            assert mse < prev_mse and bits > prev_bits
        prev_mse, prev_bits = mse, bits
