"""Pins for the oracle's 8-bit basis (Section 3.1: the PCA matrix is stored in 8 bits).

The quantiser is one symmetric scale for the whole matrix, s = max|T| / 127, entries
s * rint(T / s).  Pinned to: the integer grid itself, the distance to the unquantised basis of
the same data, the loss of orthonormality that this distance allows, and the small price in
distortion that the paper reports for it.
"""
import numpy as np
import torch

import oracle
from synth import featuremaps as fm


def _maps(c=24, n=12, seed=808):
    params = fm.layer_params(fm.LayerSpec(c, 10, 10, 0.85, None, seed))
    return fm.make_maps(params, n, calib=True)


def test_entries_sit_on_the_integer_grid_within_half_a_step_of_the_exact_basis():
    x = _maps()
    exact = oracle.fit_pca(x, 5)
    m = oracle.fit_pca(x, 5, basis_round="int8")
    s = m.basis_scale
    assert np.isclose(s, np.abs(exact.basis).max() / 127.0, rtol=1e-12)
    n = m.basis / s
    assert np.abs(n - np.rint(n)).max() <= 1e-9
    assert np.abs(n).max() == 127.0                                  # the largest entry maps to +-127
    assert np.abs(m.basis - exact.basis).max() <= s / 2 * (1 + 1e-9)
    assert np.abs(m.basis - exact.basis).max() >= s / 8              # it really was quantised
    assert np.array_equal(m.mean, exact.mean) and np.array_equal(m.eig, exact.eig)
    assert oracle.fit_pca(x, 5).basis_scale == 1.0


def test_orthonormality_is_lost_by_no_more_than_the_rounding_allows():
    x = _maps()
    m = oracle.fit_pca(x, 5, basis_round="int8")
    c = m.c
    defect = np.abs(m.basis @ m.basis.T - np.eye(c)).max()
    # rows of T are unit vectors, every entry moved by at most s/2:
    # |<t_i + e_i, t_j + e_j> - delta_ij| <= 2 * |e| + |e|^2 with |e| <= sqrt(C) * s / 2
    e = np.sqrt(c) * m.basis_scale / 2
    assert 0 < defect <= 2 * e + e * e


def test_the_range_is_taken_with_the_quantised_matrix():
    x = _maps()
    m = oracle.fit_pca(x, 6, basis_round="int8")
    y0 = oracle.project(m, x)[:, 0]
    assert np.isclose(m.lo, y0.min(), rtol=0, atol=1e-12)
    assert np.isclose(m.lo + 63 * m.step, y0.max(), rtol=1e-12)


def test_distortion_price_of_the_8_bit_matrix_is_small_and_the_chain_round_trips():
    params = fm.layer_params(fm.LayerSpec(32, 12, 12, 0.85, None, 809))
    cal = fm.make_maps(params, 16, calib=True)
    x = fm.make_maps(params, 8)
    out = {}
    for mode in ("f64", "int8"):
        m = oracle.fit_pca(cal, 6, basis_round=mode)
        q = oracle.quantize(m, oracle.project(m, x))
        ln = oracle.huffman_lengths(oracle.histogram(oracle.quantize(m, oracle.project(m, cal)), 6, False), 12)
        s = oracle.encode(q, ln, 6, chunk_pixels=1, tile_pixels=128)
        assert np.array_equal(oracle.decode_symbols(s, ln, 6), q)
        xhat = oracle.reconstruct(m, q, x.shape, out_bf16=False)
        out[mode] = (oracle.mse(x, xhat), s.total_bits / x.numel())
    # the transposed 8-bit matrix is not the exact inverse: a visible but small extra error
    assert out["int8"][0] < 2.0 * out["f64"][0] + 1e-4
    assert abs(out["int8"][1] - out["f64"][1]) < 0.05 * out["f64"][1]
