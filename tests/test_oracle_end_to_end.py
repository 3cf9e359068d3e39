"""End-to-end checks of the oracle chain on synthetic layers: the qualitative statements the
paper makes about the method (Sections 3.1, 4; Appendices D, E, G) must hold on data with the
structure the paper describes."""
import math

import numpy as np
import pytest
import torch

import oracle
from synth import featuremaps as fm


def _chain(spec, bits, n_cal=8, n_test=2, per_channel=False, identity=False, dtype=torch.float32):
    p = fm.layer_params(spec)
    cal = fm.make_maps(p, n_cal, calib=True, dtype=dtype)
    x = fm.make_maps(p, n_test, dtype=dtype)
    m = oracle.fit_pca(cal, bits, basis_bf16=(dtype == torch.bfloat16))
    if identity:                        # "Q + VLC" ablation of Section 4: no transform
        y_cal = cal.float().numpy().transpose(0, 2, 3, 1).reshape(-1, spec.c).astype(np.float64)
        lo, hi = y_cal.min(), y_cal.max()
        m = oracle.Model(spec.c, spec.c, bits, np.zeros(spec.c), np.eye(spec.c), m.eig, lo,
                         (hi - lo) / ((1 << bits) - 1), "f64")
    q_cal = oracle.quantize(m, oracle.project(m, cal))
    hist = oracle.histogram(q_cal, bits, per_channel)
    ln = oracle.huffman_lengths(hist, 12)
    q = oracle.quantize(m, oracle.project(m, x))
    s = oracle.encode(q, ln, bits, chunk_pixels=1, tile_pixels=128)
    assert np.array_equal(oracle.decode_symbols(s, ln, bits), q)
    xhat = oracle.reconstruct(m, q, x.shape, out_bf16=(dtype == torch.bfloat16))
    return dict(model=m, q=q, q_cal=q_cal, hist=hist, lengths=ln, stream=s, x=x, xhat=xhat,
                bits_per_value=s.total_bits / q.size, mse=oracle.mse(x, xhat))


def test_full_chain_round_trip_and_distortion_falls_with_bits():
    spec = fm.LayerSpec(32, 14, 14, 0.85, None, 77)
    r4 = _chain(spec, 4)
    r8 = _chain(spec, 8)
    assert r8["mse"] < r4["mse"] / 50            # step shrinks 17x -> noise ~ 290x smaller
    assert r8["bits_per_value"] > r4["bits_per_value"]
    assert r8["mse"] <= (r8["model"].step ** 2 / 12) * 1.5 + 1e-9


def test_faster_eigenvalue_decay_compresses_better():
    # Section 4 / Appendix G: fast-decaying spectra are more compressible.
    rates = [_chain(fm.LayerSpec(32, 14, 14, r, None, 31), 5)["bits_per_value"]
             for r in (0.8, 0.9, 0.97)]
    assert rates[0] < rates[1] < rates[2]


def test_tail_channels_collapse_to_one_symbol():
    # Appendix E: the last coefficient channels map to a single value, so the entropy coder
    # spends one bit on them (per-channel tables).
    spec = fm.LayerSpec(24, 16, 16, 0.6, None, 13)
    p = fm.layer_params(spec)
    cal = fm.make_plain_gaussian(p, 8).float()
    m = oracle.fit_pca(cal, 4)
    q = oracle.quantize(m, oracle.project(m, cal))
    assert len(np.unique(q[:, -1])) == 1
    hist = oracle.histogram(q, 4, True)
    ln = oracle.huffman_lengths(hist, 12)
    assert oracle.entropy(hist[-1]) == 0.0
    assert ln[-1][q[0, -1]] == 1
    assert oracle.entropy(hist[0]) > 2.0         # while the leading channel carries the bits
    s = oracle.encode(q, ln, 4, chunk_pixels=1, tile_pixels=128)
    assert np.array_equal(oracle.decode_symbols(s, ln, 4), q)


def test_transform_beats_plain_quantisation_plus_vlc():
    # Section 4 ablation ordering: PCA + Q + VLC < Q + VLC < fixed-length b bits.
    spec = fm.LayerSpec(32, 14, 14, 0.8, None, 19)
    with_pca = _chain(spec, 5)
    without = _chain(spec, 5, identity=True)
    assert with_pca["bits_per_value"] < without["bits_per_value"] < 5.0


def test_channel_entropies_differ_by_log_sigma_ratio():
    # Appendix D: under one common step, R_i - R_j = log2(sigma_i / sigma_j) while sigma >> step.
    spec = fm.LayerSpec(8, 48, 48, 0.7, None, 23)
    p = fm.layer_params(spec)
    x = fm.make_plain_gaussian(p, 24).float()
    m = oracle.fit_pca(x, 8)
    q = oracle.quantize(m, oracle.project(m, x))
    hist = oracle.histogram(q, 8, True)
    h = [oracle.entropy(hist[j]) for j in range(4)]
    for j in range(3):
        want = 0.5 * math.log2(m.eig[j] / m.eig[j + 1])
        assert h[j] - h[j + 1] == pytest.approx(want, abs=0.06)


def test_huffman_rate_within_one_bit_of_entropy_on_calibration_data():
    r = _chain(fm.LayerSpec(16, 14, 14, 0.85, None, 29), 6)
    smoothed = r["hist"][0] + 1
    h = oracle.entropy(smoothed)
    l = oracle.mean_length(smoothed, r["lengths"][0])
    assert h <= l < h + 1


def test_bf16_chain():
    r = _chain(fm.LayerSpec(16, 7, 7, 0.9, None, 41), 4, dtype=torch.bfloat16)
    assert r["mse"] < 0.05
    assert np.array_equal(torch.tensor(r["xhat"]).to(torch.bfloat16).float().numpy(), r["xhat"])
