"""A chained two-layer workload calibrated layer by layer (Section 3.1, "Linear transform": the
covariance of a layer is estimated with the layers before it already quantised; Fig. 2: encoder,
memory, decoder, non-linearity, next convolution), against the CPU oracle doing the same chain.

Layer 1 is a synthetic feature map (the output of a convolution + batch normalisation); the stage
between the layers is a seeded 3 x 3 convolution.  Checked:
  * stage by stage, on shared inputs, the library matches the oracle under the usual bars;
  * layer 2's calibration saw layer 1's *reconstruction*: its model equals a fit on those maps and
    differs from a fit on the clean maps, and it codes the maps it meets at inference no worse;
  * the whole chain's rate and distortion agree with the oracle's chain within 2 %;
  * the inverse transform folded into the next convolution (tc_fold_inverse) gives what decoding and
    then convolving gives."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10830_b200 as tc
from synth import featuremaps as fm
from tests import helpers as H

pytestmark = pytest.mark.gpu

C1, C2, SIDE, BITS = 64, 96, 14, (4, 5)


def _conv_weights(seed: int):
    g = torch.Generator().manual_seed(seed)
    w = torch.randn(C2, C1, 3, 3, generator=g) * (1.5 / np.sqrt(C1 * 9))
    b = torch.randn(C2, generator=g) * 0.1
    return w, b


def _stage2(w, b, dtype):
    def f(x):
        y = torch.nn.functional.conv2d(x.float(), w.to(x.device), b.to(x.device), padding=1)
        return y.to(dtype)
    return f


def _oracle_layer(z_cal, bits):
    m = oracle.fit_pca(z_cal, bits, basis_round="bf16", zero_level=True)
    q = oracle.quantize(m, oracle.project(m, z_cal))
    lengths = oracle.huffman_lengths(oracle.histogram(q, bits, False), 12)
    return m, lengths


def _oracle_code(m, lengths, bits, z, relu):
    q = oracle.quantize(m, oracle.project(m, z))
    nbits = oracle.encode(q, lengths, bits, chunk_pixels=1 << max(0, (127 // m.k).bit_length()), tile_pixels=128).total_bits
    xhat = oracle.reconstruct(m, q, z.shape, out_bf16=True, relu=relu)
    return torch.from_numpy(xhat).to(torch.bfloat16), nbits, q


def test_two_layer_chain_calibrated_layer_by_layer():
    dtype = torch.bfloat16
    params = fm.layer_params(fm.LayerSpec(C1, SIDE, SIDE, 0.9, None, 8100))
    cal = fm.make_maps(params, 24, calib=True, dtype=dtype)
    x = fm.make_maps(params, 6, dtype=dtype)
    w, b = _conv_weights(8101)
    stages = [lambda t: t, _stage2(w, b, dtype)]
    ctx = tc.tc_create(0)
    layers = tc.calibrate_layer_by_layer(ctx, stages, cal.cuda(), BITS, relu=(True, False))
    maps, recons, bits_gpu = tc.run_chain(ctx, stages, layers, x.cuda())
    assert tc.tc_get_status(ctx) == 0

    # ---- the oracle's chain on the CPU ------------------------------------------------------
    m1, len1 = _oracle_layer(cal, BITS[0])
    cal_hat1, _, _ = _oracle_code(m1, len1, BITS[0], cal, True)
    z2_cal = stages[1](cal_hat1)
    m2, len2 = _oracle_layer(z2_cal, BITS[1])
    x_hat1, nb1, _ = _oracle_code(m1, len1, BITS[0], x, True)
    z2 = stages[1](x_hat1)
    x_hat2, nb2, _ = _oracle_code(m2, len2, BITS[1], z2, False)

    # ---- stage by stage on shared inputs: the library's models imported into the oracle -------
    for l, (z_gpu, r_gpu) in enumerate(zip(maps, recons)):
        d = tc.tc_model_export(layers[l].model)
        m = oracle.Model(d["c"], d["k"], BITS[l], d["mean"], d["basis"], d["eig"], d["lo"], d["step"], "bf16")
        lengths = tc.tc_codebook_export(layers[l].codebook)
        enc = tc.tc_encode(ctx, layers[l].model, layers[l].codebook, z_gpu, debug=True)
        q_gpu = enc.symbols.cpu().numpy()
        q, units = oracle.quantize(m, oracle.project(m, z_gpu.cpu()), with_units=True)
        bad = q_gpu != q
        assert bad.mean() <= 1e-4
        if bad.any():
            assert np.all(np.abs(units[bad] - np.floor(units[bad]) - 0.5) <= 1e-3)
        ref = oracle.encode(q_gpu, lengths, BITS[l], chunk_pixels=enc.layout.chunk_pixels,
                            pixel_splits=enc.layout.pixel_splits, tile_pixels=128)
        assert np.array_equal(H.stream_words(enc), ref.words) and np.array_equal(H.chunk_len(enc), ref.chunk_len)
        want = oracle.reconstruct(m, q_gpu, tuple(z_gpu.shape), out_bf16=True, relu=layers[l].relu)
        got = r_gpu.float().cpu().numpy()
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
        assert np.all(np.abs(got - want) <= np.maximum(1e-3 * np.maximum(np.abs(want), m.step), ulp))
        assert H.count_output_flips(got, want) <= H.flip_allowance(H.expected_output_flips(m, q_gpu))

    # ---- layer 2 was calibrated on layer 1's reconstruction ------------------------------------
    g2 = tc.tc_model_export(layers[1].model)
    assert np.allclose(g2["mean"], m2.mean, rtol=0, atol=2e-3 * np.abs(m2.mean).max())
    assert np.allclose(g2["eig"][:16], m2.eig[:16], rtol=2e-2)
    clean = oracle.fit_pca(stages[1](torch.clamp_min(cal.float(), 0).to(dtype)), BITS[1], basis_round="bf16", zero_level=True)
    assert abs(clean.eig[0] - m2.eig[0]) > 1e-4 * m2.eig[0]                       # the clean maps have other statistics
    q_noisy = oracle.quantize(m2, oracle.project(m2, z2))
    q_clean = oracle.quantize(clean, oracle.project(clean, z2))
    mse_noisy = oracle.mse(z2, oracle.reconstruct(m2, q_noisy, z2.shape, out_bf16=True))
    mse_clean = oracle.mse(z2, oracle.reconstruct(clean, q_clean, z2.shape, out_bf16=True))
    assert mse_noisy <= 1.25 * mse_clean

    # ---- the two chains agree: rate within 2 %, distortion of the final map within 2 % ----------
    assert abs(bits_gpu[0] - nb1) <= 0.02 * nb1 and abs(bits_gpu[1] - nb2) <= 0.02 * nb2
    ref_final = stages[1](torch.clamp_min(x.float(), 0).to(dtype)).float()
    mse_gpu = float(((recons[1].float().cpu() - ref_final) ** 2).mean())
    mse_cpu = float(((x_hat2.float() - ref_final) ** 2).mean())
    assert abs(mse_gpu - mse_cpu) <= 0.02 * mse_cpu

    # ---- folding the inverse transform into the next convolution (no non-linearity in between) ---
    d1 = tc.tc_model_export(layers[0].model)
    mo = oracle.Model(d1["c"], d1["k"], BITS[0], d1["mean"], d1["basis"], d1["eig"], d1["lo"], d1["step"], "bf16")
    enc1 = tc.tc_encode(ctx, layers[0].model, layers[0].codebook, maps[0][:2].contiguous(), debug=True)
    q1 = enc1.symbols.cpu().numpy().astype(np.float64)
    yhat = (mo.lo + q1 * mo.step).reshape(2, SIDE, SIDE, mo.k).transpose(0, 3, 1, 2)       # dequantised coefficients as maps
    wf, bf = tc.tc_fold_inverse(layers[0].model, mo.k, w.double().numpy().reshape(C2, C1, 9), b.double().numpy())
    folded = torch.nn.functional.conv2d(torch.from_numpy(yhat), torch.from_numpy(wf.reshape(C2, mo.k, 3, 3)),
                                        torch.from_numpy(bf), padding=1)
    xh = (yhat.transpose(0, 2, 3, 1) @ mo.basis[:mo.k] + mo.mean).transpose(0, 3, 1, 2)        # decoder in fp64, no rounding
    direct = torch.nn.functional.conv2d(torch.from_numpy(xh), w.double(), b.double(), padding=1)
    inner = (slice(None), slice(None), slice(1, SIDE - 1), slice(1, SIDE - 1))                  # zero padding breaks the constant at the border
    assert torch.allclose(folded[inner], direct[inner], rtol=1e-10, atol=1e-10)

    for layer in layers:
        layer.close()
    ctx.close()
