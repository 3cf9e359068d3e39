"""GPU parity for the online fit (Section 3.1: the covariance can be updated online), the
non-linearity after the decoder (Section 3.1) and the folding helpers (Section 3.1, "Linear
transform"), each against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10830_b200 as tc
from synth import featuremaps as fm
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = tc.tc_create(0)
    yield c
    c.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_running_state_matches_the_oracle_and_is_additive(ctx, dtype):
    params = fm.layer_params(fm.LayerSpec(48, 10, 10, 0.9, None, 7100))
    cal = fm.make_maps(params, 9, calib=True, dtype=dtype)
    want = oracle.Moments(48).update(cal)
    st = tc.tc_fit_state_create(ctx, 48)
    for lo, hi in ((0, 2), (2, 3), (3, 9)):                     # batches of different sizes
        tc.tc_fit_state_update(ctx, st, cal[lo:hi].cuda())
    count, s1, s2 = tc.tc_fit_state_export(ctx, st)
    assert count == want.count == 900
    assert np.allclose(s1, want.sum, rtol=1e-12, atol=1e-12)
    assert np.allclose(s2, want.outer, rtol=1e-12, atol=1e-12)
    assert np.array_equal(s2, s2.T)
    # export -> merge on the host -> import (what a sum over devices, or a resumed run, does)
    a, b = tc.tc_fit_state_create(ctx, 48), tc.tc_fit_state_create(ctx, 48)
    tc.tc_fit_state_update(ctx, a, cal[:4].cuda())
    tc.tc_fit_state_update(ctx, b, cal[4:].cuda())
    ca, a1, a2 = tc.tc_fit_state_export(ctx, a)
    cb_, b1, b2 = tc.tc_fit_state_export(ctx, b)
    tc.tc_fit_state_import(ctx, a, ca + cb_, a1 + b1, a2 + b2)
    cm, m1, m2 = tc.tc_fit_state_export(ctx, a)
    assert cm == 900 and np.allclose(m1, s1, rtol=1e-13) and np.allclose(m2, s2, rtol=1e-12, atol=1e-12)
    for h in (st, a, b):
        h.close()


@pytest.mark.parametrize("dtype,basis_round", [(torch.float32, "f32"), (torch.bfloat16, "bf16")])
def test_online_fit_matches_the_oracle_and_the_one_shot_fit(ctx, dtype, basis_round):
    spec = fm.LayerSpec(32, 12, 12, 0.85, None, 7200)
    params = fm.layer_params(spec)
    cal = fm.make_maps(params, 8, calib=True, dtype=dtype)
    x = fm.make_maps(params, 3, dtype=dtype)
    bits = 5
    st = tc.tc_fit_state_create(ctx, 32)
    for i in range(0, 8, 2):
        tc.tc_fit_state_update(ctx, st, cal[i:i + 2].cuda())
    model = tc.tc_fit_state_finish(ctx, st, cal.cuda(), bits)
    got = tc.tc_model_export(model)
    want = oracle.fit_pca_moments(oracle.Moments(32).update(cal), cal, bits, basis_round=basis_round, zero_level=True)
    assert np.allclose(got["mean"], want.mean, rtol=1e-12, atol=1e-14)
    assert np.allclose(got["eig"], want.eig, rtol=1e-6, atol=1e-10 * want.eig[0])
    assert np.isclose(got["lo"], want.lo, rtol=1e-5, atol=1e-6) and np.isclose(got["step"], want.step, rtol=1e-5)
    lead = want.eig > 1e-4 * want.eig[0]
    ulp = 2.0 ** -7 if basis_round == "bf16" else 2.0 ** -22      # entries may round to the neighbouring value
    assert np.abs(got["basis"][lead] - want.basis[lead]).max() <= ulp
    # the one-shot fit of the same maps gives the same model (different summation, same estimate)
    ref = tc.tc_model_export(tc.tc_fit_pca(ctx, cal.cuda(), bits))
    assert np.allclose(got["eig"], ref["eig"], rtol=1e-8, atol=1e-12 * ref["eig"][0])
    assert np.isclose(got["lo"], ref["lo"], rtol=1e-6, atol=1e-7) and np.isclose(got["step"], ref["step"], rtol=1e-6)
    # and it codes: rate and distortion within 1 % of the oracle's model on the same maps
    stt = tc.tc_stats(ctx, model, None, cal.cuda())
    cb = tc.tc_build_codebook(ctx, model, stt.hist)
    enc = tc.tc_encode(ctx, model, cb, x.cuda())
    xh = tc.tc_decode(ctx, model, cb, enc, x.shape, dtype)
    assert tc.tc_get_status(ctx) == 0
    q = oracle.quantize(want, oracle.project(want, x))
    ref_hat = oracle.reconstruct(want, q, x.shape, out_bf16=(dtype == torch.bfloat16))
    mse_gpu = float(((xh.float().cpu() - x.float()) ** 2).mean())
    mse_ref = float(((torch.from_numpy(ref_hat) - x.float()) ** 2).mean())
    assert abs(mse_gpu - mse_ref) <= 0.01 * mse_ref + 1e-9
    # range measured on a subset of the maps can only be narrower
    sub = tc.tc_model_export(tc.tc_fit_state_finish(ctx, st, cal[:1].cuda(), bits, zero_level=False))
    whole = tc.tc_model_export(tc.tc_fit_state_finish(ctx, st, cal.cuda(), bits, zero_level=False))
    assert sub["lo"] >= whole["lo"] - 1e-9
    # the grid with zero on a level keeps the step and moves by at most half of it
    assert np.isclose(got["step"], whole["step"], rtol=1e-12) and abs(got["lo"] - whole["lo"]) <= 0.5 * got["step"] * (1 + 1e-9)
    assert abs(got["lo"] / got["step"] - np.rint(got["lo"] / got["step"])) < 1e-9
    st.close(); model.close(); cb.close()


def test_fit_state_rejects_bad_arguments(ctx):
    st = tc.tc_fit_state_create(ctx, 16)
    with pytest.raises(tc.TcError):
        tc.tc_fit_state_update(ctx, st, torch.zeros(1, 8, 4, 4, device="cuda"))      # channel mismatch
    with pytest.raises(tc.TcError):
        tc.tc_fit_state_finish(ctx, st, torch.zeros(1, 16, 4, 4, device="cuda"), 4)  # no samples yet
    tc.tc_fit_state_update(ctx, st, torch.ones(2, 16, 4, 4, device="cuda"))
    with pytest.raises(tc.TcError):
        tc.tc_fit_state_finish(ctx, st, torch.ones(1, 16, 4, 4, device="cuda"), 4)   # constant maps: no range
    st.close()


# (channels, map side, maps, dtype, kernels expected: 0 fp64, 1 / 3 tensor core, 2 fp32)
@pytest.mark.parametrize("c,s,n,dtype,route", [(32, 9, 3, torch.float32, 0), (64, 14, 3, torch.bfloat16, 1),
                                                (24, 9, 3, torch.bfloat16, 2), (320, 7, 4, torch.bfloat16, 3),
                                                (64, 5, 7, torch.bfloat16, 1)])
def test_relu_after_the_decoder_on_every_route(ctx, c, s, n, dtype, route):
    spec = fm.LayerSpec(c, s, s, 0.9, None, 7300 + c)
    o = H.oracle_side(spec, 4, max(4, (2 * c) // (s * s) + 1), n, dtype, False)
    m, lengths = o["model"], o["lengths"]
    model = H.import_model(tc, ctx, m, dtype)
    cb = tc.tc_codebook_import(ctx, lengths, 4)
    enc = tc.tc_encode(ctx, model, cb, o["x"].cuda(), debug=True)
    q_gpu = enc.symbols.cpu().numpy()
    plain = tc.tc_decode(ctx, model, cb, enc, o["x"].shape, dtype)
    relu = tc.tc_decode(ctx, model, cb, enc, o["x"].shape, dtype, relu=True)
    assert tc.tc_get_status(ctx) == 0 and tc.tc_last_path(ctx, True) == route
    # on the device: the flag clips what the plain decode returns, nothing else
    assert (plain < 0).any()
    assert torch.equal(relu, torch.clamp_min(plain, 0))
    # against the oracle: same bar as the plain decode
    want = oracle.reconstruct(m, q_gpu, o["x"].shape, out_bf16=(dtype == torch.bfloat16), relu=True)
    got = relu.float().cpu().numpy()
    if route == 0:
        assert np.array_equal(got, want)
    else:
        mant = 7 if dtype == torch.bfloat16 else 23
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - mant)
        assert np.all(np.abs(got - want) <= np.maximum(1e-3 * np.maximum(np.abs(want), m.step), ulp))
        assert (got == want).mean() >= 0.999
    model.close(); cb.close()


def test_folding_helpers_match_the_oracle(ctx):
    rng = np.random.default_rng(11)
    c, k, cin, cout = 32, 20, 5, 7
    params = fm.layer_params(fm.LayerSpec(c, 8, 8, 0.9, None, 7400))
    cal = fm.make_maps(params, 6, calib=True, dtype=torch.float32)
    m = oracle.fit_pca(cal, 6, k=k, basis_round="f32")
    model = H.import_model(tc, ctx, m, torch.float32)
    w = rng.standard_normal((c, cin * 9))
    bias, scale, shift = rng.standard_normal(c), rng.uniform(0.5, 2.0, c), rng.standard_normal(c)
    wf, bf = tc.tc_fold_forward(model, k, w, bias, scale, shift)
    wf0, bf0 = oracle.fold_forward(m, w, bias, scale, shift)
    assert np.allclose(wf, wf0, rtol=1e-12, atol=1e-13) and np.allclose(bf, bf0, rtol=1e-12, atol=1e-13)
    # defaults: no bias, no batch norm
    wf1, bf1 = tc.tc_fold_forward(model, k, w)
    wf2, bf2 = oracle.fold_forward(m, w, np.zeros(c), np.ones(c), np.zeros(c))
    assert np.allclose(wf1, wf2, rtol=1e-12, atol=1e-13) and np.allclose(bf1, bf2, rtol=1e-12, atol=1e-13)
    wn = rng.standard_normal((cout, c, 9))
    bn = rng.standard_normal(cout)
    wi, bi = tc.tc_fold_inverse(model, k, wn, bn)
    wi0, bi0 = oracle.fold_inverse(m, wn, bn)
    assert np.allclose(wi, wi0, rtol=1e-12, atol=1e-13) and np.allclose(bi, bi0, rtol=1e-12, atol=1e-13)
    model.close()
