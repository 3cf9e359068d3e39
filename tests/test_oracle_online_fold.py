"""Oracle pins for the online covariance estimate (Section 3.1: the covariance "can be updated
online"), the non-linearity after the decoder (Section 3.1) and the folding of the transform
into the neighbouring convolutions (Section 3.1, "Linear transform")."""
import numpy as np
import torch

import oracle
from synth import featuremaps as fm


def _maps(c=12, s=6, n=5, seed=42, calib=True):
    params = fm.layer_params(fm.LayerSpec(c, s, s, 0.85, None, seed))
    return fm.make_maps(params, n, calib=calib, dtype=torch.float32)


# ---- running moments --------------------------------------------------------------------------

def test_moments_hand_example():
    # two channels, three pixels: (1, 0), (2, 1), (4, 5)
    x = np.array([[[[1.0, 2.0, 4.0]], [[0.0, 1.0, 5.0]]]], dtype=np.float32)      # N=1, C=2, H=1, W=3
    st = oracle.Moments(2).update(x)
    assert st.count == 3
    assert np.array_equal(st.sum, [7.0, 6.0])
    assert np.array_equal(st.outer, [[21.0, 22.0], [22.0, 26.0]])
    mean, cov = st.mean_cov()
    assert np.allclose(mean, [7.0 / 3.0, 2.0], rtol=0, atol=1e-15)
    # (S - s s^T / 3) / 2
    assert np.allclose(cov, [[14.0 / 6.0, 4.0], [4.0, 7.0]], rtol=0, atol=1e-14)


def test_moments_are_additive_and_match_the_two_pass_estimate():
    x = _maps(n=7)
    whole = oracle.Moments(x.shape[1]).update(x)
    a = oracle.Moments(x.shape[1]).update(x[:3])
    b = oracle.Moments(x.shape[1]).update(x[3:])
    merged = a.merge(b)
    assert merged.count == whole.count == 7 * 36
    assert np.allclose(merged.sum, whole.sum, rtol=1e-13, atol=0)
    assert np.allclose(merged.outer, whole.outer, rtol=1e-13, atol=1e-13)
    # batch by batch is the same as at once
    seq = oracle.Moments(x.shape[1])
    for i in range(7):
        seq.update(x[i:i + 1])
    assert np.allclose(seq.outer, whole.outer, rtol=1e-13, atol=1e-13)
    mean, cov = whole.mean_cov()
    mean2, cov2 = oracle.mean_cov(x)
    assert np.allclose(mean, mean2, rtol=1e-13, atol=1e-15)
    assert np.allclose(cov, cov2, rtol=1e-10, atol=1e-13)
    flat = x.numpy().transpose(1, 0, 2, 3).reshape(x.shape[1], -1).astype(np.float64)
    assert np.allclose(cov, np.cov(flat), rtol=1e-10, atol=1e-13)
    assert np.allclose(cov, cov.T, rtol=0, atol=0)


def test_fit_from_moments_equals_the_one_shot_fit():
    x = _maps(c=16, n=6)
    st = oracle.Moments(16).update(x[:2]).update(x[2:])
    got = oracle.fit_pca_moments(st, x, 6)
    want = oracle.fit_pca(x, 6)
    assert np.allclose(got.eig, want.eig, rtol=1e-9, atol=1e-14)
    assert np.allclose(got.mean, want.mean, rtol=1e-13, atol=1e-15)
    lead = want.eig > 1e-6 * want.eig[0]                       # directions whose eigenvalue is well above rounding
    assert np.allclose(got.basis[lead], want.basis[lead], rtol=0, atol=1e-7)
    assert np.isclose(got.lo, want.lo, rtol=1e-9) and np.isclose(got.step, want.step, rtol=1e-9)
    # the range follows the maps it is measured on: a subset can only narrow it
    sub = oracle.fit_pca_moments(st, x[:1], 6)
    assert sub.lo >= got.lo - 1e-12 and sub.lo + 63 * sub.step <= got.lo + 63 * got.step + 1e-12
    # orthonormal rows, descending eigenvalues
    assert np.allclose(got.basis @ got.basis.T, np.eye(16), atol=1e-12)
    assert np.all(np.diff(got.eig) <= 1e-15)


# ---- non-linearity after the decoder ------------------------------------------------------------

def test_relu_after_the_decoder():
    x = _maps(c=8, n=4)
    m = oracle.fit_pca(x, 3)
    test = _maps(c=8, n=2, calib=False)
    q = oracle.quantize(m, oracle.project(m, test))
    for bf16 in (False, True):
        plain = oracle.reconstruct(m, q, test.shape, out_bf16=bf16)
        relu = oracle.reconstruct(m, q, test.shape, out_bf16=bf16, relu=True)
        assert (plain < 0).any(), "the case must have something to clip"
        # rounding is monotone and keeps zero, so the non-linearity commutes with it
        assert np.array_equal(relu, np.maximum(plain, 0.0))
    # hand example: identity basis, mean (1, -3), levels lo + q * step = -2 + q
    ident = oracle.Model(2, 2, 2, np.array([1.0, -3.0]), np.eye(2), np.ones(2), -2.0, 1.0, "f64", 1.0)
    qq = np.array([[0, 3], [3, 0]], dtype=np.uint8)                 # y_hat = (-2, 1), (1, -2)
    out = oracle.reconstruct(ident, qq, (1, 2, 1, 2), out_bf16=False, relu=True)
    # x_hat = y_hat + mean = (-1, -2), (2, -5) -> clipped
    assert np.array_equal(out.reshape(2, 2), [[0.0, 2.0], [0.0, 0.0]])


# ---- folding ------------------------------------------------------------------------------------

def _conv_valid(u, w, bias):
    """Direct convolution (cross-correlation, no padding): u [Cin][H][W], w [Cout][Cin][kh][kw]."""
    cout, cin, kh, kw = w.shape
    h, wd = u.shape[1] - kh + 1, u.shape[2] - kw + 1
    out = np.zeros((cout, h, wd))
    for o in range(cout):
        for i in range(h):
            for j in range(wd):
                acc = bias[o]
                for ci in range(cin):
                    for a in range(kh):
                        for b in range(kw):
                            acc += w[o, ci, a, b] * u[ci, i + a, j + b]
                out[o, i, j] = acc
    return out


def _small_model(c, k, seed):
    rng = np.random.default_rng(seed)
    qmat, _ = np.linalg.qr(rng.standard_normal((c, c)))
    return oracle.Model(c, k, 4, rng.standard_normal(c), np.ascontiguousarray(qmat.T), np.ones(c), -1.0, 0.25, "f64", 1.0)


def test_fold_forward_against_direct_convolution():
    rng = np.random.default_rng(7)
    c, k, cin = 4, 3, 3
    m = _small_model(c, k, 8)
    w = rng.standard_normal((c, cin, 3, 3))
    bias, scale, shift = rng.standard_normal(c), rng.uniform(0.5, 2.0, c), rng.standard_normal(c)
    u = rng.standard_normal((cin, 5, 5))
    z = scale[:, None, None] * _conv_valid(u, w, bias) + shift[:, None, None]         # conv -> batch norm
    y = np.einsum("jc,chw->jhw", m.basis[:k], z - m.mean[:, None, None])             # encoder's transform
    wf, bf = oracle.fold_forward(m, w, bias, scale, shift)
    assert wf.shape == (k, cin * 9) and bf.shape == (k,)
    y_folded = _conv_valid(u, wf.reshape(k, cin, 3, 3), bf)
    assert np.allclose(y_folded, y, rtol=1e-12, atol=1e-12)


def test_fold_inverse_against_direct_convolution():
    rng = np.random.default_rng(9)
    c, k, cout = 4, 3, 2
    m = _small_model(c, k, 10)
    wn = rng.standard_normal((cout, c, 3, 3))
    bias = rng.standard_normal(cout)
    yh = rng.standard_normal((k, 5, 5))
    xh = np.einsum("jc,jhw->chw", m.basis[:k], yh) + m.mean[:, None, None]             # decoder's inverse transform
    v = _conv_valid(xh, wn, bias)
    wi, bi = oracle.fold_inverse(m, wn.reshape(cout, c, 9), bias)
    assert wi.shape == (cout, k, 9) and bi.shape == (cout,)
    v_folded = _conv_valid(yh, wi.reshape(cout, k, 3, 3), bi)
    assert np.allclose(v_folded, v, rtol=1e-12, atol=1e-12)
    # 1 x 1 next layer: the folded weights are W T^T
    w1 = rng.standard_normal((cout, c, 1))
    wi1, bi1 = oracle.fold_inverse(m, w1, bias)
    assert np.allclose(wi1[:, :, 0], w1[:, :, 0] @ m.basis[:k].T, atol=1e-13)
    assert np.allclose(bi1, bias + w1[:, :, 0] @ m.mean, atol=1e-13)
