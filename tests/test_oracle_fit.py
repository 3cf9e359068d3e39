"""Pins for the oracle's fit, projection and reconstruction (Section 3; Section 3.1 "Linear
transform" and "Quantization").  None of these re-type the oracle's own formulas: they use a
hand-worked 2-channel example, numpy's eigensolver, a generator with a known covariance, and
the invariants the paper states (T orthonormal, T Sigma T^T diagonal)."""
import math

import numpy as np
import pytest
import torch

import oracle
from synth import featuremaps as fm


def _hand_example():
    # Four pixel vectors with mean 0 and unbiased covariance [[2,1],[1,2]]:
    # +-a(1,1), +-b(1,-1) with a^2 = 9/4, b^2 = 3/4.  Eigenpairs: 3 -> (1,1)/sqrt2,
    # 1 -> (1,-1)/sqrt2 (sign rule: first entry of largest magnitude positive).
    a, b = 1.5, math.sqrt(3) / 2
    pts = np.array([[a, a], [-a, -a], [b, -b], [-b, b]])
    x = pts.T.reshape(1, 2, 2, 2).astype(np.float32)   # N=1, C=2, H=W=2; pixel s = column s
    return x, pts, a, b


def test_mean_cov_hand_example():
    x, pts, a, b = _hand_example()
    mean, cov = oracle.mean_cov(x)
    assert np.allclose(mean, 0.0, atol=1e-7)
    assert np.allclose(cov, [[2.0, 1.0], [1.0, 2.0]], atol=1e-6)


def test_fit_hand_example_basis_range_and_projection():
    x, pts, a, b = _hand_example()
    m = oracle.fit_pca(x, bits=2)
    r = 1 / math.sqrt(2)
    assert np.allclose(m.eig, [3.0, 1.0], atol=1e-6)
    assert np.allclose(m.basis, [[r, r], [r, -r]], atol=1e-7)
    # coefficient 0 of the four pixels: +3/sqrt2, -3/sqrt2, 0, 0  -> range and step
    assert m.lo == pytest.approx(-3 * r, abs=1e-6)
    assert m.step == pytest.approx(6 * r / 3, abs=1e-6)
    y = oracle.project(m, x)
    want = np.array([[3 * r, 0], [-3 * r, 0], [0, 2 * b * r], [0, -2 * b * r]])
    assert np.allclose(y, want, atol=1e-6)
    # levels: lo + q*step = -3r, -r, +r, +3r.  y0 = 0 is a tie between q=1 and q=2 in exact
    # arithmetic; coefficient 1 = +-1.2247 -> units 1.5 +- 0.866 -> q = 2 and 1.
    q = oracle.quantize(m, y)
    assert q[0, 0] == 3 and q[1, 0] == 0
    assert q[2, 1] == 2 and q[3, 1] == 1


def test_mean_cov_matches_numpy_cov():
    p = fm.layer_params(fm.LayerSpec(12, 5, 7, 0.8, None, 11))
    x = fm.make_maps(p, 6).numpy()
    mean, cov = oracle.mean_cov(x)
    samples = x.transpose(1, 0, 2, 3).reshape(12, -1).astype(np.float64)
    assert np.allclose(mean, samples.mean(axis=1), rtol=0, atol=1e-12)
    assert np.allclose(cov, np.cov(samples), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("n", [3, 16, 64])
def test_jacobi_against_numpy_eigh(n):
    rng = np.random.default_rng(n)
    a = rng.standard_normal((n, n))
    a = a @ a.T + np.diag(rng.uniform(0, 2, n))
    ev, vt, sweeps = oracle.eigh_jacobi(a)
    assert 0 <= sweeps < 30
    ref = np.linalg.eigvalsh(a)
    assert np.allclose(np.sort(ev), ref, rtol=1e-11, atol=1e-11)
    assert np.allclose(vt @ vt.T, np.eye(n), atol=1e-12)          # T T^T = I
    assert np.allclose(vt @ a @ vt.T, np.diag(ev), atol=1e-9 * np.abs(ref).max())


def test_jacobi_diagonal_and_degenerate():
    ev, vt, _ = oracle.eigh_jacobi(np.diag([3.0, 1.0, 2.0]))
    assert np.allclose(ev, [3.0, 1.0, 2.0]) and np.allclose(vt, np.eye(3))
    ev, vt, _ = oracle.eigh_jacobi(np.zeros((4, 4)))
    assert np.allclose(ev, 0.0)


def test_fit_invariants_and_order_on_synthetic_layer():
    p = fm.layer_params(fm.LayerSpec(32, 14, 14, 0.85, None, 5))
    x = fm.make_maps(p, 8, calib=True)
    m = oracle.fit_pca(x, bits=6)
    t = m.basis
    assert np.allclose(t @ t.T, np.eye(32), atol=1e-12)
    _, cov = oracle.mean_cov(x)
    d = t @ cov @ t.T
    assert np.allclose(d, np.diag(m.eig), atol=1e-10 * np.abs(cov).max())
    assert np.all(np.diff(m.eig) <= 1e-15)
    assert m.eig.sum() == pytest.approx(np.trace(cov), rel=1e-12)
    for row in t:                                        # sign rule
        assert row[np.argmax(np.abs(row))] > 0
    # range = min/max of coefficient 0 over calibration pixels
    y = oracle.project(m, x)
    assert m.lo == y[:, 0].min()
    assert m.step == pytest.approx((y[:, 0].max() - y[:, 0].min()) / 63, rel=1e-15)
    # transformed channels are uncorrelated with variances = eigenvalues
    assert np.allclose(np.cov(y.T), np.diag(m.eig), atol=1e-9)


def test_fit_recovers_known_covariance():
    # Without blur/bias/ReLU the generator's covariance is exactly Q diag(lam) Q^T.
    spec = fm.LayerSpec(8, 32, 32, 0.6, None, 3)
    p = fm.layer_params(spec)
    x = fm.make_plain_gaussian(p, 64).float()
    m = oracle.fit_pca(x, bits=8)
    lam = p.lam.numpy()
    msamples = 64 * 32 * 32
    assert np.allclose(m.eig, lam, rtol=6 * math.sqrt(2 / msamples) + 1e-3)
    q = p.q.numpy()
    for j in range(4):                                   # well separated leading directions
        assert abs(abs(m.basis[j] @ q[:, j]) - 1.0) < 5e-3


def test_bf16_basis_is_bf16_exact_and_used_for_range():
    p = fm.layer_params(fm.LayerSpec(16, 8, 8, 0.85, None, 9))
    x = fm.make_maps(p, 8, calib=True)
    m = oracle.fit_pca(x, bits=4, basis_bf16=True)
    as_bf16 = torch.tensor(m.basis).to(torch.bfloat16).double().numpy()
    assert np.array_equal(as_bf16, m.basis)
    full = oracle.fit_pca(x, bits=4, basis_bf16=False)
    assert np.abs(m.basis - full.basis).max() <= 2.0 ** -9      # half a bf16 ulp below 1
    y = oracle.project(m, x)
    assert m.lo == y[:, 0].min()


@pytest.mark.parametrize("v,want", [(1.0, 1.0), (1.00390625, 1.0), (1.01171875, 1.015625),
                                    (1.0078125, 1.0078125), (-3.0e-5, None), (0.0, 0.0)])
def test_round_bf16_against_torch(v, want):
    got = oracle.round_bf16(v)
    ref = float(torch.tensor(v, dtype=torch.float64).to(torch.bfloat16).double())
    # torch rounds double -> float -> bf16; for these values no double rounding occurs
    assert got == ref
    if want is not None:
        assert got == want


def test_parseval_and_near_lossless_bound():
    # Orthonormal T: |x - x_hat| = |y - y_hat| (Section 3), and with every coefficient inside
    # the quantiser range each coefficient errs by at most step/2, so per pixel
    # |x - x_hat|_2 <= sqrt(C) * step / 2.
    p = fm.layer_params(fm.LayerSpec(16, 10, 10, 0.85, None, 21))
    x = fm.make_maps(p, 4, calib=True)
    m = oracle.fit_pca(x, bits=8)
    y = oracle.project(m, x)
    q = oracle.quantize(m, y)
    inside = np.all((y >= m.lo) & (y <= m.lo + 255 * m.step), axis=1)
    assert inside.mean() > 0.9
    xhat = oracle.reconstruct(m, q, x.shape, out_bf16=False)
    xs = x.numpy().transpose(0, 2, 3, 1).reshape(-1, 16).astype(np.float64)
    xh = xhat.transpose(0, 2, 3, 1).reshape(-1, 16).astype(np.float64)
    ex = np.linalg.norm(xs - xh, axis=1)
    yhat = m.lo + q * m.step
    ey = np.linalg.norm(y - yhat, axis=1)
    assert np.allclose(ex, ey, atol=1e-6)                        # fp32 output rounding only
    assert np.all(ex[inside] <= math.sqrt(16) * m.step / 2 + 1e-6)
    assert oracle.mse(x, xhat) == pytest.approx(np.mean((xs - xh) ** 2), rel=1e-9)


def test_reconstruct_hand_example():
    x, pts, a, b = _hand_example()
    m = oracle.fit_pca(x, bits=2)
    r = 1 / math.sqrt(2)
    # q = (3, 2): y_hat = (3r, r) -> x_hat = T^T y_hat = r*(3r + r, 3r - r) = (2, 1)
    # q = (0, 3): y_hat = (-3r, 3r) -> x_hat = r*(-3r + 3r, -3r - 3r) = (0, -3)
    q = np.array([[3, 2], [0, 1], [3, 0], [0, 3]], dtype=np.uint8)
    xhat = oracle.reconstruct(m, q, (1, 2, 2, 2), out_bf16=False)
    got = xhat.reshape(2, 4).T
    want = np.array([[2.0, 1.0], [-2.0, -1.0], [0.0, 3.0], [0.0, -3.0]])
    assert np.allclose(got, want, atol=1e-6)


def test_reconstruct_rounds_to_bf16():
    p = fm.layer_params(fm.LayerSpec(8, 6, 6, 0.85, None, 4))
    x = fm.make_maps(p, 2, calib=True, dtype=torch.bfloat16)
    m = oracle.fit_pca(x, bits=5, basis_bf16=True)
    q = oracle.quantize(m, oracle.project(m, x))
    full = oracle.reconstruct(m, q, x.shape, out_bf16=False)
    half = oracle.reconstruct(m, q, x.shape, out_bf16=True)
    assert np.array_equal(torch.tensor(half).to(torch.bfloat16).float().numpy(), half)
    assert np.all(np.abs(half - full) <= np.abs(full) * 2.0 ** -8 + 1e-30)


def test_lapack_step_agrees_with_jacobi_and_f32_rounding():
    # Above oracle.JACOBI_MAX_C channels the fit takes its eigendecomposition from LAPACK; on a
    # layer small enough for both, the two routes give the same transform.
    p = fm.layer_params(fm.LayerSpec(24, 9, 9, 0.8, None, 17))
    x = fm.make_maps(p, 12, calib=True)
    a = oracle.fit_pca(x, bits=6, eigensolver="jacobi")
    b = oracle.fit_pca(x, bits=6, eigensolver="lapack")
    assert np.allclose(a.eig, b.eig, rtol=1e-10, atol=1e-14)
    lead = a.eig > 1e-6 * a.eig[0]
    assert np.allclose(a.basis[lead], b.basis[lead], atol=1e-7)
    assert a.lo == pytest.approx(b.lo, rel=1e-9) and a.step == pytest.approx(b.step, rel=1e-9)
    f = oracle.fit_pca(x, bits=6, basis_round="f32")
    assert np.array_equal(f.basis.astype(np.float32).astype(np.float64), f.basis)
    assert np.abs(f.basis - a.basis).max() <= 2.0 ** -24
    m4 = oracle.with_bits(a, 4)
    assert m4.lo == a.lo and m4.step == pytest.approx(a.step * 63 / 15, rel=1e-14)


# ---- quantiser grid with zero on a level (Section 3.1 "Quantization"; Appendix E) ----------------

def test_zero_level_grid_hand_values():
    # round(-lo / step) levels below zero, ties to even; the step is kept
    assert oracle.zero_level_lo(-3.2, 1.0) == -3.0
    assert oracle.zero_level_lo(-3.7, 1.0) == -4.0
    assert oracle.zero_level_lo(-2.5, 1.0) == -2.0          # tie: two levels below zero
    assert oracle.zero_level_lo(-3.5, 1.0) == -4.0          # tie: four
    assert oracle.zero_level_lo(-0.26, 0.5) == -0.5
    assert oracle.zero_level_lo(0.2, 1.0) == 0.0            # a range that starts above zero: zero becomes the lowest level
    for lo, step in ((-1.2345, 0.071), (-17.0, 0.3), (-0.01, 2.0)):
        got = oracle.zero_level_lo(lo, step)
        assert abs(got - lo) <= 0.5 * step * (1 + 1e-12)
        assert abs(got / step - np.rint(got / step)) < 1e-9


def test_zero_level_fit_keeps_step_and_puts_zero_on_a_level():
    spec = fm.LayerSpec(24, 10, 10, 0.8, None, 321)
    x = fm.make_maps(fm.layer_params(spec), 12, calib=True).numpy()
    raw = oracle.fit_pca(x, bits=4)
    m = oracle.fit_pca(x, bits=4, zero_level=True)
    assert m.zero_level and not raw.zero_level
    assert m.step == raw.step and np.array_equal(m.basis, raw.basis) and np.array_equal(m.mean, raw.mean)
    assert m.lo == oracle.zero_level_lo(raw.lo, raw.step)
    assert m.cal_lo == raw.lo and m.cal_hi == pytest.approx(raw.lo + 15 * raw.step, rel=1e-14)
    # a zero coefficient vector (the mean map) quantises to the zero level and reconstructs exactly
    n_below = int(np.rint(-m.lo / m.step))
    q0 = oracle.quantize(m, np.zeros((1, 24)))
    assert np.all(q0 == n_below)
    xhat = oracle.reconstruct(m, q0, (1, 24, 1, 1), out_bf16=False)
    assert np.allclose(xhat.reshape(-1), m.mean.astype(np.float32), rtol=0, atol=1e-7)
    # changing the bit width re-divides the measured range, then shifts again
    m6 = oracle.with_bits(m, 6)
    assert m6.step == pytest.approx((m.cal_hi - m.cal_lo) / 63, rel=1e-14)
    assert m6.lo == oracle.zero_level_lo(m.cal_lo, m6.step)


def test_zero_level_collapses_low_variance_channels_to_one_value():
    # Appendix E: after the projection all values of a low-variance channel map to a single value.
    # With zero between two levels such a channel flips between both; with zero on a level it
    # does not, and both rate and distortion fall.
    spec = fm.LayerSpec(48, 12, 12, 0.8, None, 322)
    p = fm.layer_params(spec)
    cal = fm.make_maps(p, 24, calib=True).numpy()
    x = fm.make_maps(p, 6).numpy()
    raw = oracle.fit_pca(cal, bits=3)
    # pick a case where zero is clearly between two levels of the measured grid
    frac = (-raw.lo / raw.step) % 1.0
    assert 0.1 < frac < 0.9
    m = oracle.fit_pca(cal, bits=3, zero_level=True)
    out = {}
    for name, mod in (("raw", raw), ("zero", m)):
        q = oracle.quantize(mod, oracle.project(mod, x))
        tail = q[:, 40:]
        out[name] = dict(values=len(np.unique(tail)), entropy=oracle.entropy(oracle.histogram(q, 3, False)[0]),
                         mse=oracle.mse(x, oracle.reconstruct(mod, q, x.shape, out_bf16=False)))
    assert out["zero"]["values"] == 1
    assert out["zero"]["entropy"] < out["raw"]["entropy"]
    assert out["zero"]["mse"] < out["raw"]["mse"]
