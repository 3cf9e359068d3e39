"""The fit's device eigensolver (Section 3.1, "Linear transform": the PCA matrix comes from the
covariance of calibration data) against what the mathematics fixes -- numpy's symmetric solver,
orthonormality, the decomposition itself, a matrix built from a known spectrum -- against the
library's host solver, and the fit that uses it against the host-solver fit and the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10830_b200 as tc
from synth import featuremaps as fm

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = tc.tc_create(0)
    yield c
    c.close()


def _sym(n, seed, decay=0.9):
    """Q diag(lambda) Q^T with a geometric spectrum and a random orthogonal Q."""
    rng = np.random.default_rng(seed)
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    lam = 3.0 * decay ** np.arange(n)
    return (q * lam) @ q.T, lam, q


def _check_conventions(a, evals, evecs):
    n = a.shape[0]
    scale = max(1.0, np.abs(evals).max())
    assert np.all(np.diff(evals) <= 0.0)                                        # descending
    assert np.abs(evecs @ evecs.T - np.eye(n)).max() <= 1e-12                   # orthonormal rows
    assert np.abs(evecs @ a @ evecs.T - np.diag(evals)).max() <= 2e-13 * scale * max(1, n / 64)
    big = np.abs(evecs).argmax(axis=1)
    assert np.all(evecs[np.arange(n), big] > 0.0)                               # sign convention


@pytest.mark.parametrize("n", [1, 2, 3, 17, 64, 96, 255, 256, 511, 1024])
def test_device_eigh_against_numpy_and_the_host_solver(ctx, n):
    a, lam, _ = _sym(n, 900 + n)
    a = (a + a.T) / 2
    evals, evecs, sweeps = tc.tc_device_eigh(ctx, torch.from_numpy(a).cuda())
    evals, evecs = evals.cpu().numpy(), evecs.cpu().numpy()
    assert 1 <= sweeps <= 60 or n == 1
    _check_conventions(a, evals, evecs)
    bound = 1e-13 * max(1, n / 16) * lam.max()           # absolute accuracy: a few hundred eps |A| at n = 1024
    assert np.abs(evals - np.linalg.eigvalsh(a)[::-1]).max() <= bound
    assert np.abs(evals - lam).max() <= bound                                   # the spectrum it was built from
    h_evals, h_evecs = tc.tc_host_eigh(a)
    assert np.abs(evals - h_evals).max() <= bound
    # eigenvectors of well separated eigenvalues agree with the host solver's (same sign rule)
    gap_ok = np.ones(n, dtype=bool)
    if n > 1:
        gaps = np.minimum(np.r_[np.inf, -np.diff(h_evals)], np.r_[-np.diff(h_evals), np.inf])
        gap_ok = gaps > 1e-4 * lam.max()
    assert np.abs(evecs[gap_ok] - h_evecs[gap_ok]).max() <= 1e-8


def test_device_eigh_rank_deficient_and_repeated(ctx):
    rng = np.random.default_rng(77)
    b = rng.standard_normal((40, 12))
    a = b @ b.T                                   # rank 12 of 40: 28 null directions
    evals, evecs, sweeps = tc.tc_device_eigh(ctx, torch.from_numpy(a).cuda())
    evals, evecs = evals.cpu().numpy(), evecs.cpu().numpy()
    assert sweeps <= 20
    _check_conventions(a, evals, evecs)
    assert np.abs(evals[12:]).max() <= 1e-12 * evals[0]
    assert np.abs(evals - np.linalg.eigvalsh(a)[::-1]).max() <= 1e-12 * evals[0]
    # a multiple of the identity: nothing to rotate, one sweep, unit vectors
    evals, evecs, sweeps = tc.tc_device_eigh(ctx, torch.eye(9, dtype=torch.float64, device="cuda") * 2.5)
    assert sweeps == 1 and torch.all(evals == 2.5) and torch.equal(evecs, torch.eye(9, dtype=torch.float64, device="cuda"))
    # a diagonal matrix out of order: sorted, vectors are the unit vectors in that order
    d = torch.tensor([1.0, 5.0, 3.0], dtype=torch.float64, device="cuda")
    evals, evecs, _ = tc.tc_device_eigh(ctx, torch.diag(d))
    assert evals.tolist() == [5.0, 3.0, 1.0]
    assert torch.equal(evecs, torch.tensor([[0, 1, 0], [0, 0, 1], [1, 0, 0]], dtype=torch.float64, device="cuda"))


@pytest.mark.parametrize("dtype,basis_dtype,c", [(torch.float32, None, 64), (torch.bfloat16, None, 128),
                                                 (torch.bfloat16, tc.binding.TC_INT8, 64), (torch.bfloat16, None, 320)])
def test_fit_on_the_device_matches_the_host_solver_fit_and_the_oracle(ctx, dtype, basis_dtype, c):
    params = fm.layer_params(fm.LayerSpec(c, 8, 8, 0.92, None, 9100 + c))
    cal = fm.make_maps(params, 12, calib=True, dtype=dtype)
    dev = tc.tc_model_export(tc.tc_fit_pca(ctx, cal.cuda(), 5, basis_dtype=basis_dtype, eigensolver=tc.TC_EIG_DEVICE))
    host = tc.tc_model_export(tc.tc_fit_pca(ctx, cal.cuda(), 5, basis_dtype=basis_dtype, eigensolver=tc.TC_EIG_HOST))
    rounding = {None: "bf16" if dtype == torch.bfloat16 else "f32", tc.binding.TC_INT8: "int8"}[basis_dtype]
    want = oracle.fit_pca(cal, 5, basis_round=rounding, zero_level=True)
    assert np.array_equal(dev["mean"], host["mean"])
    for other in (host["basis"], want.basis):
        # the solvers agree to rounding: an entry may land on the neighbouring representable value
        # where its exact value sits at a rounding tie; directions of near-equal eigenvalues excepted
        gaps = np.minimum(np.r_[np.inf, -np.diff(want.eig)], np.r_[-np.diff(want.eig), np.inf])
        rows = gaps > 1e-9 * want.eig[0]
        mine, theirs = dev["basis"][rows], other[rows]
        if rounding == "int8":                     # compare the integers: the scales differ in their last bits
            mine = np.rint(mine / dev["basis_scale"])
            theirs = np.rint(theirs / (host["basis_scale"] if other is host["basis"] else want.basis_scale))
        ulp = {"bf16": 2.0 ** -8, "f32": 2.0 ** -23, "int8": 1.0}[rounding]
        assert np.abs(mine - theirs).max() <= ulp
        assert (mine == theirs).mean() >= 0.999
    assert np.allclose(dev["eig"], host["eig"], rtol=0, atol=1e-12 * host["eig"][0])
    assert np.isclose(dev["basis_scale"], host["basis_scale"], rtol=1e-12)
    assert np.isclose(dev["lo"], host["lo"], rtol=1e-9, atol=1e-12) and np.isclose(dev["step"], host["step"], rtol=1e-9)
    assert np.isclose(dev["lo"], want.lo, rtol=1e-6, atol=1e-6) and np.isclose(dev["step"], want.step, rtol=1e-6)


def test_online_fit_finishes_on_the_device(ctx):
    params = fm.layer_params(fm.LayerSpec(96, 6, 6, 0.9, None, 9300))
    cal = fm.make_maps(params, 20, calib=True, dtype=torch.bfloat16).cuda()
    st = tc.tc_fit_state_create(ctx, 96)
    for lo, hi in ((0, 7), (7, 20)):
        tc.tc_fit_state_update(ctx, st, cal[lo:hi])
    online = tc.tc_model_export(tc.tc_fit_state_finish(ctx, st, cal, 4))
    online_host = tc.tc_model_export(tc.tc_fit_state_finish(ctx, st, cal, 4, eigensolver=tc.TC_EIG_HOST))
    oneshot = tc.tc_model_export(tc.tc_fit_pca(ctx, cal, 4))
    for other in (online_host, oneshot):
        assert np.allclose(online["mean"], other["mean"], rtol=1e-12, atol=1e-12)
        assert np.allclose(online["eig"], other["eig"], rtol=0, atol=1e-10 * other["eig"][0])
        assert np.abs(online["basis"] - other["basis"]).max() <= 2.0 ** -8
        assert (online["basis"] == other["basis"]).mean() >= 0.999
        assert np.isclose(online["lo"], other["lo"], rtol=1e-6, atol=1e-6) and np.isclose(online["step"], other["step"], rtol=1e-6)
