"""CPU-side checks of the CUDA library: it loads, exports every symbol the header declares,
refuses to run without a device, and its host algorithms (Huffman lengths, eigensolver) agree
with the oracle / numpy."""
import os
import re

import numpy as np
import pytest

import oracle
import paper_1905_10830_b200 as tc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1905_10830_b200 import build
    build.build_library()
    return tc.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "tc.h")).read()
    declared = set(re.findall(r"\b(tc_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(tc.binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_no_device_means_error_not_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(tc.TcError):
        tc.tc_create(0)


def test_host_huffman_matches_oracle_lengths(lib):
    rng = np.random.default_rng(3)
    for _ in range(200):
        n = 1 << int(rng.integers(1, 9))
        counts = (rng.integers(0, 12, n) ** int(rng.integers(1, 8))).astype(np.uint64)
        for lmax in (12, max(8, int(np.log2(n)))):
            assert np.array_equal(tc.tc_host_huffman_lengths(counts, lmax), oracle.huffman_lengths(counts, lmax)[0])


def test_host_huffman_rejects_bad_arguments(lib):
    with pytest.raises(tc.TcError):
        tc.tc_host_huffman_lengths(np.zeros(256, dtype=np.uint64), 7)     # 2^7 < 256 symbols


@pytest.mark.parametrize("n", [1, 2, 17, 96, 256])
def test_host_eigh_against_numpy(lib, n):
    rng = np.random.default_rng(n)
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    lam = 0.9 ** np.arange(n)
    a = (q * lam) @ q.T
    a = (a + a.T) / 2
    ev, vt = tc.tc_host_eigh(a)
    assert np.allclose(ev, np.sort(np.linalg.eigvalsh(a))[::-1], rtol=0, atol=1e-13)
    assert np.all(np.diff(ev) <= 0)
    assert np.allclose(vt @ vt.T, np.eye(n), atol=1e-12)
    assert np.allclose(vt @ a @ vt.T, np.diag(ev), atol=1e-13)
    for row in vt:
        assert row[np.argmax(np.abs(row))] > 0


def test_host_eigh_repeated_eigenvalues(lib):
    ev, vt = tc.tc_host_eigh(np.diag([2.0, 2.0, 1.0, 2.0]))
    assert np.allclose(ev, [2, 2, 2, 1])
    assert np.allclose(vt @ vt.T, np.eye(4), atol=1e-14)
