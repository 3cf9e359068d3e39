"""Random shapes through the parity checks of test_gpu_parity.run_case: channel counts up to
1024, map sizes from 1 x 1 to 28 x 28, truncation, every bit width, per-layer and per-channel
codebooks, every chunk shape, on the default route and with the resident-basis kernels switched
off.  Seeds are fixed, so the cases are the same in every run; each case also checks that the
library picked the kernels its shape calls for."""
import random

import pytest
import torch

import paper_1905_10830_b200 as tc
from synth import featuremaps as fm
from tests.test_gpu_parity import run_case

pytestmark = pytest.mark.gpu

CASES_PER_SEED = 24


def _draw(rng: random.Random, it: int):
    c = 16 * rng.randint(1, 64 if rng.random() < 0.3 else 20)
    s = rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 12, 14, 16, 20, 28])
    k = c if rng.random() < 0.6 else 16 * rng.randint(1, c // 16)
    bits = rng.randint(2, 8)
    per_channel = rng.random() < 0.25 and c <= 256
    n = max(1, min(6, 600 // (s * s)))
    splits = rng.choice([0, 0, 1, 2, 4])
    if splits > 1 and k % (16 * splits) != 0:
        splits = 0
    cp = 1 if splits else rng.choice([0, 0, 1, 2, 8])
    mode = rng.choice([0, 0, 2])
    ratio = rng.choice([0.85, 0.9, 0.95])
    return dict(c=c, s=s, k=k, bits=bits, per_channel=per_channel, n=n, splits=splits, cp=cp, mode=mode, ratio=ratio, it=it)


def _expected_routes(d, layout):
    """Kernels the shape calls for: (encode, decode).  1 = tensor-core kernels with the basis
    resident in shared memory, 3 = tensor-core kernels that stream the basis.  Every shape drawn
    here has channel and coefficient counts that are multiples of 16, so no case may fall back to
    the fp32 kernels."""
    c, k, hw, mode = d["c"], d["k"], d["s"] * d["s"], d["mode"]
    cp, splits = layout.chunk_pixels, layout.pixel_splits
    enc_resident = mode == 0 and c <= 256 and hw % 4 == 0 and \
        (splits == 1 or (splits == 2 and k % 32 == 0) or (splits == 4 and k % 64 == 0))
    enc = 1 if enc_resident else 3
    if mode == 2 or c > 256 or (splits == 4 and d["per_channel"]):
        dec = 3
    else:
        dec = (1, 3)          # the resident-basis decoder where its shared-memory plan fits, else the streaming one
    return enc, dec


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4])
def test_random_shapes_against_the_oracle(seed):
    rng = random.Random(1905_10830 + seed)
    ctx = tc.tc_create(0)
    done = 0
    for it in range(CASES_PER_SEED):
        d = _draw(rng, it)
        tc.tc_force_exact_path(ctx, d["mode"])
        spec = fm.LayerSpec(d["c"], d["s"], d["s"], d["ratio"], None, 9000 + 100 * seed + it)
        n_cal = max(4, (2 * d["c"]) // (d["s"] * d["s"]) + 1)
        # the chunk shape the library will use (host-side query on a throw-away model of the same shape)
        probe = torch.zeros(d["n"], d["c"], d["s"], d["s"], dtype=torch.bfloat16, device="cuda")
        try:
            lay = _probe_layout(ctx, d, probe)
        except tc.TcError:
            continue                                       # a chunk shape the format cannot hold
        routes = _expected_routes(d, lay)
        try:
            run_case(ctx, spec, d["bits"], n_cal, d["n"], torch.bfloat16, d["per_channel"], exact=False,
                     chunk_pixels=d["cp"], pixel_splits=d["splits"], k=d["k"], routes=routes)
        except tc.TcError as e:
            if e.code == 1:                                # invalid argument: with this codebook a chunk would exceed 65535 bits
                continue
            raise
        except AssertionError as e:
            raise AssertionError(f"case {d}: {e}") from e
        done += 1
    ctx.close()
    assert done >= CASES_PER_SEED // 2


def _probe_layout(ctx, d, probe):
    import numpy as np
    c, k, bits = d["c"], d["k"], d["bits"]
    model = tc.tc_model_import(ctx, basis=np.eye(c), mean=np.zeros(c), lo=-1.0, step=2.0 / ((1 << bits) - 1), bits=bits,
                               basis_dtype=tc.binding.TC_BF16, k=k)
    lengths = np.full((k if d["per_channel"] else 1, 1 << bits), bits, dtype=np.uint8)
    cb = tc.tc_codebook_import(ctx, lengths, bits)
    try:
        return tc.tc_encode_bound(model, cb, probe, chunk_pixels=d["cp"], pixel_splits=d["splits"])
    finally:
        model.close()
        cb.close()
