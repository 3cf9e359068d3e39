"""tc_encode_many / tc_decode_many (Section 3.1: every layer has its own encoder and decoder):
the sixteen-layer set of the ResNet-34 configuration plus an fp32 map, a layer on the streaming
kernels and an empty tensor in one call each -- every item equal to the per-tensor entry points
byte for byte, and checked against the oracle's coder and reconstruction."""
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


def _layer_set(ctx):
    """(model, codebook, x, oracle side, dtype) per item: cfg 3's shapes with their multiplicities (two
    images per item), one fp32 map (exact kernels, symbols parked in the arena) and an empty tensor."""
    w = fm.workload(3)
    items = []
    for spec, mult in zip(w.layers, w.repeats):
        o = H.oracle_side(spec, 4, 6, 2 * mult, torch.bfloat16, False)
        model = H.import_model(tc, ctx, o["model"], torch.bfloat16)
        cb = tc.tc_codebook_import(ctx, o["lengths"], 4)
        x = o["x"].cuda()
        for j in range(mult):
            items.append((model, cb, x[2 * j: 2 * j + 2].contiguous(), o, torch.bfloat16, slice(2 * j, 2 * j + 2)))
    o = H.oracle_side(fm.LayerSpec(48, 12, 12, 0.9, None, 8800), 6, 6, 3, torch.float32, True)
    model = H.import_model(tc, ctx, o["model"], torch.float32)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 6)
    items.append((model, cb, o["x"].cuda(), o, torch.float32, slice(0, 3)))
    items.append((model, cb, o["x"].cuda()[:0].contiguous(), o, torch.float32, slice(0, 0)))
    return items


def test_many_equals_the_per_tensor_calls_and_the_oracle(ctx):
    w = fm.workload(3)
    assert sum(w.repeats) == 16
    items = _layer_set(ctx)
    encs = tc.tc_encode_many(ctx, [(m, cb, x) for m, cb, x, *_ in items])
    assert tc.tc_get_status(ctx) == 0
    outs = tc.tc_decode_many(ctx, [(m, cb, e, x.shape, x.dtype) for (m, cb, x, *_), e in zip(items, encs)])
    assert tc.tc_get_status(ctx) == 0
    routes = set()
    for (model, cb, x, o, dtype, sl), enc, xhat in zip(items, encs, outs):
        if x.shape[0] == 0:
            assert enc.total_bits() == 0
            continue
        alone = tc.tc_encode(ctx, model, cb, x, debug=True, k=o["model"].k)
        routes.add(tc.tc_last_path(ctx))
        assert enc.total_bits() == alone.total_bits()
        assert np.array_equal(H.stream_words(enc), H.stream_words(alone))
        assert np.array_equal(H.chunk_len(enc), H.chunk_len(alone)) and np.array_equal(H.tile_off(enc), H.tile_off(alone))
        xhat_alone = tc.tc_decode(ctx, model, cb, alone, x.shape, dtype)
        assert torch.equal(xhat, xhat_alone)
        # against the oracle: symbols within the tie allowance, its coder bit for bit on those symbols,
        # its reconstruction within the output tolerance
        pix = x.shape[2] * x.shape[3]
        rows = slice(sl.start * pix, sl.stop * pix)
        q_gpu = alone.symbols.cpu().numpy()
        bad = q_gpu != o["q"][rows]
        assert bad.mean() <= 1e-4
        ref = oracle.encode(q_gpu, o["lengths"], o["model"].bits, chunk_pixels=enc.layout.chunk_pixels,
                            pixel_splits=enc.layout.pixel_splits, tile_pixels=128)
        assert enc.total_bits() == ref.total_bits and np.array_equal(H.stream_words(enc), ref.words)
        assert np.array_equal(H.chunk_len(enc), ref.chunk_len) and np.array_equal(H.tile_off(enc), ref.tile_off)
        want = oracle.reconstruct(o["model"], q_gpu, x.shape, out_bf16=(dtype == torch.bfloat16))
        got = xhat.float().cpu().numpy()
        if dtype == torch.float32:
            assert np.array_equal(got, want)
        else:
            ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
            assert np.all(np.abs(got - want) <= np.maximum(1e-3 * np.maximum(np.abs(want), o["model"].step), ulp))
            assert H.count_output_flips(got, want) <= H.flip_allowance(H.expected_output_flips(o["model"], q_gpu))
    assert routes == {0, 1, 3}          # exact kernels, resident-basis and streaming tensor-core kernels all took part


def test_many_reuses_buffers_and_rejects_a_bad_item_before_launching(ctx):
    items = _layer_set(ctx)[:5]
    layers = [(m, cb, x) for m, cb, x, *_ in items]
    first = tc.tc_encode_many(ctx, layers)
    want = [H.stream_words(e).copy() for e in first]
    for e in first:
        e.words.fill_(0x5A)
    again = tc.tc_encode_many(ctx, layers, outs=first)
    assert tc.tc_get_status(ctx) == 0
    for e, w_ in zip(again, want):
        assert np.array_equal(H.stream_words(e), w_)
    # a misaligned stream buffer in the last item: refused, and the buffers of the others stay as they were
    for e in first:
        e.words.fill_(0x33)
    last = first[-1]
    skewed = tc.EncodedStream(last.words[8:], last.chunk_len, last.tile_off, last.layout)
    with pytest.raises(tc.TcError):
        tc.tc_encode_many(ctx, layers, outs=first[:-1] + [skewed])
    torch.cuda.synchronize()
    assert all(bool((e.words == 0x33).all()) for e in first)
