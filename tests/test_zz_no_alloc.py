"""tc_encode_noalloc -- the encode entry point for callers that may not allocate device memory
(a server with a memory budget fixed at start-up, a pipeline that cannot take cudaMalloc's
device-wide stall, a plug-in whose host owns the allocator) -- must write exactly what tc_encode
writes.  Its look-back state sits in a fixed array inside the library that every call reuses,
so the check is made on two calls in a row: the second one meets the first one's leftovers.

This file sorts after every other test file on purpose: a run that stops at the first failure
has then already run all the others."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10830_b200 as tc
from synth import featuremaps as fm
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _fresh_buffers(ref: tc.EncodedStream) -> tc.EncodedStream:
    # same sizes as the reference run, pre-filled with a pattern so that stale bytes show
    return tc.EncodedStream(torch.full_like(ref.words, 0x5A), torch.full_like(ref.chunk_len, -1),
                            torch.full_like(ref.tile_off, -1), ref.layout)


@pytest.mark.parametrize("dtype,c,s,n,bits,route", [
    (torch.bfloat16, 64, 28, 9, 4, 1),      # tensor-core kernels, basis resident in shared memory, 56 tiles
    (torch.float32, 32, 14, 7, 6, 0),       # fp64 kernels, 11 tiles
    (torch.bfloat16, 320, 7, 21, 5, 3),     # tensor-core kernels that stream the basis: 7x7 maps, 9 tiles
    (torch.bfloat16, 576, 14, 3, 5, 3),     # the same above 512 channels, four chunks per pixel
    (torch.bfloat16, 24, 9, 5, 4, 2)])      # fp32 kernels (channel count not a multiple of 16)
def test_noalloc_encode_matches_tc_encode_twice_in_a_row(dtype, c, s, n, bits, route):
    ctx = tc.tc_create(0)
    spec = fm.LayerSpec(c, s, s, 0.9, None, 9100 + c)
    o = H.oracle_side(spec, bits, max(6, (2 * c) // (s * s) + 1), n, dtype, False)
    model = H.import_model(tc, ctx, o["model"], dtype)
    cb = tc.tc_codebook_import(ctx, o["lengths"], bits)
    x = o["x"].cuda()
    ref = tc.tc_encode(ctx, model, cb, x, debug=True)
    assert tc.tc_get_status(ctx) == 0
    assert tc.tc_last_path(ctx) == route
    nbytes = ref.total_bits() // 8
    # a different tensor in between leaves other tile states behind in the shared array
    other = torch.flip(x, dims=[0, 2]).contiguous()
    for attempt in range(2):
        out = tc.tc_encode_noalloc(ctx, model, cb, x, _fresh_buffers(ref))
        assert tc.tc_get_status(ctx) == 0
        assert tc.tc_last_path(ctx) == route, "the entry point that allocates nothing picked other kernels than tc_encode"
        assert torch.equal(out.tile_off, ref.tile_off), f"tile offsets differ on call {attempt + 1}"
        assert torch.equal(out.chunk_len[: ref.layout.n_chunks], ref.chunk_len[: ref.layout.n_chunks])
        assert torch.equal(out.words[:nbytes], ref.words[:nbytes]), f"stream differs on call {attempt + 1}"
        if attempt == 0:
            tc.tc_encode_noalloc(ctx, model, cb, other, _fresh_buffers(ref))
            assert tc.tc_get_status(ctx) == 0
    # the stream is the oracle's coding of the symbols the kernels produced
    want = oracle.encode(ref.symbols.cpu().numpy(), o["lengths"], bits, chunk_pixels=ref.layout.chunk_pixels,
                         pixel_splits=ref.layout.pixel_splits, tile_pixels=128)
    assert np.array_equal(out.words[:nbytes].cpu().numpy().view(np.uint32), want.words)
    assert np.array_equal(out.chunk_len[: ref.layout.n_chunks].cpu().numpy().view(np.uint16), want.chunk_len)
    # and the stream it wrote decodes to what the reference stream decodes to
    a = tc.tc_decode(ctx, model, cb, out, x.shape, dtype)
    b = tc.tc_decode(ctx, model, cb, ref, x.shape, dtype)
    assert tc.tc_get_status(ctx) == 0
    assert torch.equal(a, b)
    for h in (model, cb, ctx):
        h.close()


def test_noalloc_encode_refuses_tensors_beyond_its_fixed_scratch():
    ctx = tc.tc_create(0)
    spec = fm.LayerSpec(16, 8, 8, 0.9, None, 9200)
    o = H.oracle_side(spec, 3, 4, 1, torch.bfloat16, False)
    model = H.import_model(tc, ctx, o["model"], torch.bfloat16)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 3)
    # 65 537 tiles of 128 pixels: one more than the fixed array holds
    big = torch.zeros(1, 16, 4097, 2048, dtype=torch.bfloat16, device="cuda")
    lay = tc.tc_encode_bound(model, cb, big)
    assert lay.n_tiles > 65536
    bufs = tc.EncodedStream(torch.empty(1024, dtype=torch.uint8, device="cuda"),
                            torch.empty(lay.n_chunks, dtype=torch.int32, device="cuda"),
                            torch.empty(lay.n_tiles + 1, dtype=torch.int64, device="cuda"), lay)
    with pytest.raises(tc.TcError) as err:
        tc.tc_encode_noalloc(ctx, model, cb, big, bufs)
    assert err.value.code == 2                      # TC_ERR_UNSUPPORTED, nothing launched
    assert tc.tc_get_status(ctx) == 0
    for h in (model, cb, ctx):
        h.close()
