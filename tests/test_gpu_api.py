"""GPU tests of the library's other entry points and of its error behaviour: fit, statistics,
codebook building, capacity overflow and corrupt streams (all made on the host; nothing here
traps or hangs the device)."""
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
def test_fit_pca_invariants_and_agreement_with_oracle(ctx, dtype):
    spec = fm.LayerSpec(48, 14, 14, 0.85, None, 501)
    p = fm.layer_params(spec)
    cal = fm.make_maps(p, 16, calib=True, dtype=dtype)
    m = tc.tc_fit_pca(ctx, cal.cuda(), bits=6)
    e = tc.tc_model_export(m)
    ref = oracle.fit_pca(cal, 6, basis_round=H.basis_round_for(dtype), zero_level=True)
    t = e["basis"]
    rt = 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -23
    assert np.abs(t @ t.T - np.eye(48)).max() < 48 * rt
    _, cov = oracle.mean_cov(cal)
    d = t @ cov @ t.T
    assert np.abs(d - np.diag(np.diag(d))).max() < 10 * rt * np.abs(cov).max()
    assert np.allclose(e["eig"], ref.eig, rtol=1e-9, atol=1e-12 * ref.eig[0])
    assert np.allclose(e["mean"], ref.mean, rtol=1e-12, atol=1e-14)
    lead = ref.eig > 1e-3 * ref.eig[0]
    gaps_ok = np.abs(np.diff(ref.eig))[: lead.sum() - 1] > 1e-3 * ref.eig[0]
    for j in np.nonzero(lead)[0][:-1]:
        if gaps_ok[max(j - 1, 0)] and gaps_ok[j]:
            cos = abs(t[j] @ ref.basis[j]) / (np.linalg.norm(t[j]) * np.linalg.norm(ref.basis[j]))
            assert cos > 1 - 1e-4
    assert e["lo"] == pytest.approx(ref.lo, rel=2e-2, abs=1e-3)
    assert e["step"] == pytest.approx(ref.step, rel=2e-2)
    # end to end: rate and distortion within 1 % of the oracle's fit
    x = fm.make_maps(p, 4, dtype=dtype)
    st = tc.tc_stats(ctx, m, None, x.cuda())
    q_ref = oracle.quantize(ref, oracle.project(ref, x))
    h_ref = oracle.entropy(oracle.histogram(q_ref, 6, False)[0])
    mse_ref = oracle.mse(x, oracle.reconstruct(ref, q_ref, x.shape, out_bf16=(dtype == torch.bfloat16)))
    assert st.entropy == pytest.approx(h_ref, rel=0.01)
    assert st.mse == pytest.approx(mse_ref, rel=0.02)
    m.close()


@pytest.mark.parametrize("per_channel", [False, True])
def test_stats_and_build_codebook_match_oracle(ctx, per_channel):
    spec = fm.LayerSpec(32, 14, 14, 0.85, None, 502)
    o = H.oracle_side(spec, 5, 8, 4, torch.float32, per_channel)
    m = H.import_model(tc, ctx, o["model"], torch.float32)
    groups = 32 if per_channel else 1
    st = tc.tc_stats(ctx, m, None, o["cal"].cuda(), groups=groups)
    hist_ref = oracle.histogram(o["q_cal"], 5, per_channel)
    assert np.array_equal(st.hist.cpu().numpy().view(np.uint64), hist_ref)
    want_h = np.mean([oracle.entropy(hist_ref[g]) for g in range(groups)])
    assert st.entropy == pytest.approx(want_h, rel=1e-12)
    cb = tc.tc_build_codebook(ctx, m, st.hist, groups=groups)
    assert np.array_equal(tc.tc_codebook_export(cb), o["lengths"])
    cb_host = tc.tc_build_codebook(ctx, m, hist_ref, groups=groups)
    assert np.array_equal(tc.tc_codebook_export(cb_host), o["lengths"])
    st2 = tc.tc_stats(ctx, m, cb, o["x"].cuda(), groups=groups)
    q = o["q"]
    lens = np.stack([o["lengths"][j if per_channel else 0][q[:, j]] for j in range(32)], axis=1)
    assert st2.mean_length == pytest.approx(lens.mean(), rel=1e-12)
    xhat = oracle.reconstruct(o["model"], q, o["x"].shape, out_bf16=False)
    assert st2.mse == pytest.approx(oracle.mse(o["x"], xhat), rel=1e-9)
    assert st2.zero_fraction == pytest.approx(float((o["x"] == 0).double().mean()), abs=1e-12)
    top = (1 << 5) - 1
    assert st2.clamped_fraction == pytest.approx(float(((o["units"] < 0) | (o["units"] > top)).mean()), abs=1e-12)
    for h in (m, cb, cb_host):
        h.close()


def test_model_export_round_trip_and_rejects_unrepresentable_basis(ctx):
    spec = fm.LayerSpec(16, 8, 8, 0.85, None, 503)
    o = H.oracle_side(spec, 4, 4, 1, torch.bfloat16, False)
    m = H.import_model(tc, ctx, o["model"], torch.bfloat16)
    e = tc.tc_model_export(m)
    assert np.array_equal(e["basis"], o["model"].basis) and np.array_equal(e["mean"], o["model"].mean)
    assert e["lo"] == o["model"].lo and e["step"] == o["model"].step and e["bits"] == 4
    m.close()
    full = oracle.fit_pca(o["cal"], 4)                      # fp64 basis: not bf16-exact
    with pytest.raises(tc.TcError) as err:
        H.import_model(tc, ctx, full, torch.bfloat16)
    assert err.value.code == 1


def test_argument_errors(ctx):
    spec = fm.LayerSpec(16, 8, 8, 0.85, None, 504)
    o = H.oracle_side(spec, 4, 4, 1, torch.float32, False)
    m = H.import_model(tc, ctx, o["model"], torch.float32)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 4)
    x = o["x"].cuda()
    with pytest.raises(tc.TcError) as err:                   # wrong channel count
        tc.tc_encode(ctx, m, cb, torch.zeros(1, 8, 8, 8, device="cuda"))
    assert err.value.code == 1
    with pytest.raises(tc.TcError) as err:                   # dtype does not match the basis
        tc.tc_encode(ctx, m, cb, x.bfloat16())
    assert err.value.code == 2
    with pytest.raises(tc.TcError):                          # chunk size not a power of two
        tc.tc_encode(ctx, m, cb, x, chunk_pixels=3)
    with pytest.raises(tc.TcError):                          # a pixel is split only when a chunk is one pixel
        tc.tc_encode(ctx, m, cb, x, chunk_pixels=2, pixel_splits=2)
    with pytest.raises(tc.TcError):                          # 16 coefficients do not split in four runs of 8
        tc.tc_encode(ctx, m, cb, x, chunk_pixels=1, pixel_splits=4)
    with pytest.raises(tc.TcError):                          # three splits
        tc.tc_encode(ctx, m, cb, x, chunk_pixels=1, pixel_splits=3)
    bad = o["lengths"].copy()
    bad[0, 0] += 1                                           # breaks Kraft's equality
    with pytest.raises(tc.TcError):
        tc.tc_codebook_import(ctx, bad, 4)
    # empty batch
    enc = tc.tc_encode(ctx, m, cb, torch.zeros(0, 16, 8, 8, device="cuda"))
    assert enc.total_bits() == 0
    m.close(); cb.close()


def test_capacity_overflow_is_reported_and_in_bounds(ctx):
    spec = fm.LayerSpec(32, 16, 16, 0.85, None, 505)
    o = H.oracle_side(spec, 6, 4, 2, torch.float32, False)
    m = H.import_model(tc, ctx, o["model"], torch.float32)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 6)
    x = o["x"].cuda()
    full = tc.tc_encode(ctx, m, cb, x)
    assert tc.tc_get_status(ctx) == 0
    need = full.total_bits() // 8
    lay = full.layout
    guard = 4096
    buf = torch.full((need + guard,), 0xAB, dtype=torch.uint8, device="cuda")
    small = tc.EncodedStream(buf, torch.empty(lay.n_chunks, dtype=torch.int32, device="cuda"),
                             torch.empty(lay.n_tiles + 1, dtype=torch.int64, device="cuda"), lay)
    cap = (need // 2) & ~15
    tc.tc_encode(ctx, m, cb, x, out=small, capacity=cap)
    assert tc.tc_get_status(ctx) == 3                          # TC_ERR_BUFFER_TOO_SMALL
    assert tc.tc_get_status(ctx) == 0                          # cleared
    assert bool((buf[cap:] == 0xAB).all())                     # nothing written past the capacity
    # exact capacity works
    tc.tc_encode(ctx, m, cb, x, out=small, capacity=need)
    assert tc.tc_get_status(ctx) == 0
    assert torch.equal(buf[:need], full.words[:need])
    assert bool((buf[need:] == 0xAB).all())
    m.close(); cb.close()


def test_corrupt_streams_are_reported_without_faults(ctx):
    spec = fm.LayerSpec(32, 16, 16, 0.85, None, 506)
    o = H.oracle_side(spec, 6, 4, 2, torch.float32, False)
    m = H.import_model(tc, ctx, o["model"], torch.float32)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 6)
    x = o["x"].cuda()
    enc = tc.tc_encode(ctx, m, cb, x)
    assert tc.tc_get_status(ctx) == 0
    nbytes = enc.total_bits() // 8
    # (a) truncated stream
    tc.tc_decode(ctx, m, cb, enc, x.shape, x.dtype, stream_bytes=(nbytes // 2) & ~15)
    assert tc.tc_get_status(ctx) == 5
    # (b) tile offset beyond the stream / not aligned / decreasing
    for bad_value in (nbytes * 8 + 128, 64, -128):
        broken = tc.EncodedStream(enc.words, enc.chunk_len, enc.tile_off.clone(), enc.layout)
        broken.tile_off[1] = broken.tile_off[1] + bad_value if bad_value != 64 else 64
        tc.tc_decode(ctx, m, cb, broken, x.shape, x.dtype, stream_bytes=nbytes)
        assert tc.tc_get_status(ctx) == 5
    # (c) a chunk length that runs past its tile, and one that is off by a single bit
    for delta in (30000, 1, -1):
        broken = tc.EncodedStream(enc.words, enc.chunk_len.clone(), enc.tile_off, enc.layout)
        broken.chunk_len[3] += delta
        tc.tc_decode(ctx, m, cb, broken, x.shape, x.dtype, stream_bytes=nbytes)
        assert tc.tc_get_status(ctx) == 5
    # (d) flipped payload bits: must stay in bounds; either decodes to other symbols or reports
    noisy = tc.EncodedStream(enc.words.clone(), enc.chunk_len, enc.tile_off, enc.layout)
    g = torch.Generator(device="cuda").manual_seed(1)
    idx = torch.randint(0, nbytes, (64,), generator=g, device="cuda")
    noisy.words[idx] ^= 0x5A
    out = tc.tc_decode(ctx, m, cb, noisy, x.shape, x.dtype, stream_bytes=nbytes)
    assert tc.tc_get_status(ctx) in (0, 5)
    assert out.shape == x.shape
    # the intact stream still decodes afterwards
    good = tc.tc_decode(ctx, m, cb, enc, x.shape, x.dtype, stream_bytes=nbytes)
    assert tc.tc_get_status(ctx) == 0
    want = oracle.reconstruct(o["model"], o["q"], x.shape, out_bf16=False)
    assert np.array_equal(good.cpu().numpy(), want)
    m.close(); cb.close()


def test_repeated_encodes_are_bit_identical(ctx):
    # the look-back makes the layout deterministic: every run writes the same bytes
    spec = fm.LayerSpec(64, 28, 28, 0.9, None, 507)
    o = H.oracle_side(spec, 4, 4, 8, torch.bfloat16, False)
    m = H.import_model(tc, ctx, o["model"], torch.bfloat16)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 4)
    x = o["x"].cuda()
    first = tc.tc_encode(ctx, m, cb, x)
    n = first.total_bits() // 8
    for _ in range(3):
        again = tc.tc_encode(ctx, m, cb, x)
        assert tc.tc_get_status(ctx) == 0
        assert again.total_bits() == first.total_bits()
        assert torch.equal(again.words[:n], first.words[:n])
        assert torch.equal(again.tile_off, first.tile_off)
    m.close(); cb.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_roundtrip_host_matches_the_device_path(ctx, dtype):
    spec = fm.LayerSpec(64, 14, 14, 0.9, None, 508)
    o = H.oracle_side(spec, 4, 6, 5, dtype, False)
    m = H.import_model(tc, ctx, o["model"], dtype)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 4)
    x = o["x"]
    host_in = x.clone().pin_memory()
    host_out = torch.empty_like(host_in).pin_memory()
    bits = tc.tc_roundtrip_host(ctx, m, cb, host_in, host_out)
    enc = tc.tc_encode(ctx, m, cb, x.cuda())
    dev = tc.tc_decode(ctx, m, cb, enc, x.shape, dtype)
    assert tc.tc_get_status(ctx) == 0
    assert bits == enc.total_bits()
    assert torch.equal(host_out, dev.cpu())
    m.close(); cb.close()


def test_roundtrip_host_in_several_chunks_matches_one_device_pass(ctx):
    # 150 maps of 64x56x56 bf16 are 60 MB: the call works through them in two chunks of whole
    # tiles, two in flight; reconstruction and stream length must equal those of one device pass
    params = fm.layer_params(fm.LayerSpec(64, 56, 56, 0.9, None, 509))
    cal = fm.make_maps(params, 8, calib=True, dtype=torch.bfloat16, device="cuda")
    x = fm.make_maps(params, 150, dtype=torch.bfloat16, device="cuda")
    model = tc.tc_fit_pca(ctx, cal, 4)
    st = tc.tc_stats(ctx, model, None, cal)
    cb = tc.tc_build_codebook(ctx, model, st.hist)
    host_in = x.cpu().pin_memory()
    host_out = torch.empty_like(host_in).pin_memory()
    for _ in range(2):                                         # the second call reuses slots, streams and events
        host_out.zero_()
        bits = tc.tc_roundtrip_host(ctx, model, cb, host_in, host_out)
        enc = tc.tc_encode(ctx, model, cb, x)
        dev = tc.tc_decode(ctx, model, cb, enc, x.shape, torch.bfloat16)
        assert tc.tc_get_status(ctx) == 0
        assert bits == enc.total_bits()
        assert torch.equal(host_out, dev.cpu())
    model.close(); cb.close()


# ---- the same robustness checks on the tensor-core routes (1: basis resident, 3: basis streamed) ----

@pytest.mark.parametrize("c,s,n,route", [(64, 16, 3, 1), (320, 8, 5, 3), (576, 7, 6, 3)])
def test_tensor_core_routes_overflow_corruption_and_repeatability(ctx, c, s, n, route):
    spec = fm.LayerSpec(c, s, s, 0.9, None, 520 + c)
    o = H.oracle_side(spec, 5, max(4, (2 * c) // (s * s) + 1), n, torch.bfloat16, False)
    m = H.import_model(tc, ctx, o["model"], torch.bfloat16)
    cb = tc.tc_codebook_import(ctx, o["lengths"], 5)
    x = o["x"].cuda()
    enc = tc.tc_encode(ctx, m, cb, x)
    assert tc.tc_get_status(ctx) == 0 and tc.tc_last_path(ctx) == route
    nbytes = enc.total_bits() // 8
    lay = enc.layout
    ref = tc.tc_decode(ctx, m, cb, enc, x.shape, x.dtype, stream_bytes=nbytes)
    assert tc.tc_get_status(ctx) == 0 and tc.tc_last_path(ctx, True) == route
    # repeated encodes write the same bytes
    again = tc.tc_encode(ctx, m, cb, x)
    assert torch.equal(again.words[:nbytes], enc.words[:nbytes]) and torch.equal(again.tile_off, enc.tile_off)
    assert torch.equal(again.chunk_len[:lay.n_chunks], enc.chunk_len[:lay.n_chunks])
    # capacity overflow: reported, nothing written past the capacity; exact capacity works
    guard = 4096
    buf = torch.full((nbytes + guard,), 0xAB, dtype=torch.uint8, device="cuda")
    small = tc.EncodedStream(buf, torch.empty(lay.n_chunks + (lay.n_chunks & 1), dtype=torch.int16, device="cuda"),
                             torch.empty(lay.n_tiles + 1, dtype=torch.int64, device="cuda"), lay)
    cap = (nbytes // 2) & ~15
    tc.tc_encode(ctx, m, cb, x, out=small, capacity=cap)
    assert tc.tc_get_status(ctx) == 3
    assert bool((buf[cap:] == 0xAB).all())
    tc.tc_encode(ctx, m, cb, x, out=small, capacity=nbytes)
    assert tc.tc_get_status(ctx) == 0
    assert torch.equal(buf[:nbytes], enc.words[:nbytes]) and bool((buf[nbytes:] == 0xAB).all())
    # corrupt streams (made on the host): reported, never a fault
    tc.tc_decode(ctx, m, cb, enc, x.shape, x.dtype, stream_bytes=(nbytes // 2) & ~15)
    assert tc.tc_get_status(ctx) == 5
    for bad_value in (nbytes * 8 + 128, 64, -128):
        broken = tc.EncodedStream(enc.words, enc.chunk_len, enc.tile_off.clone(), lay)
        broken.tile_off[1] = broken.tile_off[1] + bad_value if bad_value != 64 else 64
        tc.tc_decode(ctx, m, cb, broken, x.shape, x.dtype, stream_bytes=nbytes)
        assert tc.tc_get_status(ctx) == 5
    for delta in (30000, 1, -1):
        broken = tc.EncodedStream(enc.words, enc.chunk_len.clone(), enc.tile_off, lay)
        broken.chunk_len[3] += delta
        tc.tc_decode(ctx, m, cb, broken, x.shape, x.dtype, stream_bytes=nbytes)
        assert tc.tc_get_status(ctx) == 5
    noisy = tc.EncodedStream(enc.words.clone(), enc.chunk_len, enc.tile_off, lay)
    g = torch.Generator(device="cuda").manual_seed(2)
    idx = torch.randint(0, nbytes, (64,), generator=g, device="cuda")
    noisy.words[idx] ^= 0x5A
    out = tc.tc_decode(ctx, m, cb, noisy, x.shape, x.dtype, stream_bytes=nbytes)
    assert tc.tc_get_status(ctx) in (0, 5) and out.shape == x.shape
    # the intact stream still decodes to the same tensor afterwards
    good = tc.tc_decode(ctx, m, cb, enc, x.shape, x.dtype, stream_bytes=nbytes)
    assert tc.tc_get_status(ctx) == 0 and torch.equal(good, ref)
    m.close(); cb.close()


@pytest.mark.parametrize("c,s,n,bits,with_cb", [(64, 14, 1400, 4, False), (256, 14, 9, 5, True), (96, 28, 3, 8, True)])
def test_stats_on_the_tensor_core_kernels(ctx, c, s, n, bits, with_cb):
    # bf16 tensors of up to 256 channels: the encoder counts the symbols while it codes (Section 3.1,
    # "Variable length coding": the entropy needs their distribution); 1400 maps of 64 x 14 x 14 are
    # more than one chunk of the batch
    spec = fm.LayerSpec(c, s, s, 0.9, None, 520 + c)
    o = H.oracle_side(spec, bits, 8, n, torch.bfloat16, False)
    m = H.import_model(tc, ctx, o["model"], torch.bfloat16)
    cb = tc.tc_codebook_import(ctx, o["lengths"], bits) if with_cb else None
    x = o["x"].cuda()
    st = tc.tc_stats(ctx, m, cb, x, groups=c)
    assert tc.tc_get_status(ctx) == 0
    hist = st.hist.cpu().numpy().view(np.uint64)
    # exactly the histogram of the symbols the encoder produces ...
    cb_any = cb if cb is not None else tc.tc_codebook_import(ctx, o["lengths"], bits)
    enc = tc.tc_encode(ctx, m, cb_any, x, debug=True)
    assert tc.tc_last_path(ctx) == 1
    q_gpu = enc.symbols.cpu().numpy()
    assert np.array_equal(hist, oracle.histogram(q_gpu, bits, True))
    # ... which is the oracle's own up to the symbols that may differ at rounding ties
    ref = oracle.histogram(o["q"], bits, True)
    assert np.abs(hist.astype(np.int64) - ref.astype(np.int64)).sum() <= 2 * np.ceil(1e-4 * o["q"].size)
    assert hist.sum() == o["q"].size
    want_h = np.mean([oracle.entropy(hist[g]) for g in range(c)])
    assert st.entropy == pytest.approx(want_h, rel=1e-12)
    if with_cb:
        assert st.mean_length == pytest.approx(o["lengths"][0][q_gpu].mean(), rel=1e-12)
    xhat = oracle.reconstruct(o["model"], q_gpu, tuple(x.shape), out_bf16=True)
    assert st.mse == pytest.approx(oracle.mse(o["x"], xhat), rel=2e-3)
    assert st.zero_fraction == pytest.approx(float((o["x"] == 0).double().mean()), abs=1e-12)
    top = (1 << bits) - 1
    assert st.clamped_fraction == pytest.approx(float(((o["units"] < 0) | (o["units"] > top)).mean()), abs=1e-4)
    # folded to one table: the sum over the channels
    st1 = tc.tc_stats(ctx, m, cb, x, groups=1)
    assert np.array_equal(st1.hist.cpu().numpy().view(np.uint64)[0], hist.sum(axis=0))
    for h in (m, cb, cb_any):
        if h is not None:
            h.close()
