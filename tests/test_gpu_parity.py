"""GPU parity: the CUDA library against the CPU oracle on identical seeded inputs, with the
oracle's model and codebook imported into the library (identical T, mu, lo, step, lengths).

Bars: the entropy-coded stream is bit-exact given identical symbols and decode round-trips
exactly; projected coefficients agree within 1e-3 * max(|y|, step); at most 1e-4 of the
symbols differ, only by +-1 and only where the oracle's position (y - lo)/step lies within
1e-3 of a half-integer; x_hat agrees within max(1e-3 * max(|x_hat|, step), one output ulp),
and the number of values that are not bit-identical stays within what the fp32 arithmetic of
the decoder explains (tests/helpers.py: expected_output_flips, flip_allowance)."""
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
    """Context pinned to the fp64 kernels: results must be identical to the oracle's."""
    c = tc.tc_create(0)
    tc.tc_force_exact_path(c, True)
    yield c
    c.close()


@pytest.fixture(scope="module")
def ctx_tc():
    """Context on the default route: bf16 tensors take the tensor-core kernels."""
    c = tc.tc_create(0)
    yield c
    c.close()


def check_symbols(q_gpu, o, *, exact: bool):
    q, units = o["q"], o["units"]
    diff = q_gpu.astype(np.int32) - q.astype(np.int32)
    bad = diff != 0
    if exact:
        assert not bad.any(), f"{bad.sum()} symbols differ on the exact path"
        return 0.0
    rate = bad.mean()
    # at most 1e-4 of the symbols; a tensor of fewer than 10 000 symbols may still have one (a tie is a tie)
    assert bad.sum() <= max(1, int(np.ceil(1e-4 * bad.size))), f"symbol mismatch rate {rate}"
    if bad.any():
        assert np.all(np.abs(diff[bad]) == 1)
        frac = np.abs(units[bad] - np.floor(units[bad]) - 0.5)
        assert np.all(frac <= 1e-3), f"mismatch away from a rounding tie: {frac.max()}"
    return rate


def check_stream_against_oracle(enc, q_gpu, lengths, bits):
    """Entropy-coding stage: bit-exact given identical symbol arrays."""
    ref = oracle.encode(q_gpu, lengths, bits, chunk_pixels=enc.layout.chunk_pixels,
                        pixel_splits=enc.layout.pixel_splits, tile_pixels=128)
    assert enc.total_bits() == ref.total_bits
    assert np.array_equal(H.tile_off(enc), ref.tile_off)
    assert enc.layout.n_chunks == ref.chunk_len.shape[0]
    assert np.array_equal(H.chunk_len(enc), ref.chunk_len)
    assert np.array_equal(H.stream_words(enc), ref.words)
    return ref


def _as_set(route):
    return route if isinstance(route, (set, frozenset, tuple, list)) else (route,)


def run_case(ctx, spec, bits, n_cal, n_test, dtype, per_channel, *, exact, chunk_pixels=0, pixel_splits=0, model=None,
             routes=None, k=None, basis_round=None):
    """`routes`: the kernels expected for (encode, decode): 0 fp64, 1 tensor core (basis resident
    in shared memory), 2 fp32, 3 tensor core (basis streamed: wide layers, unaligned rows)."""
    if routes is None:
        routes = (0, 0) if exact else (1, 1)
    o = H.oracle_side(spec, bits, n_cal, n_test, dtype, per_channel, model=model, k=k, basis_round=basis_round)
    m, lengths = o["model"], o["lengths"]
    model_h = H.import_model(tc, ctx, m, dtype)
    cb = tc.tc_codebook_import(ctx, lengths, bits)
    x = o["x"].cuda()
    enc = tc.tc_encode(ctx, model_h, cb, x, chunk_pixels=chunk_pixels, pixel_splits=pixel_splits, debug=True, k=m.k)
    assert tc.tc_get_status(ctx) == 0
    assert tc.tc_last_path(ctx) in _as_set(routes[0]), "unexpected kernel route"
    # coefficients
    y_gpu = enc.coefficients.cpu().numpy().astype(np.float64)
    tol = 1e-3 * np.maximum(np.abs(o["y"]), m.step)
    assert np.all(np.abs(y_gpu - o["y"]) <= tol)
    # symbols
    q_gpu = enc.symbols.cpu().numpy()
    check_symbols(q_gpu, o, exact=exact)
    # stream: bit-exact against the oracle's coder on the GPU's own symbols
    ref = check_stream_against_oracle(enc, q_gpu, lengths, bits)
    assert np.array_equal(oracle.decode_symbols(ref, lengths, bits), q_gpu)
    # decode: reconstruct what the stream holds
    xhat = tc.tc_decode(ctx, model_h, cb, enc, x.shape, dtype)
    assert tc.tc_get_status(ctx) == 0
    assert tc.tc_last_path(ctx, True) in _as_set(routes[1]), "unexpected kernel route"
    want = oracle.reconstruct(m, q_gpu, x.shape, out_bf16=(dtype == torch.bfloat16))
    got = xhat.float().cpu().numpy()
    if exact:
        assert np.array_equal(got, want)
    else:
        # fp32 accumulation may land on the other side of an output rounding boundary: allow one
        # unit in the last place of the output type there, and demand bit equality for 99.9 %
        mant = 7 if dtype == torch.bfloat16 else 23
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - mant)
        assert np.all(np.abs(got - want) <= np.maximum(1e-3 * np.maximum(np.abs(want), m.step), ulp))
        # how many values may land on the neighbouring output number follows from the fp32 arithmetic
        flips, expected = H.count_output_flips(got, want), H.expected_output_flips(m, q_gpu, out_bf16=(dtype == torch.bfloat16))
        assert flips <= H.flip_allowance(expected), f"{flips} values differ from the oracle's, {expected:.2f} expected"
        assert int((got != want).sum()) <= max(H.flip_allowance(expected), int(np.ceil(1e-3 * got.size)))   # and never more than 0.1 %
    model_h.close()
    cb.close()
    return o, enc


def test_cfg1_single_map_f32(ctx):
    w = fm.workload(1)
    run_case(ctx, w.layers[0], 8, w.calib_maps, 1, torch.float32, False, exact=True)


@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_cfg2_resnet18_layers_all_bit_widths_per_channel(ctx, layer):
    w = fm.workload(2)
    spec = w.layers[layer]
    base = None
    for bits in w.bits:
        o, _ = run_case(ctx, spec, bits, w.calib_maps, 1, torch.float32, True, exact=True, model=base)
        base = o["model"]


@pytest.mark.parametrize("c,s,n", [(64, 56, 1), (128, 28, 2), (256, 14, 3), (512, 7, 5)])
def test_cfg3_shapes_bf16_exact_path(ctx, c, s, n):
    spec = fm.LayerSpec(c, s, s, 0.9, None, 3000 + c)
    run_case(ctx, spec, 4, 4, n, torch.bfloat16, False, exact=True)


@pytest.mark.parametrize("c,s,n", [(96, 28, 2), (144, 14, 3), (960, 7, 3)])
def test_cfg4_like_shapes_bf16(ctx, c, s, n):
    spec = fm.LayerSpec(c, s, s, 0.95, 0.6, 4000 + c)
    run_case(ctx, spec, 5, max(4, (2 * c) // (s * s) + 1), n, torch.bfloat16, False, exact=True)


@pytest.mark.parametrize("cp", [1, 2, 8, 128])
def test_chunk_sizes_and_ragged_tail(ctx, cp):
    # 3 maps of 9x9 = 243 pixels: one full tile and a ragged second one
    spec = fm.LayerSpec(32, 9, 9, 0.85, None, 77)
    run_case(ctx, spec, 6, 8, 3, torch.float32, False, exact=True, chunk_pixels=cp)
    run_case(ctx, spec, 3, 8, 3, torch.bfloat16, True, exact=True, chunk_pixels=cp)


@pytest.mark.parametrize("splits", [1, 2, 4])
def test_pixel_splits_exact_path(ctx, splits):
    # chunks of a half or a quarter of a pixel's coefficients, one full tile and a ragged one
    spec = fm.LayerSpec(32, 9, 9, 0.85, None, 78)
    _, enc = run_case(ctx, spec, 6, 8, 3, torch.float32, False, exact=True, chunk_pixels=1, pixel_splits=splits)
    assert enc.layout.pixel_splits == splits and enc.layout.n_chunks == 243 * splits
    run_case(ctx, spec, 3, 8, 3, torch.bfloat16, True, exact=True, chunk_pixels=1, pixel_splits=splits)


def test_default_chunk_shapes(ctx):
    # side information stays at 16 bits per 96..255 symbols: K = 16 -> 8 pixels per chunk, K = 48 and
    # K = 64 -> 2, K = 96 and K = 128 -> 1, K = 256 -> two chunks per pixel, K = 512 -> four
    for c, want in ((16, (8, 1)), (48, (2, 1)), (64, (2, 1)), (96, (1, 1)), (128, (1, 1)), (256, (1, 2)), (384, (1, 2)),
                    (512, (1, 4)), (960, (1, 4))):
        spec = fm.LayerSpec(c, 4, 4, 0.9, None, 90 + c)
        o = H.oracle_side(spec, 4, 4, 1, torch.bfloat16, False)
        model_h = H.import_model(tc, ctx, o["model"], torch.bfloat16)
        cb = tc.tc_codebook_import(ctx, o["lengths"], 4)
        lay = tc.tc_encode_bound(model_h, cb, o["x"].cuda())
        assert (lay.chunk_pixels, lay.pixel_splits) == want
        assert lay.chunk_len_bytes == 2 * lay.n_chunks
        model_h.close()
        cb.close()


# ---- tensor-core path (bf16 products, fp32 accumulation) -------------------------------------

@pytest.mark.parametrize("c,s,n,bits", [(64, 56, 2, 4), (128, 28, 3, 4), (256, 14, 5, 4), (96, 28, 2, 5),
                                        (144, 14, 5, 5), (192, 28, 2, 5), (16, 8, 9, 3), (256, 14, 3, 8)])
def test_tensor_core_path_shapes(ctx_tc, c, s, n, bits):
    spec = fm.LayerSpec(c, s, s, 0.9, None, 5000 + c + s)
    run_case(ctx_tc, spec, bits, 6, n, torch.bfloat16, False, exact=False)


@pytest.mark.parametrize("bits", [2, 3, 5, 6, 7])
def test_tensor_core_path_bit_width_sweep(ctx_tc, bits):
    spec = fm.workload(5).layers[0]
    run_case(ctx_tc, spec, bits, 8, 7, torch.bfloat16, False, exact=False)


def test_tensor_core_path_per_channel_codebook_and_chunks(ctx_tc):
    spec = fm.LayerSpec(64, 14, 14, 0.9, None, 5100)
    for cp in (1, 4, 32):
        run_case(ctx_tc, spec, 4, 6, 3, torch.bfloat16, True, exact=False, chunk_pixels=cp)
    run_case(ctx_tc, spec, 4, 6, 3, torch.bfloat16, True, exact=False, chunk_pixels=1, pixel_splits=2)


@pytest.mark.parametrize("c,splits", [(256, 1), (256, 2), (64, 2), (128, 2), (192, 2), (256, 4), (128, 4), (64, 4), (192, 4)])
def test_tensor_core_path_pixel_splits(ctx_tc, c, splits):
    spec = fm.LayerSpec(c, 14, 14, 0.9, None, 5300 + c)
    _, enc = run_case(ctx_tc, spec, 5, 6, 5, torch.bfloat16, False, exact=False, chunk_pixels=1, pixel_splits=splits)
    assert enc.layout.pixel_splits == splits


def test_four_splits_per_channel_codebook_and_high_rate(ctx_tc):
    spec = fm.LayerSpec(64, 14, 14, 0.9, None, 5400)
    run_case(ctx_tc, spec, 4, 6, 3, torch.bfloat16, True, exact=False, chunk_pixels=1, pixel_splits=4, routes=(1, 3))
    run_case(ctx_tc, fm.LayerSpec(256, 14, 14, 0.9, None, 5401), 8, 6, 3, torch.bfloat16, False, exact=False,
             chunk_pixels=1, pixel_splits=4, routes=(1, 1))
    # quarters of 24 coefficients: the tensor-core encoders want multiples of 16
    run_case(ctx_tc, fm.LayerSpec(96, 14, 14, 0.9, None, 5402), 4, 6, 3, torch.bfloat16, False, exact=False,
             chunk_pixels=1, pixel_splits=4, routes=(2, 1))


# ---- PCA truncation: only the K leading components are coded (Section 4, ablation) -----------

@pytest.mark.parametrize("c,k,dtype,bits", [(64, 32, torch.float32, 6), (64, 8, torch.float32, 4), (96, 40, torch.bfloat16, 5)])
def test_truncation_exact_path(ctx, c, k, dtype, bits):
    spec = fm.LayerSpec(c, 12, 12, 0.9, None, 5700 + c + k)
    _, enc = run_case(ctx, spec, bits, 6, 3, dtype, False, exact=True, k=k)
    assert enc.symbols.shape[1] == k
    run_case(ctx, spec, bits, 6, 3, dtype, True, exact=True, k=k)


@pytest.mark.parametrize("c,k,bits,splits", [(256, 128, 4, 0), (256, 64, 4, 0), (256, 160, 5, 2), (128, 32, 6, 0),
                                             (192, 96, 3, 1), (64, 16, 4, 0), (256, 256, 4, 1)])
def test_truncation_tensor_core_path(ctx_tc, c, k, bits, splits):
    spec = fm.LayerSpec(c, 14, 14, 0.9, None, 5800 + c + k)
    _, enc = run_case(ctx_tc, spec, bits, 6, 5, torch.bfloat16, False, exact=False, k=k, pixel_splits=splits,
                      chunk_pixels=1 if splits else 0)
    assert enc.symbols.shape[1] == k


def test_truncation_fp32_and_streaming_routes(ctx_tc):
    # K not a multiple of 16 (fp32 kernels), and wide layers (tensor-core kernels that stream the basis)
    run_case(ctx_tc, fm.LayerSpec(64, 14, 14, 0.9, None, 5900), 5, 6, 3, torch.bfloat16, False, exact=False, k=24, routes=(2, 2))
    run_case(ctx_tc, fm.LayerSpec(512, 7, 7, 0.95, None, 5901), 4, 12, 5, torch.bfloat16, False, exact=False, k=128, routes=(3, 3))
    run_case(ctx_tc, fm.LayerSpec(384, 14, 14, 0.95, None, 5902), 5, 4, 2, torch.bfloat16, False, exact=False, k=32, routes=(3, 3))
    run_case(ctx_tc, fm.LayerSpec(576, 14, 14, 0.95, None, 5903), 5, 4, 2, torch.bfloat16, False, exact=False, k=304, routes=(3, 3))


# ---- 8-bit basis (Section 3.1: the PCA matrix is stored in 8 bits) -------------------------------

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_int8_basis_exact_path(ctx, dtype):
    spec = fm.LayerSpec(48, 12, 12, 0.9, None, 6000)
    o, _ = run_case(ctx, spec, 6, 6, 3, dtype, False, exact=True, basis_round="int8")
    assert o["model"].basis_round == "int8"
    run_case(ctx, spec, 4, 6, 3, dtype, True, exact=True, basis_round="int8", k=16)


@pytest.mark.parametrize("c,s,bits,k", [(256, 14, 4, None), (128, 28, 6, None), (64, 28, 8, None), (256, 14, 5, 96)])
def test_int8_basis_tensor_core_path(ctx_tc, c, s, bits, k):
    spec = fm.LayerSpec(c, s, s, 0.9, None, 6100 + c)
    run_case(ctx_tc, spec, bits, 6, 4, torch.bfloat16, False, exact=False, basis_round="int8", k=k)


def test_int8_basis_streaming_route(ctx_tc):
    run_case(ctx_tc, fm.LayerSpec(384, 7, 7, 0.95, None, 6200), 5, 16, 4, torch.bfloat16, False, exact=False,
             basis_round="int8", routes=(3, 3))


def test_library_fit_with_int8_basis_matches_the_oracle(ctx_tc):
    spec = fm.LayerSpec(64, 14, 14, 0.9, None, 6300)
    params = fm.layer_params(spec)
    cal = fm.make_maps(params, 8, calib=True, dtype=torch.bfloat16)
    want = oracle.fit_pca(cal, 5, basis_round="int8", zero_level=True)
    model = tc.tc_fit_pca(ctx_tc, cal.cuda(), 5, basis_dtype=tc.binding.TC_INT8)
    got = tc.tc_model_export(model)
    assert got["basis_dtype"] == tc.binding.TC_INT8
    n_got, n_want = got["basis"] / got["basis_scale"], want.basis / want.basis_scale
    assert np.abs(n_got - np.rint(n_got)).max() <= 1e-9 and abs(np.abs(n_got).max() - 127) <= 1e-9
    assert np.isclose(got["basis_scale"], want.basis_scale, rtol=1e-9)
    # the two eigensolvers agree to rounding: an entry may land on the neighbouring integer at a tie
    assert np.abs(np.rint(n_got) - np.rint(n_want)).max() <= 1
    assert (np.rint(n_got) == np.rint(n_want)).mean() >= 0.999
    assert np.isclose(got["lo"], want.lo, rtol=1e-6, atol=1e-6) and np.isclose(got["step"], want.step, rtol=1e-6)
    # the fitted model codes a bf16 tensor on the tensor-core kernels and an fp32 one on the fp64 kernels
    x = fm.make_maps(params, 3, dtype=torch.bfloat16).cuda()
    st = tc.tc_stats(ctx_tc, model, None, cal.cuda())
    cb = tc.tc_build_codebook(ctx_tc, model, st.hist)
    enc = tc.tc_encode(ctx_tc, model, cb, x)
    assert tc.tc_last_path(ctx_tc) == 1
    a = tc.tc_decode(ctx_tc, model, cb, enc, x.shape, torch.bfloat16)
    enc32 = tc.tc_encode(ctx_tc, model, cb, x.float())
    assert tc.tc_last_path(ctx_tc) == 0
    b = tc.tc_decode(ctx_tc, model, cb, enc32, x.shape, torch.float32)
    assert tc.tc_get_status(ctx_tc) == 0
    assert torch.equal(enc.words[: enc.total_bits() // 8], enc32.words[: enc32.total_bits() // 8]) or \
        (enc.total_bits() - enc32.total_bits()) ** 2 < 1e-6 * enc.total_bits() ** 2
    assert (a.float() - b).abs().max().item() <= 0.02 * b.abs().max().item()
    model.close(); cb.close()


# ---- tensor-core kernels that stream the basis: wide layers, unaligned rows ---------------------

@pytest.mark.parametrize("c,s,n,bits", [(512, 7, 5, 4), (384, 14, 2, 5), (576, 14, 1, 5), (960, 7, 3, 5), (1024, 4, 9, 3),
                                        (272, 6, 8, 6), (960, 7, 6, 8)])
def test_streaming_route_wide_layers(ctx_tc, c, s, n, bits):
    spec = fm.LayerSpec(c, s, s, 0.95, 0.6 if c != 512 else None, 5500 + c)
    run_case(ctx_tc, spec, bits, max(4, (2 * c) // (s * s) + 1), n, torch.bfloat16, False, exact=False, routes=(3, 3))


@pytest.mark.parametrize("splits", [1, 2, 4])
def test_streaming_route_pixel_splits_and_per_channel_codebook(ctx_tc, splits):
    # 640 channels: five blocks of 128 channels, half-tile work items in the decoder
    spec = fm.LayerSpec(640, 7, 7, 0.95, None, 5650)
    _, enc = run_case(ctx_tc, spec, 5, 28, 6, torch.bfloat16, False, exact=False, chunk_pixels=1, pixel_splits=splits,
                      routes=(3, 3))
    assert enc.layout.pixel_splits == splits
    spec = fm.LayerSpec(320, 10, 10, 0.95, None, 5651)
    run_case(ctx_tc, spec, 4, 8, 3, torch.bfloat16, True, exact=False, chunk_pixels=1, pixel_splits=splits, routes=(3, 3))


@pytest.mark.parametrize("cp", [2, 16, 64])
def test_streaming_route_chunks_of_several_pixels(ctx_tc, cp):
    # few coefficients of a wide layer: a chunk holds several pixels; 245 pixels leave a ragged tile
    spec = fm.LayerSpec(576, 7, 7, 0.95, None, 5660)
    run_case(ctx_tc, spec, 5, 24, 5, torch.bfloat16, False, exact=False, k=48, chunk_pixels=cp, routes=(3, 3))
    spec = fm.LayerSpec(288, 7, 7, 0.95, None, 5661)
    run_case(ctx_tc, spec, 5, 12, 5, torch.bfloat16, True, exact=False, k=32, chunk_pixels=cp, routes=(3, 3))


def test_odd_map_sizes_and_shapes_left_to_the_fp32_kernels(ctx_tc):
    # 5x5 maps: the resident-basis encoder needs H*W % 4 == 0 (its decoder does not); the
    # streaming encoder loads such rows element by element
    spec = fm.LayerSpec(64, 5, 5, 0.9, None, 5600)
    run_case(ctx_tc, spec, 6, 8, 7, torch.bfloat16, False, exact=False, routes=(3, 1))
    run_case(ctx_tc, spec, 4, 8, 7, torch.bfloat16, True, exact=False, routes=(3, 1))
    # 24 channels: no tensor-core kernel (C % 16 != 0)
    spec = fm.LayerSpec(24, 9, 9, 0.9, None, 5601)
    run_case(ctx_tc, spec, 5, 8, 3, torch.bfloat16, False, exact=False, chunk_pixels=4, routes=(2, 2))


def test_tensor_core_path_high_rate_tile_overflows_staging(ctx_tc):
    # nearly uniform symbols at 8 bits: a 128-pixel tile of 256 channels packs to more than the
    # staging buffer holds, which exercises the direct-to-global packing route
    spec = fm.LayerSpec(256, 14, 14, 0.999, None, 5200)
    run_case(ctx_tc, spec, 8, 6, 3, torch.bfloat16, False, exact=False)


# ---- the streaming kernels on shapes the resident-basis kernels would take ----------------------

@pytest.fixture(scope="module")
def ctx_stream():
    """Context whose bf16 tensors skip the resident-basis kernels."""
    c = tc.tc_create(0)
    tc.tc_force_exact_path(c, 2)
    yield c
    c.close()


@pytest.mark.parametrize("c,s,n,bits,splits", [(256, 14, 5, 4, 0), (64, 28, 2, 4, 0), (192, 28, 2, 5, 2), (128, 14, 7, 8, 1),
                                               (256, 14, 3, 6, 4)])
def test_streaming_kernels_on_narrow_layers(ctx_stream, c, s, n, bits, splits):
    spec = fm.LayerSpec(c, s, s, 0.9, None, 6400 + c + s)
    run_case(ctx_stream, spec, bits, 6, n, torch.bfloat16, False, exact=False, pixel_splits=splits,
             chunk_pixels=1 if splits else 0, routes=(3, 3))


def test_rate_hint_picks_the_decoder_for_per_channel_tables(ctx_tc):
    # 256 channels at 8 bits with per-channel code tables.  tc_decode never reads a rate into
    # `stream_bytes`; told (tc_encode_params.mean_tile_bytes) that a tile's segment is longer than the
    # resident-basis decoder stages in shared memory, it picks the streaming kernel, which stages up
    # to 32 KB; without the hint, or with a small one, the resident-basis decoder runs.  The hint
    # changes speed only: all three calls return the same tensor.
    spec = fm.LayerSpec(256, 14, 14, 0.9, None, 6500)
    o = H.oracle_side(spec, 8, 6, 8, torch.bfloat16, True)
    model = H.import_model(tc, ctx_tc, o["model"], torch.bfloat16)
    cb = tc.tc_codebook_import(ctx_tc, o["lengths"], 8)
    x = o["x"].cuda()
    enc = tc.tc_encode(ctx_tc, model, cb, x, debug=True)
    nbytes = enc.total_bits() // 8
    outs = []
    for hint, route in ((30000, 3), (None, 1), (2000, 1)):
        outs.append(tc.tc_decode(ctx_tc, model, cb, enc, x.shape, torch.bfloat16, stream_bytes=nbytes if hint else None,
                                 mean_tile_bytes=hint))
        assert tc.tc_get_status(ctx_tc) == 0 and tc.tc_last_path(ctx_tc, True) == route
    want = oracle.reconstruct(o["model"], enc.symbols.cpu().numpy(), x.shape, out_bf16=True)
    expected = H.expected_output_flips(o["model"], enc.symbols.cpu().numpy())
    for got in (t.float().cpu().numpy() for t in outs):
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
        assert np.all(np.abs(got - want) <= np.maximum(1e-3 * np.maximum(np.abs(want), o["model"].step), ulp))
        assert H.count_output_flips(got, want) <= H.flip_allowance(expected)
    assert torch.equal(outs[1], outs[2])
    model.close(); cb.close()


@pytest.mark.parametrize("c,s,n,routes", [(320, 1, 1, (3, 3)), (1024, 2, 1, (3, 3)), (64, 1, 3, (3, 1))])
def test_single_pixels_and_tiny_maps(ctx_tc, c, s, n, routes):
    # one to four pixels: a single, mostly empty tile; 1 x 1 maps have unaligned rows
    spec = fm.LayerSpec(c, s, s, 0.9, None, 6600 + c)
    run_case(ctx_tc, spec, 4, 40 if c > 512 else 24, n, torch.bfloat16, False, exact=False, routes=routes)
