"""Runs the five workload configurations through the library on one GPU and prints a Markdown
table: bits/value, encode / decode / round-trip GB/s of raw activations, fraction of the HBM
roofline, which kernels ran, and parity against the CPU oracle on a sample of each layer.

    python report.py [--cfg 1 2 3 4 5] [--reps 5] [--out FILE]

The oracle (test infrastructure) is imported only for the parity columns; with --no-oracle the
table has the throughput columns alone."""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import paper_1905_10830_b200 as tc
from synth import featuremaps as fm


def _peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"])
    return 6650.0


def _tensor_peak():
    """Measured bf16 matmul rate in TFLOP/s (the burst figure: these kernels are timed alone)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["bf16_tflops"])
    return 1590.0


def _time(fn, reps):
    fn()
    torch.cuda.synchronize()
    best = 1e30
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b))
    return best


def _parity(ctx, model, cb, x_sample, bits, per_channel):
    import oracle
    d = tc.tc_model_export(model)
    dtype = x_sample.dtype
    m = oracle.Model(d["c"], d["k"], bits, d["mean"], d["basis"], d["eig"], d["lo"], d["step"],
                     "bf16" if dtype == torch.bfloat16 else "f32")
    lengths = tc.tc_codebook_export(cb)
    enc = tc.tc_encode(ctx, model, cb, x_sample, debug=True)
    xhat = tc.tc_decode(ctx, model, cb, enc, x_sample.shape, dtype)
    assert tc.tc_get_status(ctx) == 0
    q_gpu = enc.symbols.cpu().numpy()
    y = oracle.project(m, x_sample.cpu())
    q, units = oracle.quantize(m, y, with_units=True)
    y_gpu = enc.coefficients.cpu().numpy().astype(np.float64)
    coef_err = float(np.max(np.abs(y_gpu - y) / np.maximum(np.abs(y), m.step)))
    bad = q_gpu != q
    ties_only = bool(np.all(np.abs(units[bad] - np.floor(units[bad]) - 0.5) <= 1e-3)) if bad.any() else True
    ref = oracle.encode(q_gpu, lengths, bits, chunk_pixels=enc.layout.chunk_pixels,
                        pixel_splits=enc.layout.pixel_splits, tile_pixels=128)
    words = enc.words[: enc.total_bits() // 8].cpu().numpy().view(np.uint32)
    lens = enc.chunk_len[: enc.layout.n_chunks].cpu().numpy().view(np.uint16)
    stream_exact = bool(np.array_equal(words, ref.words) and np.array_equal(lens, ref.chunk_len))
    want = oracle.reconstruct(m, q_gpu, x_sample.shape, out_bf16=(dtype == torch.bfloat16))
    got = xhat.float().cpu().numpy()
    flips = "-"
    if dtype == torch.bfloat16:       # how many outputs the fp32 accumulation may round to the neighbouring value (tests/helpers.py)
        from tests import helpers as H
        flips = f"{H.count_output_flips(got, want)} / {H.flip_allowance(H.expected_output_flips(m, q_gpu))}"
    return dict(stream_exact=stream_exact, coef_err=coef_err, mismatch=float(bad.mean()), ties_only=ties_only,
                xhat_equal=float((got == want).mean()), flips=flips)


def run(cfgs, reps, with_oracle, max_batch):
    peak = _peak()
    ctx = tc.tc_create(0)
    rows = []
    for cfg in cfgs:
        w = fm.workload(cfg)
        for spec, repeat in zip(w.layers, w.repeats):
            params = fm.layer_params(spec)
            batch = min(w.batch, max_batch)
            cal = fm.make_maps(params, w.calib_maps, calib=True, dtype=w.dtype, device="cuda")
            x = fm.make_maps(params, batch, dtype=w.dtype, device="cuda")
            values = x.numel()
            raw = values * x.element_size()
            groups = spec.c if w.per_channel_codebook else 1
            for bits in w.bits:
                model = tc.tc_fit_pca(ctx, cal, bits=bits)
                st = tc.tc_stats(ctx, model, None, cal, groups=groups)
                cb = tc.tc_build_codebook(ctx, model, st.hist, groups=groups)
                enc = tc.tc_encode(ctx, model, cb, x)
                xhat = torch.empty_like(x)
                nbytes = enc.total_bits() // 8
                t_enc = _time(lambda: tc.tc_encode(ctx, model, cb, x, out=enc), reps)
                t_dec = _time(lambda: tc.tc_decode(ctx, model, cb, enc, x.shape, x.dtype, out=xhat, stream_bytes=nbytes), reps)
                q_enc = _time_back_to_back(lambda: tc.tc_encode(ctx, model, cb, x, out=enc))
                q_dec = _time_back_to_back(lambda: tc.tc_decode(ctx, model, cb, enc, x.shape, x.dtype, out=xhat, stream_bytes=nbytes))
                assert tc.tc_get_status(ctx) == 0
                side = enc.layout.chunk_len_bytes + enc.layout.tile_off_bytes
                algo = raw + nbytes + side
                # which roofline binds the layer: bytes at the copy bandwidth, or the projection's
                # 2 P C K flops at the matmul rate (the wide layers), and how close each kernel comes
                flops = 2.0 * (values / spec.c) * spec.c * spec.c                  # K = C in every configuration
                t_hbm, t_tensor = algo / (peak * 1e9) * 1e3, flops / (_tensor_peak() * 1e12) * 1e3      # ms
                bound, t_ideal = ("tensor", t_tensor) if t_tensor > t_hbm else ("hbm", t_hbm)
                tst = tc.tc_stats(ctx, model, cb, x[: min(batch, 64)], groups=groups, want_hist=False)
                row = dict(cfg=cfg, layer=spec.name + (f" x{repeat}" if repeat > 1 else ""), batch=batch, dtype=str(w.dtype).split(".")[-1],
                           b=bits, entropy=tst.entropy, huffman=tst.mean_length, stream=8 * nbytes / values,
                           total=8 * (nbytes + side) / values, mse=tst.mse,
                           enc_gbs=raw / t_enc / 1e6, dec_gbs=raw / t_dec / 1e6, rt_gbs=raw / (t_enc + t_dec) / 1e6,
                           enc_ms=t_enc, dec_ms=t_dec, q_enc_ms=q_enc, q_dec_ms=q_dec, enc_frac=algo / t_enc / 1e6 / peak, dec_frac=algo / t_dec / 1e6 / peak,
                           enc_frac8=algo / t_enc / 1e6 / 8000, dec_frac8=algo / t_dec / 1e6 / 8000,
                           bound=bound, enc_bound_frac=t_ideal / t_enc, dec_bound_frac=t_ideal / t_dec,
                           kernels=["fp64", "tcgen05", "fp32", "tcgen05-stream"][tc.tc_last_path(ctx, False)] + "/" + ["fp64", "tcgen05", "fp32", "tcgen05-stream"][tc.tc_last_path(ctx, True)])
                if with_oracle:
                    row.update(_parity(ctx, model, cb, x[: max(1, min(batch, 2))].contiguous(), bits, w.per_channel_codebook))
                rows.append(row)
                model.close()
                cb.close()
            del x, cal
            torch.cuda.empty_cache()
    return rows, peak


def layer_sets(cfgs, reps, max_batch):
    """Configurations with several layers: the whole set coded by one tc_encode_many / tc_decode_many
    call each, against the same layers coded by one call per layer (queued back to back)."""
    ctx = tc.tc_create(0)
    out = []
    for cfg in cfgs:
        w = fm.workload(cfg)
        if sum(w.repeats) < 2 or w.per_channel_codebook:
            continue
        bits = w.bits[0]
        batch = min(w.batch, max_batch)
        layers = []
        for spec, repeat in zip(w.layers, w.repeats):
            params = fm.layer_params(spec)
            cal = fm.make_maps(params, w.calib_maps, calib=True, dtype=w.dtype, device="cuda")
            model = tc.tc_fit_pca(ctx, cal, bits=bits)
            st = tc.tc_stats(ctx, model, None, cal)
            cb = tc.tc_build_codebook(ctx, model, st.hist)
            for r in range(repeat):
                layers.append((model, cb, fm.make_maps(params, batch, dtype=w.dtype, device="cuda", offset=1000 * r)))
            del cal
        encs = tc.tc_encode_many(ctx, layers)
        dec_layers = [(m, cb, e, x.shape, x.dtype) for (m, cb, x), e in zip(layers, encs)]
        outs = tc.tc_decode_many(ctx, dec_layers)

        def enc_each():
            for (m, cb, x), e in zip(layers, encs):
                tc.tc_encode(ctx, m, cb, x, out=e)

        def dec_each():
            for (m, cb, e, shape, dtype), o in zip(dec_layers, outs):
                tc.tc_decode(ctx, m, cb, e, shape, dtype, out=o)

        raw = sum(x.numel() * x.element_size() for _, _, x in layers)
        row = dict(cfg=cfg, name=w.name, layers=len(layers), batch=batch, bits=bits, raw_mb=raw / 1e6,
                   enc_many=_time(lambda: tc.tc_encode_many(ctx, layers, outs=encs), reps),
                   dec_many=_time(lambda: tc.tc_decode_many(ctx, dec_layers, outs=outs), reps),
                   enc_each=_time(enc_each, reps), dec_each=_time(dec_each, reps))
        assert tc.tc_get_status(ctx) == 0
        out.append(row)
        del layers, encs, outs, dec_layers
        torch.cuda.empty_cache()
    return out


def layer_sets_markdown(rows):
    out = ["", "Whole layer sets in one call (`tc_encode_many` / `tc_decode_many`) against one call per layer, queued back to back:", "",
           "| cfg | layers | N | b | raw MB | encode: many ms | per layer ms | decode: many ms | per layer ms | round trip GB/s (many) |",
           "|---|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        out.append(f"| {r['cfg']} | {r['layers']} | {r['batch']} | {r['bits']} | {r['raw_mb']:.1f} | {r['enc_many']:.3f} | {r['enc_each']:.3f} | "
                   f"{r['dec_many']:.3f} | {r['dec_each']:.3f} | {r['raw_mb'] / (r['enc_many'] + r['dec_many']) / 1e3 * 1e3:.1f} |")
    return "\n".join(out)


def _time_back_to_back(fn, calls=20):
    """Milliseconds per call when `calls` calls are queued one after the other (one event pair
    around all of them): what a layer costs inside a pipeline that does not wait between layers."""
    fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(calls):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / calls


def to_markdown(rows, peak, with_oracle):
    head = ["cfg", "layer", "N", "dtype", "b", "entropy", "Huffman", "stream+pad", "+offsets", "MSE", "enc ms", "dec ms", "enc / dec ms queued x20", "enc GB/s", "dec GB/s",
            "round trip GB/s", f"HBM frac enc/dec (of {peak:.0f} GB/s measured)", "(of 8000 GB/s)",
            f"binding roofline (bytes at the copy rate, or 2PCK flops at {_tensor_peak():.0f} TF/s measured)", "frac of it enc/dec", "kernels enc/dec"]
    if with_oracle:
        head += ["stream bit-exact", "coef max rel err", "symbol mismatch", "only at ties", "x_hat bit-equal", "x_hat values off by one / allowed"]
    out = ["| " + " | ".join(head) + " |", "|" + "---|" * len(head)]
    for r in rows:
        cells = [r["cfg"], r["layer"], r["batch"], r["dtype"], r["b"], f"{r['entropy']:.3f}", f"{r['huffman']:.3f}", f"{r['stream']:.3f}",
                 f"{r['total']:.3f}", f"{r['mse']:.3g}", f"{r['enc_ms']:.3f}", f"{r['dec_ms']:.3f}", f"{r['q_enc_ms']:.3f} / {r['q_dec_ms']:.3f}", f"{r['enc_gbs']:.1f}", f"{r['dec_gbs']:.1f}",
                 f"{r['rt_gbs']:.1f}", f"{r['enc_frac']:.3f} / {r['dec_frac']:.3f}", f"{r['enc_frac8']:.3f} / {r['dec_frac8']:.3f}",
                 r["bound"], f"{r['enc_bound_frac']:.3f} / {r['dec_bound_frac']:.3f}", r["kernels"]]
        if with_oracle:
            cells += ["yes" if r["stream_exact"] else "NO", f"{r['coef_err']:.1e}", f"{r['mismatch']:.1e}", "yes" if r["ties_only"] else "NO",
                      f"{r['xhat_equal']:.5f}", r["flips"]]
        out.append("| " + " | ".join(str(c) for c in cells) + " |")
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--cfg", type=int, nargs="*", default=[1, 2, 3, 4, 5])
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--max-batch", type=int, default=1 << 30)
    ap.add_argument("--no-oracle", action="store_true")
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    rows, peak = run(args.cfg, args.reps, not args.no_oracle, args.max_batch)
    md = to_markdown(rows, peak, not args.no_oracle)
    sets = layer_sets(args.cfg, args.reps, args.max_batch)
    if sets:
        md += "\n" + layer_sets_markdown(sets)
    print(md)
    if args.out:
        with open(args.out, "w") as f:
            f.write(md + "\n")


if __name__ == "__main__":
    main()
