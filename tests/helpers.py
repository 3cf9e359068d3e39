"""Shared set-up for the parity tests: build the oracle's model and codebook on the CPU and
import them into the CUDA library, so that both sides use identical T, mu, lo, step and code
lengths on identical input bytes."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from synth import featuremaps as fm


def basis_round_for(dtype) -> str:
    return "bf16" if dtype == torch.bfloat16 else "f32"


def oracle_side(spec: fm.LayerSpec, bits: int, n_cal: int, n_test: int, dtype, per_channel: bool,
                lmax: int = 12, model: oracle.Model | None = None, k: int | None = None,
                basis_round: str | None = None):
    """Returns dict(model, lengths, cal, x, y, q, units) computed by the oracle on CPU maps."""
    params = fm.layer_params(spec)
    cal = fm.make_maps(params, n_cal, calib=True, dtype=dtype)
    x = fm.make_maps(params, n_test, dtype=dtype)
    if model is None:
        model = oracle.fit_pca(cal, bits, basis_round=basis_round or basis_round_for(dtype), k=k)
    elif model.bits != bits:
        model = oracle.with_bits(model, bits)
    q_cal = oracle.quantize(model, oracle.project(model, cal))
    lengths = oracle.huffman_lengths(oracle.histogram(q_cal, bits, per_channel), lmax)
    y = oracle.project(model, x)
    q, units = oracle.quantize(model, y, with_units=True)
    return dict(model=model, lengths=lengths, cal=cal, x=x, y=y, q=q, units=units, q_cal=q_cal)


def import_model(tc, ctx, m: oracle.Model, dtype):
    if m.basis_round == "int8":
        basis_dtype = tc.binding.TC_INT8
    else:
        basis_dtype = tc.binding.TC_BF16 if dtype == torch.bfloat16 else tc.binding.TC_F32
    return tc.tc_model_import(ctx, basis=m.basis, mean=m.mean, lo=m.lo, step=m.step, bits=m.bits,
                              basis_dtype=basis_dtype, k=m.k, eig=m.eig, basis_scale=m.basis_scale)


def stream_words(enc) -> np.ndarray:
    total = enc.total_bits()
    return enc.words[: total // 8].cpu().numpy().view(np.uint32)


def chunk_len(enc) -> np.ndarray:
    return enc.chunk_len[: enc.layout.n_chunks].cpu().numpy().view(np.uint16)


def tile_off(enc) -> np.ndarray:
    return enc.tile_off.cpu().numpy().view(np.uint64)
