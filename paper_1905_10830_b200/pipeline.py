"""Layer-by-layer calibration and chained coding of several layers' feature maps.

Section 3.1 ("Linear transform"): the covariance of a layer is estimated on a calibration batch
*with the layers before it already quantised*, so that every encoder sees, at calibration time,
the inputs it will see at inference.  Fig. 2 puts the codec between the layers: the feature map
a layer produces is encoded, stored, decoded, passed through the layer's non-linearity and
consumed by the next convolution.

The network itself is the caller's: a stage is any callable that maps the (reconstructed,
activated) feature map of the stage before to this stage's pre-activation feature map -- a
convolution and batch normalisation in the paper, any torch function here.  This module only
orders the calls of the C-ABI library (fit, statistics, codebook, encode, decode); every step
of the coding path runs in the library's kernels."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Sequence

import torch

from . import binding as tc


@dataclass
class CodedLayer:
    """What calibration leaves behind for one layer: its transform / quantiser and its code table."""
    model: tc.Model
    codebook: tc.Codebook
    bits: int
    relu: bool

    def close(self) -> None:
        self.model.close()
        self.codebook.close()


def code_layer(ctx: tc.Context, layer: CodedLayer, z: torch.Tensor):
    """Encode `z`, decode it again (with the layer's non-linearity when it has one) and return
    (reconstruction, coded bits): what the next stage reads from memory."""
    enc = tc.tc_encode(ctx, layer.model, layer.codebook, z)
    xhat = tc.tc_decode(ctx, layer.model, layer.codebook, enc, z.shape, z.dtype, relu=layer.relu)
    return xhat, enc.total_bits()


def calibrate_layer_by_layer(ctx: tc.Context, stages: Sequence[Callable[[torch.Tensor], torch.Tensor]],
                             calib_input: torch.Tensor, bits: Sequence[int], relu: Sequence[bool], *,
                             per_channel_codebook: bool = False, k: Sequence[int] | None = None) -> list[CodedLayer]:
    """Fit one CodedLayer per stage on `calib_input`.  Stage l's feature maps are computed from the
    *reconstruction* of stage l - 1 (encode, decode, non-linearity), never from its clean output, so
    the statistics each fit sees include the quantisation noise of everything upstream."""
    layers: list[CodedLayer] = []
    cur = calib_input
    for l, stage in enumerate(stages):
        z = stage(cur).contiguous()
        model = tc.tc_fit_pca(ctx, z, bits=bits[l], k=0 if k is None else k[l])
        groups = (k[l] if k is not None and k[l] else z.shape[1]) if per_channel_codebook else 1
        st = tc.tc_stats(ctx, model, None, z, groups=groups)
        cb = tc.tc_build_codebook(ctx, model, st.hist, groups=groups)
        layer = CodedLayer(model, cb, bits[l], bool(relu[l]))
        layers.append(layer)
        cur, _ = code_layer(ctx, layer, z)
    return layers


def run_chain(ctx: tc.Context, stages: Sequence[Callable[[torch.Tensor], torch.Tensor]], layers: Sequence[CodedLayer],
              x: torch.Tensor):
    """Inference through the chain: every stage's feature map goes through its encoder and decoder
    before the next stage reads it.  Returns (feature maps as coded, reconstructions, bits per layer)."""
    maps, recons, bits = [], [], []
    cur = x
    for stage, layer in zip(stages, layers):
        z = stage(cur).contiguous()
        cur, nbits = code_layer(ctx, layer, z)
        maps.append(z)
        recons.append(cur)
        bits.append(nbits)
    return maps, recons, bits
