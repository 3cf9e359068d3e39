"""Seeded synthetic CNN feature maps (inputs only: none of the codec's arithmetic lives here).

The paper measures on ImageNet activations of pretrained ResNet / MobileNetV2 networks
(Section 4, Table 1).  Neither the dataset nor the weights are available, so the maps made
here stand in for them: they have the paper's layer shapes and a controllable amount of
inter-channel correlation (the property Section 3 and Appendix G say the method exploits).

Recipe, per layer shape (C, H, W), eigenvalue decay ratio r and seed:
  1. Q    = orthogonal factor of a seeded C x C standard-normal matrix (QR, diag(R) > 0).
  2. lam  = r**i, i = 0..C-1, rescaled so that sum(lam) = C (unit mean channel variance).
  3. Z    ~ N(0,1)^{C x H x W};  S[:, h, w] = Q diag(sqrt(lam)) Z[:, h, w].
  4. 3x3 box blur per channel, zero padding, divided by 9.
  5. bias beta_c ~ N(0.2, 0.1^2), drawn once per layer; or, when `zero_fraction` is given,
     beta_c = -sigma_c * Phi^{-1}(zero_fraction) with sigma_c the interior post-blur standard
     deviation, so that about `zero_fraction` of the values are ReLU zeros.
  6. x = max(S_blur + beta, 0), cast (round to nearest even) to fp32 or bf16.
Calibration and test maps share (Q, lam, beta) and use independent Z streams.

Both the CPU oracle's tests and the CUDA library's tests / benchmark take their inputs from
this module, so that the two sides always see identical bytes.
"""
from __future__ import annotations

import dataclasses
import math
from statistics import NormalDist

import torch

BASE_SEED = 190510830

# Named sub-streams of a layer seed.
_STREAM_Q, _STREAM_BETA, _STREAM_CALIB, _STREAM_TEST = 1, 2, 3, 4


@dataclasses.dataclass
class LayerSpec:
    """Shape and statistics of one synthetic layer."""
    c: int
    h: int
    w: int
    ratio: float = 0.85
    zero_fraction: float | None = None
    seed: int = BASE_SEED
    name: str = ""

    @property
    def hw(self) -> int:
        return self.h * self.w


@dataclasses.dataclass
class LayerParams:
    spec: LayerSpec
    mix: torch.Tensor      # C x C, Q diag(sqrt(lam)), float32, CPU
    beta: torch.Tensor     # C, float32, CPU
    lam: torch.Tensor      # C, float64, CPU
    q: torch.Tensor        # C x C orthogonal, float64, CPU


def _gen(seed: int, stream: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + stream * 7919) % (2**63 - 1))
    return g


def layer_params(spec: LayerSpec) -> LayerParams:
    """Draw the per-layer constants (Q, lam, beta). Always on the CPU, in fp64."""
    c = spec.c
    a = torch.randn(c, c, generator=_gen(spec.seed, _STREAM_Q), dtype=torch.float64)
    q, r = torch.linalg.qr(a)
    q = q * torch.sign(torch.diagonal(r)).unsqueeze(0)   # make diag(R) > 0
    lam = torch.tensor([spec.ratio ** i for i in range(c)], dtype=torch.float64)
    lam = lam * (c / lam.sum())
    mix = q * lam.sqrt().unsqueeze(0)
    if spec.zero_fraction is None:
        beta = 0.2 + 0.1 * torch.randn(c, generator=_gen(spec.seed, _STREAM_BETA),
                                       dtype=torch.float64)
    else:
        sigma = ((mix * mix).sum(dim=1) / 9.0).sqrt()
        beta = -sigma * NormalDist().inv_cdf(spec.zero_fraction)
    return LayerParams(spec, mix.float().contiguous(), beta.float().contiguous(), lam, q)


def make_maps(params: LayerParams, n: int, *, calib: bool = False, dtype=torch.float32,
              device: str = "cpu", batch: int = 256, offset: int = 0) -> torch.Tensor:
    """Return `n` maps as a dense NCHW tensor of `dtype` on `device`.

    `calib` picks the calibration stream instead of the test stream; `offset` shifts the
    stream (e.g. a rank index) so that shards draw different maps from the same layer.
    """
    spec = params.spec
    stream = (_STREAM_CALIB if calib else _STREAM_TEST) + 16 * offset
    g = _gen(spec.seed, stream, device)
    mix = params.mix.to(device)
    beta = params.beta.to(device).view(1, -1, 1, 1)
    out = torch.empty(n, spec.c, spec.h, spec.w, dtype=dtype, device=device)
    for i0 in range(0, n, batch):
        m = min(batch, n - i0)
        z = torch.randn(m, spec.c, spec.h, spec.w, generator=g, dtype=torch.float32,
                        device=device)
        s = torch.matmul(mix, z.view(m, spec.c, spec.hw)).view(m, spec.c, spec.h, spec.w)
        s = torch.nn.functional.avg_pool2d(s, 3, stride=1, padding=1, count_include_pad=True)
        out[i0:i0 + m] = torch.clamp_min(s + beta, 0.0).to(dtype)
    return out


def make_plain_gaussian(params: LayerParams, n: int, *, device: str = "cpu") -> torch.Tensor:
    """Maps with steps 4-6 skipped (no blur, bias or ReLU): covariance is exactly
    Q diag(lam) Q^T, which the fit tests use as a known answer."""
    spec = params.spec
    g = _gen(spec.seed, _STREAM_TEST + 8, device)
    z = torch.randn(n, spec.c, spec.hw, generator=g, dtype=torch.float64, device=device)
    s = torch.matmul(params.q.to(device) * params.lam.sqrt().to(device).unsqueeze(0), z)
    return s.view(n, spec.c, spec.h, spec.w)


# --------------------------------------------------------------------------------------
# The five workload configurations (shapes from the paper's networks).
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class Workload:
    name: str
    layers: list[LayerSpec]
    repeats: list[int]          # how many network blocks share each layer shape
    batch: int
    dtype: torch.dtype
    bits: list[int]
    calib_maps: int
    per_channel_codebook: bool


def _seed(cfg: int, layer: int) -> int:
    return BASE_SEED + cfg * 101 + layer


def workload(cfg: int) -> Workload:
    """cfg 1..5, in the order of the benchmark's configuration list."""
    if cfg == 1:
        return Workload("cfg1_single_map_64x56x56_f32",
                        [LayerSpec(64, 56, 56, 0.85, None, _seed(1, 0), "64x56x56")], [1],
                        1, torch.float32, [8], 16, False)
    if cfg == 2:
        shapes = [(64, 56), (128, 28), (256, 14), (512, 7)]
        return Workload("cfg2_resnet18_b1_f32",
                        [LayerSpec(c, s, s, 0.85, None, _seed(2, i), f"{c}x{s}x{s}")
                         for i, (c, s) in enumerate(shapes)], [1, 1, 1, 1],
                        1, torch.float32, [2, 3, 4, 6, 8], 32, True)
    if cfg == 3:
        shapes = [(64, 56), (128, 28), (256, 14), (512, 7)]
        return Workload("cfg3_resnet34_b64_bf16",
                        [LayerSpec(c, s, s, 0.9, None, _seed(3, i), f"{c}x{s}x{s}")
                         for i, (c, s) in enumerate(shapes)], [3, 4, 6, 3],
                        64, torch.bfloat16, [4], 256, False)
    if cfg == 4:
        shapes = [(96, 112), (144, 56), (192, 28), (384, 14), (576, 14), (960, 7)]
        return Workload("cfg4_mobilenetv2_b128_bf16",
                        [LayerSpec(c, s, s, 0.95, 0.6, _seed(4, i), f"{c}x{s}x{s}")
                         for i, (c, s) in enumerate(shapes)], [1] * 6,
                        128, torch.bfloat16, [5], 64, False)
    if cfg == 5:
        return Workload("cfg5_256x14x14_b4096_bf16",
                        [LayerSpec(256, 14, 14, 0.9, None, _seed(5, 0), "256x14x14")], [1],
                        4096, torch.bfloat16, [2, 3, 4, 5, 6, 7, 8], 256, False)
    raise ValueError(f"unknown workload configuration {cfg}")
