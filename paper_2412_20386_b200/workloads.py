"""Seeded synthetic inputs shaped like the linear layers of Vim / VMamba.

This module only draws random tensors.  It contains none of the method's
arithmetic (no smoothing, no quantization, no matmul): the static parameters
``s`` and ``dx`` are derived from the calibration batch by whoever consumes
these tensors.  Both the CUDA library's tests/benchmark and the CPU oracle's
tests read their inputs from here, so the two sides see identical bytes.

The tensors stand in for activations of pretrained Visual Mamba backbones on
ImageNet (Sec. 6.1, Quantization Setting), which are not available offline.  Their
structure follows the paper's three observations (Sec. 4.1-4.3): token-wise variance
that is consistent across images, a class token of much smaller magnitude,
outliers confined to a few channels, and a long-tailed value distribution.

    x[b,t,k] = sat_fp16( StudentT(df)[b,t,k] * g[t] * o[k] )
    g[t]     = exp(Normal(0, 0.5)), drawn once per layer and shared by the
               calibration and evaluation batches; the class-token position
               (index 98 of 197 in Vim) is additionally scaled by 0.1
    o[k]     = outlier_scale on n_outliers seeded channels, 1 elsewhere
    Wq       = uniform integers in [-127, 127]      (symmetric range, Sec. 2.3)
    dw[n]    = uniform in [1e-3, 1e-2]
    bias[n]  = Normal(0, 1), dt_proj only
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional

import numpy as np

ROOT_SEED = 241220386
ROLE_EVAL, ROLE_CALIB, ROLE_WEIGHTS, ROLE_STRUCTURE = 0, 1, 2, 3
CALIB_IMAGES = 8
FP16_MAX = 65504.0


@dataclass(frozen=True)
class LinearSpec:
    """One quantized linear layer of one workload configuration."""
    config: int           # workload configuration index (0..4)
    layer: int            # block / stage index inside the configuration
    linear: int           # 0 in_proj, 1 x_proj, 2 dt_proj, 3 out_proj
    name: str
    B: int                # images in the evaluation batch
    T: int                # token positions per image
    K: int                # input channels  (D_in)
    N: int                # output channels (D_out)
    bias: bool = False
    df: float = 3.0       # Student-t degrees of freedom
    n_outliers: int = 4
    outlier_scale: float = 20.0
    cls_index: Optional[int] = None

    @property
    def M(self) -> int:
        return self.B * self.T

    def with_batch(self, B: int) -> "LinearSpec":
        return replace(self, B=B)


_LINEAR_NAMES = ("in_proj", "x_proj", "dt_proj", "out_proj")


def _vim(config, layer, linear, B, K, N, **kw):
    return LinearSpec(config, layer, linear, _LINEAR_NAMES[linear], B, 197, K, N,
                      cls_index=98, **kw)


def configs() -> Dict[int, List[LinearSpec]]:
    """The five workload configurations (shapes of Vim-Ti/S/B and a VMamba-like stack)."""
    c: Dict[int, List[LinearSpec]] = {}
    # 0: Vim-Ti out_proj alone, one image.
    c[0] = [_vim(0, 0, 3, 1, 384, 192)]
    # 1: every block linear of Vim-Ti, batch 64, 24 layers.
    c[1] = []
    for layer in range(24):
        c[1] += [_vim(1, layer, 0, 64, 192, 768),
                 _vim(1, layer, 1, 64, 384, 44),
                 _vim(1, layer, 2, 64, 12, 384, bias=True),
                 _vim(1, layer, 3, 64, 384, 192)]
    # 2: Vim-S, batch 128.
    c[2] = [_vim(2, 0, 0, 128, 384, 1536), _vim(2, 0, 3, 128, 768, 384)]
    # 3: Vim-B, batch 256, heavier tail and stronger outliers.
    heavy = dict(df=2.5, n_outliers=8, outlier_scale=50.0)
    c[3] = [_vim(3, 0, 0, 256, 768, 3072, **heavy), _vim(3, 0, 3, 256, 1536, 768, **heavy)]
    # 4: VMamba-like hierarchical stages, batch 64 at 224x224.
    c[4] = []
    for stage, (T, d) in enumerate(((3136, 96), (784, 192), (196, 384), (49, 768))):
        c[4] += [LinearSpec(4, stage, 0, "in_proj", 64, T, d, 4 * d),
                 LinearSpec(4, stage, 3, "out_proj", 64, T, 2 * d, d)]
    return c


def _rng(spec: LinearSpec, role: int) -> np.random.Generator:
    seq = np.random.SeedSequence([ROOT_SEED, spec.config, spec.layer, spec.linear, role])
    return np.random.Generator(np.random.Philox(seq))


def structure(spec: LinearSpec):
    """Per-layer token gains g[T] and channel gains o[K] (float64)."""
    rng = _rng(spec, ROLE_STRUCTURE)
    g = np.exp(rng.normal(0.0, 0.5, size=spec.T))
    if spec.cls_index is not None and spec.cls_index < spec.T:
        g[spec.cls_index] *= 0.1
    o = np.ones(spec.K)
    n_out = min(spec.n_outliers, spec.K)
    o[rng.choice(spec.K, size=n_out, replace=False)] = spec.outlier_scale
    return g, o


def activations(spec: LinearSpec, role: int = ROLE_EVAL, B: Optional[int] = None) -> np.ndarray:
    """fp16 activations [B, T, K] for the evaluation (role 0) or calibration (role 1) batch."""
    if B is None:
        B = CALIB_IMAGES if role == ROLE_CALIB else spec.B
    g, o = structure(spec)
    scale = (g[:, None] * o[None, :])
    rng = _rng(spec, role)
    x = np.empty((B, spec.T, spec.K), np.float16)
    # Image by image keeps the float64 scratch small; the stream of random numbers
    # (and therefore the tensor) does not depend on the chunking.
    for b in range(B):
        v = rng.standard_t(spec.df, size=(spec.T, spec.K)) * scale
        np.clip(v, -FP16_MAX, FP16_MAX, out=v)
        x[b] = v.astype(np.float16)
    return x


def weights(spec: LinearSpec):
    """(Wq int8 [N,K], dw fp32 [N], bias fp32 [N] or None)."""
    rng = _rng(spec, ROLE_WEIGHTS)
    wq = rng.integers(-127, 128, size=(spec.N, spec.K), dtype=np.int64).astype(np.int8)
    dw = rng.uniform(1e-3, 1e-2, size=spec.N).astype(np.float32)
    bias = rng.normal(0.0, 1.0, size=spec.N).astype(np.float32) if spec.bias else None
    return wq, dw, bias
