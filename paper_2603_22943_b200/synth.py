"""Seeded synthetic inputs shaped like SD-1.5 / SDXL cross-attention layers.

This module holds no arithmetic of the method (no quantizer, no attention): it only draws random
tensors.  It is the one piece of code that both the CUDA path's tests and the CPU oracle's tests
use, so both sides see bit-identical inputs.  The tensors stand in for the activations and weights
of personalised Stable-Diffusion checkpoints, which are not available offline; only their shapes,
value distributions and trigger structure are reproduced:

* hidden states X[B,N,C]: N(0,1), with max(1, round(C/100)) "outlier" channels scaled by 20,
  rounded once to fp16 (the layer input *is* fp16 data);
* text context ctx[B,T,Dc]: N(0,1), rows at trigger positions scaled by 3, rounded once to fp16;
* weights W_q, W_out [C,C], W_k, W_v [C,Dc]: N(0, 1/fan_in) in fp32; to_out bias N(0, 0.1^2);
* trigger mask [B,T] uint8, 1 at the trigger span.

Draw order (numpy ``default_rng(seed)``, PCG64) is fixed: X, outlier channel indices, ctx, W_q, W_k,
W_v, W_out, b_out.  Checkpoint weights for the multi-checkpoint serving sweep come from their own
seeds so that a checkpoint does not depend on the request that uses it.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class LayerShape:
    """One cross-attention layer problem.  Names follow the paper's notation (Sec. III-B)."""
    batch: int           # B
    n_query: int         # N  (image tokens)
    channels: int        # C = heads * d
    heads: int           # H
    n_ctx: int           # T  (text tokens)
    ctx_dim: int         # Dc (text-encoder width)
    w_bits: int          # 8 or 4
    w_group: int         # 0 = one scale per output channel, 128 = groups along fan-in
    trigger: Tuple[int, ...]  # trigger span positions (I_sks)
    q_bits: int = 8      # 8: Q is quantized (Eq. 2, third line); 0: Q stays unquantized
    kv_bits: int = 8     # 8 or 4: width of the ordinary K/V rows (Table 1 lists 8 and 4)
    p_bits: int = 8      # 8 or 4: width of the ordinary attention probabilities
    p_log: int = 0       # 1: those probabilities through the logarithmic quantizer (power-of-two codes)
    seed: int = 0
    name: str = ""

    @property
    def d_head(self) -> int:
        return self.channels // self.heads

    @property
    def rows(self) -> int:
        return self.batch * self.n_query


def config1() -> LayerShape:
    """SD-1.5 lowest-resolution block: B=1, 8x8 latent, C=1280, W8."""
    return LayerShape(1, 64, 1280, 8, 77, 768, 8, 0, (5,), seed=0, name="config1_sd15_lowres_w8")


def config2() -> LayerShape:
    """SD-1.5 highest-resolution block: CFG pair, 64x64 latent, C=320, W4 group 128."""
    return LayerShape(2, 4096, 320, 8, 77, 768, 4, 128, (4, 5), seed=0, name="config2_sd15_highres_w4")


def config3_layers() -> List[LayerShape]:
    """All 16 cross-attention layers of one SD-1.5 UNet step (5/5/5/1 split over resolutions)."""
    shapes = [(4096, 320)] * 5 + [(1024, 640)] * 5 + [(256, 1280)] * 5 + [(64, 1280)]
    out = []
    for i, (n, c) in enumerate(shapes):
        out.append(LayerShape(2, n, c, 8, 77, 768, 4, 128, (4, 5), seed=i, name=f"config3_layer{i:02d}_N{n}_C{c}"))
    return out


def config4_layers() -> List[LayerShape]:
    """SDXL-shaped layers: d_head 64, context width 2048, three trigger sub-tokens."""
    return [
        LayerShape(2, 4096, 640, 10, 77, 2048, 4, 128, (3, 4, 5), seed=0, name="config4_sdxl_N4096_C640"),
        LayerShape(2, 1024, 1280, 20, 77, 2048, 4, 128, (3, 4, 5), seed=1, name="config4_sdxl_N1024_C1280"),
    ]


def shrink(shape: LayerShape, n_query: int) -> LayerShape:
    """Same layer with fewer query rows (rows are independent, so this is a prefix of the problem
    only in shape, not in values: the generator is re-drawn)."""
    return replace(shape, n_query=n_query, name=shape.name + f"_n{n_query}")


def _f16(a: np.ndarray) -> np.ndarray:
    return a.astype(np.float16)


def make_mask(shape: LayerShape, trigger: Sequence[int] | None = None) -> np.ndarray:
    trig = shape.trigger if trigger is None else tuple(trigger)
    m = np.zeros((shape.batch, shape.n_ctx), dtype=np.uint8)
    for j in trig:
        m[:, j] = 1
    return m


def make_weights(channels: int, ctx_dim: int, rng: np.random.Generator) -> Dict[str, np.ndarray]:
    """W_q, W_k, W_v, W_out, b_out in that order from ``rng``."""
    def w(n_out, k_in):
        return (rng.standard_normal((n_out, k_in)) / np.sqrt(k_in)).astype(np.float32)
    out = {}
    out["Wq"] = w(channels, channels)
    out["Wk"] = w(channels, ctx_dim)
    out["Wv"] = w(channels, ctx_dim)
    out["Wout"] = w(channels, channels)
    out["bout"] = (0.1 * rng.standard_normal(channels)).astype(np.float32)
    return out


def make_activations(shape: LayerShape, rng: np.random.Generator, mask: np.ndarray,
                     keep_f32: bool = False) -> Dict[str, np.ndarray]:
    """X (with outlier channels) then ctx (trigger rows x3) from ``rng``."""
    B, N, C, T, Dc = shape.batch, shape.n_query, shape.channels, shape.n_ctx, shape.ctx_dim
    X = rng.standard_normal((B, N, C)).astype(np.float32)
    n_outlier = max(1, int(round(0.01 * C)))
    idx = rng.choice(C, size=n_outlier, replace=False)
    X[:, :, idx] *= 20.0
    ctx = rng.standard_normal((B, T, Dc)).astype(np.float32)
    ctx = np.where(mask[:, :, None] != 0, ctx * 3.0, ctx).astype(np.float32)
    out = {"X": _f16(X), "ctx": _f16(ctx), "outlier_channels": np.sort(idx)}
    if keep_f32:
        out["X_f32"] = X
        out["ctx_f32"] = ctx
    return out


def make_layer(shape: LayerShape, keep_f32: bool = False) -> Dict[str, np.ndarray]:
    """Everything one layer needs: X, ctx (fp16), fp32 weights and bias, trigger mask."""
    rng = np.random.default_rng(shape.seed)
    mask = make_mask(shape)
    out = make_activations(shape, rng, mask, keep_f32=keep_f32)
    out.update(make_weights(shape.channels, shape.ctx_dim, rng))
    out["mask"] = mask
    return out


# ----------------------------------------------------------------------------------------------
# Multi-checkpoint serving sweep (config 5)
# ----------------------------------------------------------------------------------------------

@dataclass
class Checkpoint:
    ckpt_id: int
    trigger: Tuple[int, ...]                 # contiguous span of 1-3 sub-tokens, never position 0
    weights: Dict[str, np.ndarray] = field(repr=False, default_factory=dict)


def make_checkpoint(ckpt_id: int, channels: int, ctx_dim: int, n_ctx: int = 77) -> Checkpoint:
    """Weights from seed 1000+id; trigger span length 1..3 starting in [1, T-len]."""
    rng = np.random.default_rng(1000 + ckpt_id)
    span = int(rng.integers(1, 4))
    start = int(rng.integers(1, n_ctx - span + 1))
    weights = make_weights(channels, ctx_dim, rng)
    return Checkpoint(ckpt_id, tuple(range(start, start + span)), weights)


def make_request_batch(n_requests: int, n_checkpoints: int, seed: int) -> np.ndarray:
    """Checkpoint id of each request, uniform over the repository."""
    rng = np.random.default_rng(50_000 + seed)
    return rng.integers(0, n_checkpoints, size=n_requests).astype(np.int64)


def make_request_activations(ckpt: Checkpoint, n_query: int, channels: int, ctx_dim: int,
                             n_ctx: int, seed: int) -> Dict[str, np.ndarray]:
    """One request = one sequence (batch 1) with its own X, ctx and the checkpoint's trigger mask."""
    shape = LayerShape(1, n_query, channels, 8, n_ctx, ctx_dim, 4, 128, ckpt.trigger, seed=seed)
    rng = np.random.default_rng(70_000 + seed)
    mask = make_mask(shape)
    out = make_activations(shape, rng, mask)
    out["mask"] = mask
    return out
