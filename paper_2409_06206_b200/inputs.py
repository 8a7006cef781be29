"""Seeded synthetic inputs for one GSWA layer.

This module only draws random tensors and rounds them to a storage type.  It
holds none of the method's arithmetic, so both the CUDA path and the CPU
checker can be fed from it without sharing anything else.

Recipe (stands in for the paper's DIV2K training patches and test images,
Sec. "Experimental Setup"): activations entering the attention layer follow a
LayerNorm (Eq. 4), hence x ~ N(0,1); projection weights and the
relative-position bias table ~ N(0, 0.02^2); projection biases zero unless a
test asks otherwise; upstream gradient dy ~ N(0,1).  Tests that must excite
the attention scores (a softmax far from uniform) raise the weight and table
standard deviations through `w_std` / `table_std`.  For bf16 workloads every
sample is rounded to the nearest bf16 value (ties to even) before anybody sees
it, and returned as float32 holding exactly that value.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Tuple

import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    """Shape of one GSWA layer call (notation of Sec. "Group Shifted Window Attention")."""

    name: str
    B: int
    H: int
    W: int
    C: int
    num_heads: int
    window: int                      # M
    group_heads: Tuple[int, ...]     # heads per group, consecutive
    group_shift: Tuple[int, ...]     # cyclic shift of each group (0 = plain windows)
    dtype: str = "bf16"              # "f32" | "bf16"
    seed: int = 0
    layers: int = 1                  # stacked-inference workloads call the layer this many times
    backward: bool = True
    bias_std: float = 0.0            # std of b_qkv / b_proj (0 in the paper-shaped workloads)
    w_std: float = 0.02              # std of w_qkv / w_proj
    table_std: float = 0.02          # std of the relative-position bias table
    qk_dim: int = 0                  # per-head width of Q and K (0 = head dim; Sec. "Parameter Allocation")
    v_dim: int = 0                   # per-head width of V (0 = head dim)

    @property
    def tokens(self) -> int:
        return self.B * self.H * self.W

    @property
    def head_dim(self) -> int:
        return self.C // self.num_heads

    @property
    def qkv_rows(self) -> int:
        """Rows of w_qkv: heads * (2 * qk width + v width); 3C by default."""
        d = self.head_dim
        return self.num_heads * (2 * (self.qk_dim or d) + (self.v_dim or d))

    @property
    def v_cols(self) -> int:
        """Columns of w_proj: heads * v width; C by default."""
        return self.num_heads * (self.v_dim or self.head_dim)


# The workloads the layer is measured and checked on.  Batch 16..256 and C=60
# are the paper's training batch sizes and lightweight width; 64x64 patches,
# C=180 and window 8 are the classical-SR shape of the same model family.
CONFIGS: Dict[str, LayerConfig] = {
    "c1": LayerConfig("c1", 1, 16, 16, 60, 6, 8, (3, 3), (0, 4), dtype="f32", seed=0),
    "c2": LayerConfig("c2", 64, 64, 64, 60, 6, 8, (3, 3), (0, 4), seed=2),
    "c3": LayerConfig("c3", 32, 64, 64, 180, 6, 8, (3, 3), (0, 4), seed=3),
    "cM": LayerConfig("cM", 64, 64, 64, 180, 6, 8, (3, 3), (0, 4), seed=6),
    "c4": LayerConfig("c4", 256, 64, 64, 180, 6, 8, (3, 3), (0, 4), seed=4),
    "c5": LayerConfig("c5", 1, 512, 512, 180, 6, 8, (3, 3), (0, 4), seed=5, layers=6, backward=False),
}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Upper 16 bits of already-bf16-representable float32 values, as uint16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


_TENSOR_STREAM = {"x": 1, "w_qkv": 2, "b_qkv": 3, "w_proj": 4, "b_proj": 5, "bias_table": 6, "dy": 7,
                  "ln1_g": 8, "ln1_b": 9, "ln2_g": 10, "ln2_b": 11, "w_fc1": 12, "b_fc1": 13, "w_fc2": 14, "b_fc2": 15,
                  "w_heads": 16, "b_heads": 17}


def _normal(seed: int, layer: int, name: str, shape, std: float) -> np.ndarray:
    ss = np.random.SeedSequence([int(seed), int(layer), _TENSOR_STREAM[name]])
    rng = np.random.Generator(np.random.Philox(ss))
    out = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out


def make_inputs(cfg: LayerConfig, layer: int = 0, batch: int | None = None,
                tensors=("x", "w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table", "dy")) -> Dict[str, np.ndarray]:
    """Draw the tensors of one layer call as float32 arrays.

    `batch` overrides cfg.B with a smaller leading count (the first `batch`
    images of the full draw are NOT reproduced; it is a separate, equally
    distributed draw) -- used for bounded CPU samples.
    """
    B = cfg.B if batch is None else int(batch)
    C, M, nh = cfg.C, cfg.window, cfg.num_heads
    shapes = {
        "x": ((B, cfg.H, cfg.W, C), 1.0),
        "w_qkv": ((cfg.qkv_rows, C), cfg.w_std),
        "b_qkv": ((cfg.qkv_rows,), cfg.bias_std),
        "w_proj": ((C, cfg.v_cols), cfg.w_std),
        "b_proj": ((C,), cfg.bias_std),
        "bias_table": (((2 * M - 1) ** 2, nh), cfg.table_std),
        "dy": ((B, cfg.H, cfg.W, C), 1.0),
    }
    out = {}
    for name in tensors:
        shape, std = shapes[name]
        if std == 0.0:
            a = np.zeros(shape, dtype=np.float32)
        else:
            a = _normal(cfg.seed, layer, name, shape, std)
        if cfg.dtype == "bf16":
            a = round_to_bf16(a)
        out[name] = a
    return out


def make_layer_inputs(cfg: LayerConfig, mlp_hidden: int, layer: int = 0, batch: int | None = None) -> Dict[str, np.ndarray]:
    """The tensors of one whole layer call (attention inside LayerNorm + skip, optionally followed by the MLP):
    those of make_inputs plus LayerNorm scales ~ 1 + N(0, 0.1^2), shifts ~ N(0, 0.1^2), and the two
    fully-connected layers ~ N(0, w_std^2) with biases ~ N(0, bias_std^2).  Here x is NOT normalised input: it is
    drawn ~ N(0.5, 2^2) so that the LayerNorm has something to do."""
    out = make_inputs(cfg, layer=layer, batch=batch)
    C = cfg.C
    out["x"] = (out["x"] * np.float32(2.0) + np.float32(0.5)).astype(np.float32)
    shapes = {"ln1_g": ((C,), 0.1, 1.0), "ln1_b": ((C,), 0.1, 0.0), "ln2_g": ((C,), 0.1, 1.0), "ln2_b": ((C,), 0.1, 0.0),
              "w_fc1": ((mlp_hidden, C), cfg.w_std, 0.0), "b_fc1": ((mlp_hidden,), cfg.bias_std, 0.0),
              "w_fc2": ((C, mlp_hidden), cfg.w_std, 0.0), "b_fc2": ((C,), cfg.bias_std, 0.0)}
    for name, (shape, std, mean) in shapes.items():
        if 0 in shape:
            continue
        a = _normal(cfg.seed, layer, name, shape, std) if std > 0 else np.zeros(shape, np.float32)
        out[name] = (a + np.float32(mean)).astype(np.float32)
    if cfg.dtype == "bf16":
        out = {k: round_to_bf16(v) for k, v in out.items()}
    return out


def make_sliced_inputs(cfg: LayerConfig, layer: int = 0, batch: int | None = None) -> Dict[str, np.ndarray]:
    """The tensors of a channel-sliced layer call: per-head projections w_heads [heads, 2*qk + ds, ds] (ds = C / heads
    input channels per head; rows q | k | v) and b_heads, in place of w_qkv / b_qkv.  Weights ~ N(0, w_std^2 * heads)
    (a head sees 1/heads of the channels)."""
    out = make_inputs(cfg, layer=layer, batch=batch, tensors=("x", "w_proj", "b_proj", "bias_table", "dy"))
    nh, ds = cfg.num_heads, cfg.head_dim
    dq = cfg.qk_dim or ds
    out["w_heads"] = _normal(cfg.seed, layer, "w_heads", (nh, 2 * dq + ds, ds), cfg.w_std * float(nh) ** 0.5)
    out["b_heads"] = _normal(cfg.seed, layer, "b_heads", (nh, 2 * dq + ds), cfg.bias_std) if cfg.bias_std > 0 else np.zeros((nh, 2 * dq + ds), np.float32)
    if cfg.dtype == "bf16":
        out = {k: round_to_bf16(v) for k, v in out.items()}
    return out


def layer_groups(cfg: LayerConfig, layer: int) -> Tuple[Tuple[int, ...], Tuple[int, ...]]:
    """Head-group split of the `layer`-th stacked layer: odd layers swap which group shifts."""
    if layer % 2 == 0:
        return cfg.group_heads, cfg.group_shift
    return cfg.group_heads, tuple(reversed(cfg.group_shift))
