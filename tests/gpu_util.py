"""Helpers for the GPU parity tests: run the CUDA library through its C ABI and the fp64 checker on the same inputs."""
from __future__ import annotations

import numpy as np

from oracle import gswa_oracle as orc
from paper_2409_06206_b200 import binding as gb
from paper_2409_06206_b200.inputs import LayerConfig, layer_groups, make_inputs

GRADS = ("dx", "dw_qkv", "db_qkv", "dw_proj", "db_proj", "dbias_table")
TOL = {"f32": 1e-4, "bf16": 2e-2}   # max |gpu - ref| / max |ref| per tensor


def to_device(a: np.ndarray, dtype: str):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def run_gpu(cfg: LayerConfig, inp: dict, flags: int = 0, backward: bool = True, layer: int = 0,
            use_bias: bool = True, inference: bool = False, as_float32: bool = False):
    """One forward (+ backward) through the C ABI.  Returns float64 numpy arrays (float32 on request: the
    largest workloads would otherwise hold several GB of host memory)."""
    import torch
    B = inp["x"].shape[0]
    desc = gb.Desc.from_config(cfg, layer=layer, batch=B, flags=flags)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    dev = {k: to_device(v, cfg.dtype) for k, v in inp.items()}
    saved_b, fwd_b, infer_b, bwd_b = gb.gswa_workspace_query(desc)
    y = torch.empty(inp["x"].shape, dtype=tdt, device="cuda")
    saved = None if inference else torch.empty(max(saved_b, 16), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(max(infer_b if inference else fwd_b, bwd_b, 16), dtype=torch.uint8, device="cuda")
    b_qkv = dev["b_qkv"] if use_bias else None
    b_proj = dev["b_proj"] if use_bias else None
    gb.gswa_forward(desc, dev["x"], dev["w_qkv"], b_qkv, dev["w_proj"], b_proj, dev["bias_table"], y, saved, scratch)
    gb.gswa_scratch_status(desc, scratch)
    ndt = np.float32 if as_float32 else np.float64
    out = {"y": y.float().cpu().numpy().astype(ndt)}
    if backward and not inference:
        C, M, nh = cfg.C, cfg.window, cfg.num_heads
        g = {"dx": torch.empty_like(y),
             "dw_qkv": torch.full((cfg.qkv_rows, C), 7.0, device="cuda"), "db_qkv": torch.full((cfg.qkv_rows,), 7.0, device="cuda"),
             "dw_proj": torch.full((C, cfg.v_cols), 7.0, device="cuda"), "db_proj": torch.full((C,), 7.0, device="cuda"),
             "dbias_table": torch.full(((2 * M - 1) ** 2, nh), 7.0, device="cuda")}
        gb.gswa_backward(desc, dev["x"], dev["w_qkv"], b_qkv, dev["w_proj"], dev["bias_table"], saved, dev["dy"],
                         g["dx"], g["dw_qkv"], g["db_qkv"], g["dw_proj"], g["db_proj"], g["dbias_table"], scratch)
        gb.gswa_scratch_status(desc, scratch)
        for k, v in g.items():
            out[k] = v.float().cpu().numpy().astype(ndt)
    torch.cuda.synchronize()
    return out


def run_oracle(cfg: LayerConfig, inp: dict, backward: bool = True, layer: int = 0, chunk: int = 8):
    gh, gs = layer_groups(cfg, layer)
    args = (inp["w_qkv"], inp["b_qkv"], inp["w_proj"], inp["b_proj"], inp["bias_table"], cfg.window, gh, gs)
    kw = dict(qk_dim=cfg.qk_dim or None, v_dim=cfg.v_dim or None)
    if not backward:
        y, _ = orc.forward(inp["x"], *args, keep=False, **kw)
        return {"y": y}
    y, g = orc.forward_backward_chunked(inp["x"], *args, inp["dy"], chunk=chunk, **kw)
    g["y"] = y
    return g


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.abs(ref).max())
    if den == 0.0:
        return float(np.abs(got).max())
    return float(np.abs(got - ref).max() / den)


def split_blocks(t: dict, C: int) -> dict:
    """The q-, k- and v-row blocks of dw_qkv and db_qkv as tensors of their own, so that each is measured
    against its own largest entry (the v rows are much larger than the q and k rows and would hide them).
    The key-bias gradient is identically zero (adding a constant to every key shifts each score row
    uniformly), so db_qkv_k stays out: it is covered by the whole-tensor comparison of db_qkv."""
    out = dict(t)
    if "dw_qkv" in t:
        for i, n in enumerate("qkv"):
            out["dw_qkv_" + n] = t["dw_qkv"][i * C:(i + 1) * C]
    if "db_qkv" in t:
        out["db_qkv_q"] = t["db_qkv"][0:C]
        out["db_qkv_v"] = t["db_qkv"][2 * C:3 * C]
    return out


def assert_close(got: dict, ref: dict, dtype: str, names=None, tol=None, blocks_of: int = 0):
    """`blocks_of` = C adds the q / k / v row blocks of dw_qkv and db_qkv as separately measured tensors."""
    tol = TOL[dtype] if tol is None else tol
    if blocks_of:
        got, ref = split_blocks(got, blocks_of), split_blocks(ref, blocks_of)
    errs = {n: rel_err(got[n], ref[n]) for n in (names or ref.keys()) if n in got}
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, "beyond tolerance %g: %s (all: %s)" % (tol, bad, errs)
    return errs


def excited(name, B, H, W, C, nh, gh, gs, seed, dtype="bf16"):
    """A layer whose attention scores are far from uniform: q k^T / sqrt(d) has standard deviation about one
    (weights ~ N(0, 1/C)) and the relative-position table about 0.7, so that a mistake in the score path
    (bias gather, scale, mask) moves the outputs and gradients far beyond the tolerance."""
    return LayerConfig(name, B, H, W, C, nh, 8, gh, gs, dtype=dtype, seed=seed, bias_std=0.1,
                       w_std=float(C) ** -0.5, table_std=0.7)


EXCITED = [
    excited("x180", 2, 16, 16, 180, 6, (3, 3), (0, 4), seed=41),
    excited("x60", 2, 16, 24, 60, 6, (3, 3), (4, 0), seed=42),
    excited("x192-12heads", 1, 16, 16, 192, 12, (6, 6), (0, 3), seed=43),
]
