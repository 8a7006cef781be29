"""GPU parity of the layer around GSWA (Sec. "Agile Swin Transformer Block", Eq. 4 and Eq. 5) through the C ABI
against the fp64 CPU checker: LayerNorm + attention + skip, with and without the MLP, forward and backward, on the
tensor-core and the shape-generic attention paths.  Tolerances as for the attention itself."""
import dataclasses

import numpy as np
import pytest

from oracle import astl_oracle as ao
from paper_2409_06206_b200 import binding as gb
from paper_2409_06206_b200 import build as gbuild
from paper_2409_06206_b200.inputs import LayerConfig, layer_groups, make_layer_inputs

from gpu_util import TOL, rel_err, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


def _mk(name, B, H, W, C, nh, M, gh, gs, dtype, seed=5, **kw):
    return LayerConfig(name, B, H, W, C, nh, M, gh, gs, dtype=dtype, seed=seed, bias_std=0.1, w_std=float(C) ** -0.5,
                       table_std=0.3, **kw)


CASES = [
    (_mk("l0", 1, 16, 16, 60, 6, 8, (3, 3), (0, 4), "f32"), 0),
    (_mk("l1", 2, 16, 16, 60, 6, 8, (3, 3), (0, 4), "f32"), 120),
    (_mk("l2", 2, 16, 24, 180, 6, 8, (3, 3), (0, 4), "bf16"), 0),
    (_mk("l3", 2, 16, 24, 180, 6, 8, (3, 3), (4, 0), "bf16"), 360),
    (_mk("l4", 1, 24, 16, 60, 6, 8, (3, 3), (0, 3), "bf16"), 120),
    (_mk("l5", 1, 24, 24, 180, 6, 12, (3, 3), (0, 6), "bf16", qk_dim=16), 360),
]


def run_layer_gpu(cfg, hidden, inp, inference=False):
    import torch
    desc = gb.Desc.from_config(cfg, batch=inp["x"].shape[0])
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    dev = {k: to_device(v, cfg.dtype) for k, v in inp.items()}
    saved_b, fwd_b, infer_b, bwd_b = gb.gswa_astl_workspace_query(desc, hidden)
    y = torch.full(inp["x"].shape, float("nan"), dtype=tdt, device="cuda")
    saved = None if inference else torch.empty(max(saved_b, 16), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(max(infer_b if inference else fwd_b, bwd_b, 256), dtype=torch.uint8, device="cuda")
    gb.gswa_astl_forward(desc, hidden, dev["x"], dev, y, saved, scratch)
    gb.gswa_scratch_status(desc, scratch)
    out = {"y": y.float().cpu().numpy().astype(np.float64)}
    if inference:
        return out
    grads = {"d" + n: torch.full(dev[n].shape, 7.0, device="cuda") for n in gb.ASTL_PARAMS if n in dev}
    dx = torch.empty_like(y)
    gb.gswa_astl_backward(desc, hidden, dev["x"], dev, saved, dev["dy"], dx, grads, scratch)
    gb.gswa_scratch_status(desc, scratch)
    torch.cuda.synchronize()
    out["dx"] = dx.float().cpu().numpy().astype(np.float64)
    for k, v in grads.items():
        out[k] = v.cpu().numpy().astype(np.float64)
    return out


def run_layer_oracle(cfg, hidden, inp):
    gh, gs = layer_groups(cfg, 0)
    y, cache = ao.astl_forward(inp["x"], inp, cfg.window, gh, gs, qk_dim=cfg.qk_dim or None, v_dim=cfg.v_dim or None,
                               with_mlp=hidden > 0)
    g = ao.astl_backward(cache, inp["dy"])
    g["y"] = y
    return g


@pytest.mark.parametrize("cfg,hidden", CASES, ids=["%s-h%d" % (c.name, h) for c, h in CASES])
def test_layer_forward_backward(cfg, hidden):
    inp = make_layer_inputs(cfg, hidden)
    got = run_layer_gpu(cfg, hidden, inp)
    ref = run_layer_oracle(cfg, hidden, inp)
    errs = {n: rel_err(got[n], ref[n]) for n in ref}
    bad = {n: e for n, e in errs.items() if not e <= TOL[cfg.dtype]}
    assert not bad, "beyond %g: %s (all: %s)" % (TOL[cfg.dtype], bad, errs)
    want = {"y", "dx", "dln1_g", "dln1_b", "dw_qkv", "db_qkv", "dw_proj", "db_proj", "dbias_table"}
    if hidden:
        want |= {"dln2_g", "dln2_b", "dw_fc1", "db_fc1", "dw_fc2", "db_fc2"}
    assert set(errs) == want
    inf = run_layer_gpu(cfg, hidden, inp, inference=True)
    assert rel_err(inf["y"], got["y"]) == 0.0
