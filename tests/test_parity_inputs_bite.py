"""Do the score-exciting parity inputs bite?  CPU only.

The default workload recipe (weights and table ~ N(0, 0.02^2)) gives a nearly uniform softmax, under which a
wrong bias gather or a mis-scaled query moves y and the gradients by about the bf16 tolerance.  The GPU parity
tests therefore also run the layers of gpu_util.EXCITED, and compare the q / k / v row blocks of dw_qkv and
db_qkv separately.  This file proves that those cases would notice a mistake in the score path: each case
plants one mistake in a copy of the CPU checker and requires that at least one compared tensor moves by at
least five times the bf16 tolerance (Sec. "Group Shifted Window Attention", Eq. 6; Sec. "Learnable Relative
Shifted Bias")."""
import inspect
import types

import numpy as np
import pytest

from oracle import gswa_oracle as orc
from paper_2409_06206_b200.inputs import layer_groups, make_inputs

from gpu_util import EXCITED, TOL, rel_err, split_blocks

SRC = inspect.getsource(orc)

MISTAKES = [
    ("bias-dropped", "S = S + table[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]", "pass"),
    ("bias-index-transposed", "rel = (a[:, None] - a[None, :] + M - 1) * (2 * M - 1) + (c[:, None] - c[None, :] + M - 1)",
     "rel = (a[None, :] - a[:, None] + M - 1) * (2 * M - 1) + (c[None, :] - c[:, None] + M - 1)"),
    ("bias-of-another-head", "S = S + table[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]",
     "S = S + np.roll(table, 1, axis=1)[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]"),
    ("bias-row-off-by-one", "S = S + table[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]",
     "S = S + np.roll(table, 1, axis=0)[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]"),
    ("scores-dropped", 'S = np.einsum("nphd,nqhd->nhpq", qw, kw)', 'S = 0.0 * np.einsum("nphd,nqhd->nhpq", qw, kw)'),
    ("query-scale-wrong", "scale = float(dq) ** -0.5", "scale = 1.3 * float(dq) ** -0.5"),
    ("mask-dropped", "S = (S.reshape(B, nW, gh, N, N) + mask[None, :, None]).reshape(B * nW, gh, N, N)", "pass"),
    ("dq-zeroed", "dqkv = np.concatenate([dq * scale, dk, dv], axis=-1)", "dqkv = np.concatenate([dq * 0.0, dk, dv], axis=-1)"),
    ("dk-zeroed", "dqkv = np.concatenate([dq * scale, dk, dv], axis=-1)", "dqkv = np.concatenate([dq * scale, dk * 0.0, dv], axis=-1)"),
]


def _run(mod, cfg, inp):
    gh, gs = layer_groups(cfg, 0)
    y, g = mod.forward_backward_chunked(inp["x"], inp["w_qkv"], inp["b_qkv"], inp["w_proj"], inp["b_proj"],
                                        inp["bias_table"], cfg.window, gh, gs, inp["dy"], chunk=2)
    g["y"] = y
    return split_blocks(g, cfg.C)


@pytest.mark.parametrize("cfg", EXCITED, ids=[c.name for c in EXCITED])
def test_score_path_mistakes_move_the_compared_tensors(cfg):
    inp = make_inputs(cfg)
    ref = _run(orc, cfg, inp)
    for name, old, new in MISTAKES:
        assert SRC.count(old) >= 1, name
        mod = types.ModuleType("gswa_oracle_mistake")
        exec(compile(SRC.replace(old, new), "gswa_oracle_mistake", "exec"), mod.__dict__)
        with np.errstate(all="ignore"):
            bad = _run(mod, cfg, inp)
        moved = {n: rel_err(bad[n], ref[n]) for n in ref}
        worst = max(moved.values())
        assert worst >= 5 * TOL["bf16"], "%s on %s moves nothing by more than %.3g: %s" % (name, cfg.name, worst, moved)
        if name in ("bias-dropped", "bias-index-transposed", "scores-dropped", "query-scale-wrong"):
            # a forward mistake must show in the forward output itself, not only in a gradient
            assert moved["y"] >= 5 * TOL["bf16"], (name, cfg.name, moved["y"])
