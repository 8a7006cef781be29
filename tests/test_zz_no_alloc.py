"""gswa_forward_static: the inference forward for callers that cannot allocate device memory (a plug-in
inside an application that owns all of it, a C program with no GPU allocator, a loop where cudaMalloc's
device-wide synchronisation is not acceptable).  Its intermediates live in a fixed array inside the
library's device image instead of a caller-provided scratch buffer.  Called through the C ABI twice in
a row, it must give what gswa_forward gives in inference mode (same tolerance as the parity tests), the
second call included, since every call reuses the array with the previous call's contents still in it.
Collected last on purpose, so that a run which stops at the first failure has already run the rest."""
import numpy as np
import pytest

from paper_2409_06206_b200 import binding as gb
from paper_2409_06206_b200 import build as gbuild
from paper_2409_06206_b200.inputs import LayerConfig, make_inputs

from gpu_util import TOL, rel_err, run_gpu, to_device

pytestmark = pytest.mark.gpu

CASES = [
    LayerConfig("na-bf16", 2, 16, 24, 180, 6, 8, (3, 3), (0, 4), dtype="bf16", seed=31, bias_std=0.1),
    LayerConfig("na-f32", 1, 16, 16, 60, 6, 8, (3, 3), (4, 0), dtype="f32", seed=32, bias_std=0.1),
]


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


@pytest.mark.parametrize("cfg", CASES, ids=[c.name for c in CASES])
def test_static_scratch_forward_matches_forward_twice(cfg):
    import torch
    inp = make_inputs(cfg)
    inp2 = make_inputs(LayerConfig(**{**cfg.__dict__, "seed": cfg.seed + 100}))
    desc = gb.Desc.from_config(cfg)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    for which in (inp, inp2):                      # two calls in a row, different data each time
        ref = run_gpu(cfg, which, backward=False, inference=True)["y"]
        dev = {k: to_device(v, cfg.dtype) for k, v in which.items()}
        y = torch.full(which["x"].shape, float("nan"), dtype=tdt, device="cuda")
        gb.gswa_forward_static(desc, dev["x"], dev["w_qkv"], dev["b_qkv"], dev["w_proj"], dev["b_proj"],
                               dev["bias_table"], y)
        torch.cuda.synchronize()
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert rel_err(got, ref) <= TOL[cfg.dtype]


def test_static_scratch_rejects_layers_beyond_its_size():
    big = gb.Desc(64, 64, 64, 180, 6, 8, (3, 3), (0, 4), "bf16")
    assert gb.gswa_workspace_query(big)[2] > gb.STATIC_SCRATCH_BYTES
    n0 = gb.gswa_launch_count()
    with pytest.raises(gb.GswaError) as e:
        gb.gswa_forward_static(big, 256, 256, None, 256, None, 256, 256, stream=0)
    assert e.value.status == -5
    assert gb.gswa_launch_count() == n0
