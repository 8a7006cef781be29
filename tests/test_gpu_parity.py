"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU checker on the same
seeded inputs.  Index maps must be bit-exact; tensors within 1e-4 (f32) / 2e-2 (bf16) of the checker,
measured as max |gpu - ref| / max |ref| per tensor."""
import dataclasses

import numpy as np
import pytest

from oracle import gswa_oracle as orc
from paper_2409_06206_b200 import binding as gb
from paper_2409_06206_b200 import build as gbuild
from paper_2409_06206_b200.inputs import CONFIGS, LayerConfig, make_inputs

from gpu_util import EXCITED, GRADS, assert_close, rel_err, run_gpu, run_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


@pytest.mark.parametrize("H,W,M,s", [(16, 16, 8, 4), (16, 24, 8, 3), (64, 64, 8, 4), (8, 8, 8, 7), (24, 12, 4, 1),
                                     (36, 24, 12, 6), (16, 16, 8, 0)])
def test_index_maps_bit_exact(H, W, M, s):
    import torch
    d = gb.Desc(1, H, W, 12, 2, M, (1, 1), (0, s), "f32")
    N = M * M
    bufs = [torch.full((H * W,), -1, dtype=torch.int32, device="cuda") for _ in range(4)]
    rel = torch.full((N * N,), -1, dtype=torch.int32, device="cuda")
    gb.gswa_index_maps(d, 1, *bufs, rel)
    torch.cuda.synchronize()
    win, slot, region, rel_ref = orc.index_maps(H, W, M, s)
    got = [b.cpu().numpy() for b in bufs]
    assert np.array_equal(got[0], win.ravel())
    assert np.array_equal(got[1], slot.ravel())
    assert np.array_equal(got[2], region.ravel())
    token_of = np.empty(H * W, np.int32)
    token_of[win.ravel() * N + slot.ravel()] = np.arange(H * W, dtype=np.int32)
    assert np.array_equal(got[3], token_of)
    assert np.array_equal(rel.cpu().numpy(), rel_ref.ravel())


@pytest.mark.parametrize("B,H,W,s,dtype,C,nh", [(2, 16, 16, 4, "bf16", 64, 2), (3, 16, 24, 3, "bf16", 180, 6), (1, 64, 64, 4, "bf16", 60, 6),
                                               (2, 8, 8, 7, "bf16", 64, 4), (1, 8, 16, 1, "bf16", 96, 6), (2, 24, 12, 1, "f32", 12, 2)])
def test_debug_index_maps_of_the_running_path_bit_exact(B, H, W, s, dtype, C, nh):
    """The maps as the kernels that run the layer compute them (on the bf16 path: the window set-up and the
    fragment-wise bias rows of the tensor-core attention kernels), over the whole batch, bit for bit."""
    import torch
    M = 8 if dtype == "bf16" else 4
    d = gb.Desc(B, H, W, C, nh, M, (nh - 1, 1), (0, s), dtype)
    N, nW = M * M, (H // M) * (W // M)
    win_id = torch.full((B * H * W,), -1, dtype=torch.int32, device="cuda")
    slot = torch.full((H * W,), -1, dtype=torch.int32, device="cuda")
    region = torch.full((H * W,), -1, dtype=torch.int32, device="cuda")
    rel = torch.full((N * N,), -1, dtype=torch.int32, device="cuda")
    gb.gswa_debug_index_maps(d, 1, win_id, slot, region, rel)
    torch.cuda.synchronize()
    win, slot_ref, region_ref, rel_ref = orc.index_maps(H, W, M, s)
    want = (np.arange(B, dtype=np.int32)[:, None] * nW + win.ravel()[None, :]).ravel()
    assert np.array_equal(win_id.cpu().numpy(), want)
    assert np.array_equal(slot.cpu().numpy(), slot_ref.ravel())
    assert np.array_equal(region.cpu().numpy(), region_ref.ravel())
    assert np.array_equal(rel.cpu().numpy(), rel_ref.ravel())


def test_a_bounded_wait_that_runs_out_is_reported_and_harmless():
    """A device-side wait expires on purpose (a barrier nobody arrives on, about two thousand polls): the error word
    is set, gswa_scratch_status reports GSWA_ERR_DEVICE, and the next call on the same scratch is correct."""
    import torch
    cfg = SWEEP[8]
    inp = make_inputs(cfg)
    desc = gb.Desc.from_config(cfg)
    scratch = torch.zeros(max(gb.gswa_workspace_query(desc)[1:]), dtype=torch.uint8, device="cuda")
    gb.gswa_scratch_status(desc, scratch)                       # clean
    gb.gswa_debug_expire_wait(desc, scratch)
    with pytest.raises(gb.GswaError) as e:
        gb.gswa_scratch_status(desc, scratch)
    assert e.value.status == -7
    torch.cuda.synchronize()
    got = run_gpu(cfg, inp)                                     # the context is intact
    assert_close(got, run_oracle(cfg, inp), cfg.dtype)
    # a forward call on the same scratch clears the word
    dev = {k: __import__("gpu_util").to_device(v, cfg.dtype) for k, v in inp.items()}
    y = torch.empty(inp["x"].shape, dtype=torch.bfloat16, device="cuda")
    gb.gswa_forward(desc, dev["x"], dev["w_qkv"], dev["b_qkv"], dev["w_proj"], dev["b_proj"], dev["bias_table"], y, None, scratch)
    gb.gswa_scratch_status(desc, scratch)


def test_config1_f32_forward_backward():
    cfg = CONFIGS["c1"]
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp)
    ref = run_oracle(cfg, inp)
    errs = assert_close(got, ref, "f32")
    assert set(errs) == set(GRADS) | {"y"}


def _mk(name, B, H, W, C, nh, M, gh, gs, dtype, seed=1):
    return LayerConfig(name, B, H, W, C, nh, M, gh, gs, dtype=dtype, seed=seed, bias_std=0.1)


SWEEP = [
    _mk("s0", 2, 8, 8, 12, 2, 8, (2,), (0,), "f32"),
    _mk("s1", 1, 8, 8, 12, 2, 8, (1, 1), (3, 7), "f32"),
    _mk("s2", 2, 16, 24, 60, 6, 8, (3, 3), (0, 4), "f32"),
    _mk("s3", 1, 24, 16, 60, 6, 8, (1, 2, 3), (1, 0, 5), "f32"),
    _mk("s4", 2, 16, 16, 180, 6, 8, (3, 3), (4, 0), "f32"),
    _mk("s5", 1, 24, 24, 24, 2, 12, (1, 1), (0, 6), "f32"),
    _mk("s6", 3, 12, 8, 16, 4, 4, (2, 2), (0, 2), "f32"),
    _mk("s7", 2, 16, 24, 60, 6, 8, (3, 3), (0, 4), "bf16"),
    _mk("s8", 1, 24, 16, 180, 6, 8, (3, 3), (4, 0), "bf16"),
    _mk("s9", 2, 16, 16, 180, 6, 8, (2, 4), (3, 0), "bf16"),
    _mk("s10", 3, 24, 40, 60, 6, 8, (6,), (4,), "bf16"),
    _mk("s11", 5, 16, 16, 64, 2, 8, (1, 1), (0, 1), "bf16"),
    _mk("s12", 1, 24, 24, 36, 3, 12, (1, 2), (0, 6), "bf16"),
    # more heads than the attention kernels have one-head work units for: their multi-head CTAs run
    _mk("s13", 2, 16, 24, 192, 12, 8, (6, 6), (0, 4), "bf16"),
    _mk("s14", 1, 24, 16, 180, 10, 8, (5, 5), (3, 0), "bf16"),
    _mk("s15", 2, 16, 16, 240, 12, 8, (4, 8), (4, 1), "bf16"),
]


# The paper's own layer settings (Sec. "Parameter Allocation", Sec. "Experimental Setup"): Q and K narrowed to 16
# channels (read per head, and read as the total over heads), window 12; plus the window-12 layer at C = 180 whose
# backward needs the most shared memory of all supported shapes.
PAPER_SHAPES = [
    dataclasses.replace(_mk("p0", 2, 24, 24, 180, 6, 12, (3, 3), (0, 6), "f32"), qk_dim=16),
    dataclasses.replace(_mk("p1", 2, 24, 24, 180, 6, 12, (3, 3), (0, 6), "bf16"), qk_dim=16),
    dataclasses.replace(_mk("p2", 2, 24, 36, 60, 4, 12, (2, 2), (6, 0), "f32"), qk_dim=4),
    dataclasses.replace(_mk("p3", 2, 24, 36, 60, 4, 12, (2, 2), (6, 0), "bf16"), qk_dim=4),
    dataclasses.replace(_mk("p4", 1, 16, 16, 60, 6, 8, (3, 3), (0, 4), "bf16"), qk_dim=16, v_dim=12),
    _mk("p5", 1, 24, 24, 180, 6, 12, (3, 3), (0, 6), "f32"),
    _mk("p6", 1, 24, 24, 180, 6, 12, (3, 3), (0, 6), "bf16"),
]


@pytest.mark.parametrize("cfg", PAPER_SHAPES, ids=[c.name for c in PAPER_SHAPES])
def test_narrowed_qk_projections_and_window_12(cfg):
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp)
    ref = run_oracle(cfg, inp)
    assert_close(got, ref, cfg.dtype)


@pytest.mark.parametrize("cfg", SWEEP, ids=[c.name for c in SWEEP])
def test_small_shapes_forward_backward(cfg):
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp)
    ref = run_oracle(cfg, inp)
    assert_close(got, ref, cfg.dtype)


def _random_fast_path_shapes(n, seed=1234):
    """Seeded random layer shapes that the tensor-core path accepts (window 8, even head dim <= 32, padded
    attention width >= 64): odd window counts, every shift, one to four groups, all K paddings."""
    rng = np.random.default_rng(seed)
    out = []
    choices = [(64, 2), (64, 4), (96, 3), (96, 6), (120, 4), (128, 4), (128, 8), (144, 6), (180, 6), (192, 6), (224, 7),
               (240, 8), (252, 7), (56, 4), (72, 6)]
    while len(out) < n:
        C, nh = choices[int(rng.integers(len(choices)))]
        d = C // nh
        if d % 2 or d > 32 or nh * (16 if d <= 16 else 32) < 64:
            continue
        G = int(rng.integers(1, min(4, nh) + 1))
        cuts = sorted(rng.choice(np.arange(1, nh), size=G - 1, replace=False).tolist()) if G > 1 else []
        gh = tuple(int(b - a) for a, b in zip([0] + cuts, cuts + [nh]))
        gs = tuple(int(rng.integers(0, 8)) for _ in range(G))
        B, H, W = int(rng.integers(1, 4)), 8 * int(rng.integers(1, 5)), 8 * int(rng.integers(1, 6))
        out.append(_mk("r%d" % len(out), B, H, W, C, nh, 8, gh, gs, "bf16", seed=100 + len(out)))
    return out


RANDOM_SHAPES = _random_fast_path_shapes(14)


@pytest.mark.parametrize("cfg", RANDOM_SHAPES, ids=["%s-B%dx%dx%d-C%d-h%s-s%s" % (c.name, c.B, c.H, c.W, c.C, "".join(map(str, c.group_heads)),
                                                   "".join(map(str, c.group_shift))) for c in RANDOM_SHAPES])
def test_random_shapes_tensor_core_path(cfg):
    inp = make_inputs(cfg)
    ref = run_oracle(cfg, inp)
    assert_close(run_gpu(cfg, inp), ref, cfg.dtype)
    assert_close(run_gpu(cfg, inp, flags=gb.FLAG_FUSED_FWD), ref, cfg.dtype)
    assert_close(run_gpu(cfg, inp, flags=gb.FLAG_TCGEN05_ATTN), ref, cfg.dtype)
    assert_close(run_gpu(cfg, inp, flags=gb.FLAG_COPY_LOADERS), ref, cfg.dtype)


@pytest.mark.parametrize("flags", [0, gb.FLAG_FUSED_FWD, gb.FLAG_TCGEN05_ATTN, gb.FLAG_COPY_LOADERS, gb.FLAG_GENERIC],
                         ids=["default", "fused-fwd", "tcgen05-attn", "copy-loaders", "generic"])
@pytest.mark.parametrize("cfg", EXCITED, ids=[c.name for c in EXCITED])
def test_score_exciting_inputs(cfg, flags):
    """Weights ~ N(0, 1/C) and a table of std 0.7: the softmax is far from uniform, so the bias gather, the query
    scale and the mask all move y and the gradients well beyond the tolerance if they are wrong
    (tests/test_parity_inputs_bite.py proves that on the CPU).  The q / k / v row blocks of dw_qkv and db_qkv are
    measured separately, each against its own largest entry."""
    inp = make_inputs(cfg)
    ref = run_oracle(cfg, inp)
    errs = assert_close(run_gpu(cfg, inp, flags=flags), ref, cfg.dtype, blocks_of=cfg.C)
    assert {"dw_qkv_q", "dw_qkv_k", "dw_qkv_v", "db_qkv_q", "db_qkv_v"} <= set(errs)


@pytest.mark.parametrize("cfg", [SWEEP[2], SWEEP[7], SWEEP[8]], ids=["f32", "bf16-c60", "bf16-c180"])
def test_generic_kernels_forced(cfg):
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp, flags=gb.FLAG_GENERIC)
    ref = run_oracle(cfg, inp)
    assert_close(got, ref, cfg.dtype)


@pytest.mark.parametrize("cfg", [SWEEP[7], SWEEP[8], SWEEP[9], SWEEP[11]], ids=["c60", "c180", "uneven-groups", "two-heads"])
def test_fused_forward_kernel(cfg):
    """The opt-in kernel that fuses the QKV projection with the forward attention (training and inference mode)."""
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp, flags=gb.FLAG_FUSED_FWD)
    ref = run_oracle(cfg, inp)
    assert_close(got, ref, cfg.dtype)
    inf = run_gpu(cfg, inp, flags=gb.FLAG_FUSED_FWD, inference=True)
    assert rel_err(inf["y"], got["y"]) == 0.0


@pytest.mark.parametrize("cfg", [SWEEP[6], SWEEP[7], SWEEP[8], SWEEP[9], SWEEP[10]],
                         ids=["c60", "c180", "uneven-groups-odd-shift", "one-group", "two-heads-odd-window-count"])
def test_tcgen05_attention_backward(cfg):
    """The opt-in attention backward on tcgen05 (window pairs, TMEM accumulators, tiled bulk stores): windows inside
    the image, windows that wrap around its edge (even shift: four boxes; odd shift: row by row), an odd number
    of windows (the last pair holds one window), both padded head widths."""
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp, flags=gb.FLAG_TCGEN05_ATTN)
    ref = run_oracle(cfg, inp)
    assert_close(got, ref, cfg.dtype)


def test_tcgen05_attention_backward_training_shape():
    cfg = CONFIGS["c3"]
    inp = make_inputs(cfg, batch=3)
    got = run_gpu(cfg, inp, flags=gb.FLAG_TCGEN05_ATTN)
    ref = run_oracle(cfg, inp, chunk=3)
    assert_close(got, ref, cfg.dtype)


def test_null_biases_inference_mode_and_accumulate():
    import torch
    cfg = dataclasses.replace(SWEEP[7], bias_std=0.0)
    inp = make_inputs(cfg)
    ref = run_oracle(cfg, inp)
    got = run_gpu(cfg, inp, use_bias=False)
    assert_close(got, ref, cfg.dtype)
    inf = run_gpu(cfg, inp, inference=True)
    assert rel_err(inf["y"], got["y"]) == 0.0
    # accumulate flag: gradients are added to what the buffers hold (run_gpu pre-fills them with 7)
    acc = run_gpu(cfg, inp, flags=gb.FLAG_ACCUMULATE)
    for n in GRADS[1:]:
        assert rel_err(acc[n] - 7.0, ref[n]) <= 2e-2, n


def test_empty_batch_is_a_no_op():
    import torch
    cfg = SWEEP[7]
    d = gb.Desc(0, cfg.H, cfg.W, cfg.C, cfg.num_heads, cfg.window, cfg.group_heads, cfg.group_shift, "bf16")
    t = torch.zeros(64, dtype=torch.uint8, device="cuda")
    n0 = gb.gswa_launch_count()
    gb.gswa_forward(d, t, t, None, t, None, t, t, t, t)
    assert gb.gswa_launch_count() == n0


@pytest.mark.parametrize("name,batch", [("c2", 8), ("c3", 4)])
def test_training_shapes_reduced_batch(name, batch):
    """The paper-shaped training layers at a batch the checker finishes in seconds (weight gradients included)."""
    cfg = CONFIGS[name]
    inp = make_inputs(cfg, batch=batch)
    got = run_gpu(cfg, inp)
    ref = run_oracle(cfg, inp, chunk=4)
    assert_close(got, ref, cfg.dtype)


@pytest.mark.parametrize("name", ["cM", "c4"])
def test_full_size_every_tensor_against_the_checker(name):
    """Full-size launch configuration, the one bench.py times: all seven result tensors against the checker, which
    walks the whole batch a few images at a time (y and dx are compared chunk by chunk, the parameter gradients
    are summed over all chunks and compared at the end).  The weight-gradient GEMMs wrap their operand rings
    dozens of times only at this size."""
    cfg = CONFIGS[name]
    inp = make_inputs(cfg)
    got = run_gpu(cfg, inp, as_float32=True)
    gh, gs = cfg.group_heads, cfg.group_shift
    chunk, acc = 4, None
    num = {"y": 0.0, "dx": 0.0}
    den = {"y": 0.0, "dx": 0.0}
    for b0 in range(0, cfg.B, chunk):
        sl = slice(b0, b0 + chunk)
        y, cache = orc.forward(inp["x"][sl], inp["w_qkv"], inp["b_qkv"], inp["w_proj"], inp["b_proj"], inp["bias_table"],
                               cfg.window, gh, gs)
        g = orc.backward(cache, inp["dy"][sl])
        for n, r in (("y", y), ("dx", g.pop("dx"))):
            num[n] = max(num[n], float(np.abs(got[n][sl] - r).max()))
            den[n] = max(den[n], float(np.abs(r).max()))
        acc = g if acc is None else {n: acc[n] + g[n] for n in acc}
    errs = {n: num[n] / den[n] for n in num}
    errs.update({n: rel_err(got[n].astype(np.float64), acc[n]) for n in acc})
    bad = {n: e for n, e in errs.items() if not e <= 2e-2}
    assert not bad, "beyond 2e-2: %s (all: %s)" % (bad, errs)
    assert set(errs) == set(GRADS) | {"y"}


def test_stacked_inference_layers():
    """Six stacked layers with alternating group assignment on a reduced image; every layer checked."""
    cfg = dataclasses.replace(CONFIGS["c5"], H=64, W=64)
    x = make_inputs(cfg, tensors=("x",))["x"]
    for layer in range(cfg.layers):
        inp = make_inputs(cfg, layer=layer, tensors=("w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table"))
        inp["x"] = x
        got = run_gpu(cfg, inp, backward=False, layer=layer, inference=True)
        ref = run_oracle(cfg, inp, backward=False, layer=layer)
        assert rel_err(got["y"], ref["y"]) <= 2e-2
        from paper_2409_06206_b200.inputs import round_to_bf16
        x = round_to_bf16(got["y"].astype(np.float32)) * np.float32(4.0)   # keep activations O(1) between layers
        x = round_to_bf16(x)


def test_stacked_inference_full_size_image():
    """The 512 x 512 inference image at full size: six layers with alternating group assignment run back to
    back in inference mode; the first and the last layer are checked against the checker on the full image."""
    import torch
    from paper_2409_06206_b200.inputs import round_to_bf16
    cfg = CONFIGS["c5"]
    x = make_inputs(cfg, tensors=("x",))["x"]
    for layer in range(cfg.layers):
        inp = make_inputs(cfg, layer=layer, tensors=("w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table"))
        inp["x"] = x
        got = run_gpu(cfg, inp, backward=False, layer=layer, inference=True)
        assert np.isfinite(got["y"]).all()
        if layer in (0, cfg.layers - 1):
            ref = run_oracle(cfg, inp, backward=False, layer=layer)
            assert rel_err(got["y"], ref["y"]) <= 2e-2
        x = round_to_bf16(round_to_bf16(got["y"].astype(np.float32)) * np.float32(4.0))
    torch.cuda.synchronize()


def test_step_host_matches_device_path():
    import torch
    cfg = SWEEP[7]
    inp = make_inputs(cfg)
    ref = run_gpu(cfg, inp)
    desc = gb.Desc.from_config(cfg)
    tdt = torch.bfloat16
    host = {k: torch.from_numpy(v).to(tdt).pin_memory() for k, v in inp.items()}
    C, M, nh = cfg.C, cfg.window, cfg.num_heads
    out = {"y": torch.empty(inp["x"].shape, dtype=tdt).pin_memory(), "dx": torch.empty(inp["x"].shape, dtype=tdt).pin_memory(),
           "dw_qkv": torch.empty(3 * C, C).pin_memory(), "db_qkv": torch.empty(3 * C).pin_memory(),
           "dw_proj": torch.empty(C, C).pin_memory(), "db_proj": torch.empty(C).pin_memory(),
           "dbias_table": torch.empty((2 * M - 1) ** 2, nh).pin_memory()}
    arena = torch.empty(gb.gswa_step_host_arena_bytes(desc), dtype=torch.uint8, device="cuda")
    gb.gswa_step_host(desc, host["x"], host["w_qkv"], host["b_qkv"], host["w_proj"], host["b_proj"], host["bias_table"],
                      host["dy"], out["y"], out["dx"], out["dw_qkv"], out["db_qkv"], out["dw_proj"], out["db_proj"],
                      out["dbias_table"], arena)
    for n, t in out.items():
        assert rel_err(t.float().numpy().astype(np.float64), ref[n]) <= 1e-3, n
