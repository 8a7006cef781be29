"""Multi-rank host logic of bench.py on CPU (gloo, world size 2): the layer does not shard (replicas
only), so the one collective of a multi-GPU run is the max-over-ranks of the timings; and under a
multi-rank launch only rank 0 of the CPU-checker arm prints a line."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    out[rank] = bench.max_over_ranks(10.0 + 5.0 * rank)
    dist.destroy_process_group()


def test_timing_is_reduced_with_max_over_two_gloo_ranks():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5                      # no process group: the value itself
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        procs = [ctx.Process(target=_rank, args=(r, 2, 29611, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        assert dict(out) == {0: 15.0, 1: 15.0}


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "c2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_cost_model_covers_every_kernel_the_library_names():
    import bench
    from paper_2409_06206_b200.inputs import CONFIGS
    names = ["qkv_gemm", "attn_fwd", "proj_gemm", "dattn_gemm", "dwproj_gemm", "attn_bwd", "dx_gemm", "dwqkv_gemm"]
    cfg = CONFIGS["cM"]
    fl = sum(bench.kernel_cost(cfg, n)[0] for n in names)
    assert fl == bench.flops_per_token(cfg)                       # the kernels' flops add up to the layer's
    src = open(os.path.join(ROOT, "paper_2409_06206_b200", "csrc", "fast.cu")).read()
    for n in names:
        assert '"%s"' % n in src or n in ("attn_fwd", "attn_bwd"), n
