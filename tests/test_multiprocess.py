"""The N > 1 path of the benchmark on CPU: the attention path has no exchange step, so ranks
are independent replicas and the only collectives are the timing barrier and the max over
ranks.  Two gloo ranks check that reduction and the whole-job throughput formula."""
import os
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r pretends to have measured (10 + r) ms per K steps and (3 - r) ms end to end
        got = bench.max_over_ranks([10.0 + rank, 3.0 - rank], dist, "cpu")
        dist.barrier()
        out[rank] = got
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    world, port = 2, 29611
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 3.0]


def test_helpers_without_process_group():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, "cpu") == [1.5, 2.5]
    # two replicas that each do 1e12 FLOPs in one second make a 2 TFLOP/s job
    assert bench.job_throughput(1e12, 2, 1.0) == 2.0


def test_reference_arm_prints_one_json_line_on_cpu():
    import json
    import subprocess
    env = dict(os.environ, OMP_NUM_THREADS="4")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, check=True)
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    # other ranks of a torchrun launch exit without work or output
    env["RANK"] = "1"
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, check=True)
    assert res.stdout.strip() == ""


def test_reduction_path_bytes_match_the_profiled_launch():
    """The bytes of dQ partial bench.py charges to the L2 reduction path are the ones ncu counted for the
    profiled launch (profiles/bwd_main_kernel_llama2_7b.md: 1.107 GB), and ragged / unmasked shapes follow
    the executed tile pairs."""
    sys.path.insert(0, str(ROOT))
    import bench
    from paper_2606_10415_b200 import workloads
    r = bench.reduction_path(workloads.ALL_CONFIGS["llama2_7b"], 0.4, {"sm_mhz": 1600.0})
    assert r["bytes_per_launch"] == 32 * 528 * 128 * 128 * 4 == 1107296256
    assert abs(r["achieved"] - 1107296256 / 0.4e-3 / 1e9) < 1e-6
    assert abs(r["peak"] - 20.7 * 148 * 1.6) < 1e-6 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-12
    full = bench.reduction_path(workloads.ALL_CONFIGS["llama2_7b_full_mask_off"], 0.7, {})
    assert full["bytes_per_launch"] == 32 * 32 * 32 * 128 * 128 * 4 and "frac" not in full
    ragged = bench.reduction_path(workloads.ALL_CONFIGS["llama2_7b_s3000_ragged"], 0.2, {"sm_mhz": 1600.0})
    assert ragged["bytes_per_launch"] == 32 * (24 * 25 // 2) * 128 * 128 * 4
