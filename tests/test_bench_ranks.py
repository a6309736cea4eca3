"""Host-side logic of the multi-rank bench (replicas only), on CPU with gloo and two ranks."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"ms": ms, "units": units}, f)
    dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sums_units(tmp_path):
    out = str(tmp_path / "agg.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    res = json.load(open(out))
    assert res["ms"] == 15.0 and res["units"] == 300.0        # whole-job value = all ranks' units / slowest rank


def test_single_rank_passthrough():
    import bench
    assert bench.aggregate_over_ranks(3.0, 7.0) == (3.0, 7.0)


def test_reference_arm_non_zero_ranks_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_launch_count_and_workloads_are_host_computable():
    import bench
    for name in ("config1", "config2", "config3"):
        spec, lib, route, fixed = bench.workload_spec(name, 1024 if name != "config1" else None)
        assert spec.n_q_heads % spec.n_kv_heads == 0
    assert sorted(set(bench.fixed_choice_for([(1, 128, 1024), (2, 1000, 6096), (3, 100, 0), (0, 0, 0)], 32).tolist())) == [0, 1, 2, 3]
