"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing, whole-job
aggregation; the reference arm runs on rank 0 only) exercised with world_size-2 gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")     # rank 1 is the slow one
    dist.barrier()
    # the A/F pair part of a multi-GPU run: rank 0 gets the two devices, the others wait at the host-side rendezvous
    role = bench.af_pair_devices(world, rank, rank, 8)
    host_group = dist.new_group(backend="gloo")
    if isinstance(role, tuple):
        import time
        time.sleep(0.3)                                           # rank 0 "measures"; rank 1 must still be waiting afterwards
        out["done"] = True
    bench.wait_for_rank0(dist, host_group)
    out[("role", rank)] = role
    out[("saw_done", rank)] = bool(out.get("done", False))
    out[rank] = ms
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_aggregate():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29511, out), nprocs=world, join=True)
        assert out[0] == 15.0 and out[1] == 15.0
        assert out[("role", 0)] == (0, 1) and out[("role", 1)] is None
        assert out[("saw_done", 0)] and out[("saw_done", 1)]       # nobody left the rendezvous before rank 0 was done
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.0, None, "cpu") == 3.0
    one = bench.whole_job_tokens_per_s(1, 32, 0.25)
    assert one == 128000.0 and bench.whole_job_tokens_per_s(2, 32, 0.25) == 2 * one
    assert isinstance(bench.af_pair_devices(1, 0, 0, 8), str)         # one GPU: a reason, not a device pair
    assert isinstance(bench.af_pair_devices(2, 0, 0, 1), str)
    assert bench.af_pair_devices(8, 0, 7, 8) == (7, 0) and bench.af_pair_devices(8, 3, 3, 8) is None


def test_reference_arm_runs_on_rank0_only_and_prints_one_json_line():
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="1", RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, WORLD_SIZE="1", LOCAL_RANK="0", RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                        "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "tokens/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
