"""The N > 1 path of bench.py on CPU: two gloo ranks reduce their timings to the slowest rank's and the
whole-job value counts every replica (the GPU work itself needs no collective: replicas only)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" (2 + r) ms per step and (10 - r) ms end to end
    ms_step, e2e_ms = bench.max_over_ranks([2.0 + rank, 10.0 - rank], dist, "cpu")
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{ms_step} {e2e_ms} {bench.whole_job_value(ms_step, world)}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        ms_step, e2e_ms, value = (float(x) for x in open(tmp_path / f"rank{rank}.txt").read().split())
        assert ms_step == 3.0 and e2e_ms == 10.0          # max over ranks, identical on every rank
        assert value == world * 1e3 / 3.0                  # both replicas' steps counted against the slowest time


def test_single_process_is_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_value(4.0, 1) == 250.0


def test_reference_arm_prints_one_json_line():
    """`bench.py --impl reference` times the oracle on host cores and needs no GPU."""
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "c2", "--oracle-flops", "2e9"], check=True, capture_output=True, text=True).stdout
    lines = [l for l in out.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "signmuon_optimizer_steps_per_sec" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["config"]["workload"] == "c2_resnet50"
    assert d["cpu_baseline"]["extrapolated"] is True


def test_reference_arm_and_cpu_baseline_share_one_sample_plan():
    """Both oracle timings of bench.py draw their sample from the same plan: one parameter per distinct shape
    inside the operation budget, at least one matrix, so their extrapolations agree by construction."""
    import bench
    from paper_2605_16311_b200 import workloads as wlmod
    c4 = wlmod.config4()
    idx, c_sample, c_total = bench.oracle_sample_plan(c4, 3.0e12)
    assert idx == [0]                                           # one 4096 x 4096 matrix
    assert c_total / c_sample > 30                              # 8 workers x 6 matrices against one worker of one
    c2 = wlmod.config2()
    idx2, s2, t2 = bench.oracle_sample_plan(c2, 3.0e12)
    assert len(idx2) == len({(p.rows, p.cols) for p in c2.params})   # every distinct ResNet-50 shape fits
    assert bench.shard_workers(8, 4, 3) == (6, 2) and bench.shard_workers(8, 3, 0) is None
    assert bench.whole_job_value(4.0, 2, sharded=True) == 250.0
