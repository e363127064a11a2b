"""Host-side logic of the multi-GPU benchmark, on CPU with gloo and two ranks: every rank
searches its own batch of failure sets (no data-path collective), the timings are gathered
once, and the whole-job number is all plans over the slowest rank's time."""
import os
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    w = bench.rank_workload("tiny", rank)
    rows = bench.gather_rows([float(1000 * (rank + 1)), 0.5 + rank, 2.0 - rank], world, "cpu")
    out.put((rank, [list(s) for s in w.scenarios], rows))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gather_and_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, scen0, rows0), (r1, scen1, rows1) = got
    assert rows0 == rows1 == [[1000.0, 0.5, 2.0], [2000.0, 1.5, 1.0]]
    # same shape of work on every rank, different failure sets beyond rank 0
    assert len(scen0) == len(scen1) and [len(s) for s in scen0] == [len(s) for s in scen1]
    assert scen0 != scen1
    import bench
    plans, seconds = bench.aggregate([(r[0], r[1]) for r in rows0])
    assert (plans, seconds) == (3000.0, 1.5)          # units summed, time = slowest rank
    assert bench.aggregate([(r[0], r[2]) for r in rows0]) == (3000.0, 2.0)


def test_reference_arm_prints_one_json_line():
    import json
    import subprocess
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1", "--ref-scenarios", "2"], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_reference_arm_in_integer_mode_on_a_named_workload():
    import json
    import subprocess
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "tiny", "--cost-mode", "1"],
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["dtype"] == "i64" and line["config"] == {"workload": "tiny", "scenarios_per_step": 1, "cost_mode": "int64ns"}
