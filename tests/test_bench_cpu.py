"""CPU-side checks of bench.py: the reference arm's JSON line, and the N > 1
aggregation (max of step time, sum of units) over two gloo ranks."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
           "--workload", "toy", "--steps", "2", "--warmup", "3"]
    out = subprocess.run(cmd, capture_output=True, text=True, check=True, cwd=ROOT).stdout
    lines = [l for l in out.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle"
    assert d["cpu_baseline"]["cores"] == 1 and d["value"] > 1e6
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert d["metric"] == "replica_param_updates_per_sec" and d["higher_is_better"] is True
    assert d["config"]["workload"] == "toy" and "model" not in d["config"]
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT)
    assert r.returncode == 0 and r.stdout.strip() == ""


WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}",
                        rank=int(os.environ["RANK"]), world_size=2)
rank = dist.get_rank()
ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), 2)
dist.barrier()
print("RESULT", rank, ms, units)
dist.destroy_process_group()
"""


def test_two_rank_aggregation_over_gloo():
    port = free_port()
    code = WORKER.format(root=ROOT, port=port)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    for rank, p in enumerate(procs):
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        line = [l for l in out.splitlines() if l.startswith("RESULT")][0].split()
        assert int(line[1]) == rank
        assert float(line[2]) == 15.0      # max over ranks of the step time
        assert float(line[3]) == 3000.0    # units of all ranks


def test_single_rank_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0, 1) == (3.5, 7.0)
    assert bench.measured_peak_gbs()[0] > 1000


def _shard_worker(rank, world, port, numel, out):
    import torch.distributed as dist
    from paper_2601_22442_b200.layouts import coordinate_shard
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    sizes, bases = coordinate_shard(numel, rank, world)
    mine = torch.tensor([sizes, bases], dtype=torch.int64)
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)          # host-side bookkeeping only: the data path has no collective
    if rank == 0:
        out.put([g.tolist() for g in gathered])
    dist.destroy_process_group()


def test_coordinate_shards_of_two_ranks_tile_every_stage():
    import multiprocessing as mp
    from paper_2601_22442_b200.layouts import coordinate_shard, workloads
    numel = workloads()["llama125m"]["numel"] + [4099]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, numel, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (s0, b0), (s1, b1) = got
    for j, n in enumerate(numel):
        assert b0[j] == 0 and b1[j] == s0[j] and s0[j] + s1[j] == n     # exact tiling, in order
        assert b1[j] % 1024 == 0 and s0[j] > 0 and s1[j] > 0
    with pytest.raises(ValueError):
        coordinate_shard([1000], 0, 2)
    with pytest.raises(ValueError):
        coordinate_shard([5000], 0, 2, align=6)


def test_traffic_ratio_is_looked_up_by_kernel_name_and_p():
    import bench
    assert bench.measured_traffic_ratio("owner R=4 compact entries=32", 0.05) == pytest.approx(1.035)
    assert bench.measured_traffic_ratio("pipelined R=8 compact wide", 0.05) == pytest.approx(1.012)
    assert bench.measured_traffic_ratio("owner R=4 compact entries=32", 0.07) is None      # no capture at that p
    assert bench.measured_traffic_ratio("no such kernel", 0.05) is None
