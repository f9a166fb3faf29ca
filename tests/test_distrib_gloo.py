"""The N > 1 path of the benchmark on CPU: two gloo ranks, the same helpers bench.py uses
(barrier, max over ranks, per-rank seeds, whole-job throughput)."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2503_05066_b200 import distrib, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    info = distrib.rank_info_from_env()
    distrib.init(info, backend="gloo")
    distrib.barrier(info)
    # rank r pretends its step took (r + 1) ms: every rank must see the slowest one
    worst = distrib.max_over_ranks(float(rank + 1), info)
    value = distrib.job_throughput(1000, worst, info)
    cfg = synth.CONFIGS["tiny_f32"].with_(N=8, d=16, seed=distrib.shard_seed(0, info))
    x = synth.hidden_states(cfg)
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([worst, value, float(x.sum())]))
    distrib.finish(info)


def test_two_ranks_weak_scaling_accounting(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "r0.npy")
    r1 = np.load(tmp_path / "r1.npy")
    assert r0[0] == r1[0] == 2.0                         # MAX over ranks
    assert r0[1] == r1[1] == 2 * 1000 / 2e-3             # all ranks' units over the slowest time
    assert r0[2] != r1[2]                                # different seeds -> different batches


def test_single_process_is_a_no_op():
    info = distrib.RankInfo(0, 1, 0)
    distrib.init(info)
    distrib.barrier(info)
    assert distrib.max_over_ranks(3.5, info) == 3.5
    assert distrib.job_throughput(10, 5.0, info) == 2000.0
    assert distrib.shard_seed(7, distrib.RankInfo(3, 4, 3)) == 10


def test_bench_starts_its_own_ranks_when_called_with_gpus(tmp_path):
    """`python bench.py --gpus 2` without a launcher around it re-runs itself as two ranks
    (torch.distributed.run on 127.0.0.1).  Checked on CPU with the reference arm, which needs no
    GPU: rank 0 prints the one JSON line for n_gpus = 2, the other rank exits 0 without output."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference",
                        "--config", "tiny_f32", "--steps", "1", "--warmup", "0", "--ref-tokens", "4"],
                       capture_output=True, text=True, timeout=600, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["extrapolated"] is True
    assert line["value"] > 0 and line["e2e"]["h2d_bytes_per_step"] == 0
