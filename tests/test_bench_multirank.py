"""The N > 1 path of bench.py on CPU: independent replicas, no data-path collective; the
whole-job value is tokens summed over ranks divided by the slowest rank's time.  Two gloo
ranks on 127.0.0.1."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank 0: 100 tokens in 500 ms; rank 1: 80 tokens in 800 ms
    tokens, ms = ((100.0, 500.0), (80.0, 800.0))[rank]
    value, ms_max = bench.aggregate(tokens, ms, dist, "cpu")
    out[rank] = (value, ms_max)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for rank in (0, 1):
        value, ms_max = out[rank]
        assert ms_max == 800.0
        assert abs(value - 180.0 / 0.8) < 1e-9


def test_single_rank_aggregation_and_reference_line_shape():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(50.0, 250.0) == (200.0, 250.0)
    cfg = bench.workload_config()
    assert "workload" in cfg and "model" not in cfg


def test_gpus_flag_spawns_replicas_that_share_one_weight_copy():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself (the stand-in
    step of --selftest-launcher replaces the GPU work): both ranks rendezvous on 127.0.0.1, map
    the weights rank 0 generated, and rank 0 prints the whole-job value."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-launcher"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                      # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["ms_max"] == 800.0 and abs(out["value"] - 180.0 / 0.8) < 1e-9
    assert out["weights_identical_on_all_ranks"] is True
