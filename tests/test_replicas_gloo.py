"""CPU, world_size 2 over gloo: the replica aggregation used by bench.py --gpus N."""
import os
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import importlib.util
    import torch.distributed as dist
    spec = importlib.util.spec_from_file_location("replicas", os.path.join(ROOT, "paper_2603_04716_b200", "replicas.py"))
    rep = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(rep)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0 takes 2.0 s, rank 1 takes 3.0 s for 4096 units each
    secs = 2.0 + rank
    thr, t_max, w = rep.replica_throughput(4096, secs, dist)
    mx = rep.max_over_ranks([secs, 10.0 - rank], dist)
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{thr} {t_max} {w} {mx[0]} {mx[1]}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_to_slowest_rank(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        thr, t_max, w, m0, m1 = map(float, open(tmp_path / f"r{rank}.txt").read().split())
        assert w == 2 and t_max == 3.0 and thr == pytest.approx(2 * 4096 / 3.0)
        assert (m0, m1) == (3.0, 10.0)


def test_single_process_is_identity():
    import importlib.util
    spec = importlib.util.spec_from_file_location("replicas", os.path.join(ROOT, "paper_2603_04716_b200", "replicas.py"))
    rep = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(rep)
    assert rep.replica_throughput(100, 4.0) == (25.0, 4.0, 1)
