"""The N > 1 path on CPU: two gloo ranks run the replica bookkeeping bench.py uses (per-rank
problems, barrier, max over ranks, whole-job rate).  No GPU and no data-path collective."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2101_06983_b200 import replicas
    prob = replicas.replica_problem(1, rank)
    dist.barrier()
    mine = [10.0 + rank, 5.0 - rank, float(prob.Q[0, 0])]
    got = replicas.max_over_ranks(mine)
    torch.save({"got": got, "mine": mine, "shape": (prob.B, prob.N, prob.d),
                "q00": float(prob.Q[0, 0]), "pos_ok": bool((prob.pos_idx[:3] == [0, 2, 4]).all())},
               os.path.join(out_dir, f"r{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_gloo_ranks_share_only_bookkeeping(tmp_path):
    world, port = 2, 29500 + os.getpid() % 1000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(tmp_path / f"r{k}.pt") for k in range(world)]
    # every rank sees the same maxima; they are the element-wise max of the per-rank values
    assert r[0]["got"] == r[1]["got"]
    assert r[0]["got"][0] == 11.0 and r[0]["got"][1] == 5.0
    assert r[0]["got"][2] == max(r[0]["q00"], r[1]["q00"])
    # replicas: same shape and structure, different data
    assert r[0]["shape"] == r[1]["shape"] == (128, 256, 768)
    assert r[0]["q00"] != r[1]["q00"] and r[0]["pos_ok"] and r[1]["pos_ok"]


def test_single_process_is_identity_and_rate_is_aggregate():
    from paper_2101_06983_b200 import replicas
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    # 4 replicas of 100 units per step, slowest rank 2 ms per step -> 200 000 units/s
    assert replicas.whole_job_rate(100.0, 4, 2.0) == pytest.approx(2.0e5)
