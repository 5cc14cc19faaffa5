"""The multi-GPU variant of Step 2 (Section 3.4) on CPU: two gloo ranks run the host-side
plumbing of `sharded.sharded_build_cache` (row ranges, the all-gather of representations, the
exchange of row logsumexps, the loss all-reduce) with the two compute steps supplied by the CPU
oracle.  The ranks' results, put together, must be the oracle's full-batch results."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

B, N, D, TAU = 37, 75, 24, 0.5          # ragged: 19 + 18 queries, 38 + 37 passages


class OracleKernels:
    """Stand-in for the library's rank-local calls, written from their documented contract."""

    def fwd_dq(self, Q_all, P_all, pos_all, tau, mask_mode, q0, q_count, p_count, loss_part,
               row_lse, dQ):
        import oracle
        rows = np.arange(q0, q0 + q_count)
        out = oracle.query_rows(Q_all.numpy(), P_all.numpy(), pos_all.numpy(), rows, tau, mask_mode)
        row_lse[q0:q0 + q_count] = torch.from_numpy(out["row_lse"]).float()
        dQ.copy_(torch.from_numpy(out["dQ"]).float())
        loss_part[0] = float((out["row_lse"] - out["pos_logit"]).sum() / Q_all.shape[0])

    def dp(self, Q_all, P_all, pos_all, tau, mask_mode, row_lse, p0, p_count, q_count, dP):
        import oracle
        rows = np.arange(p0, p0 + p_count)
        out = oracle.passage_rows(Q_all.numpy(), P_all.numpy(), pos_all.numpy(),
                                  row_lse.double().numpy(), rows, tau, mask_mode)
        dP.copy_(torch.from_numpy(out).float())


def _problem():
    from paper_2101_06983_b200 import inputs
    return inputs.random_problem(B, N, D, "f32", seed=77, tau=TAU, scale=0.3)


def inputs_even():
    from paper_2101_06983_b200 import inputs
    return inputs.random_problem(36, 74, D, "f32", seed=78, tau=TAU, scale=0.3)


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2101_06983_b200 import sharded
    prob = _problem()
    (q0, b), (p0, n) = sharded.row_ranges(B, world)[rank], sharded.row_ranges(N, world)[rank]
    Ql = torch.from_numpy(prob.Q[q0:q0 + b].copy())
    Pl = torch.from_numpy(prob.P[p0:p0 + n].copy())
    posl = torch.from_numpy(prob.pos_idx[q0:q0 + b].copy())
    # the reusable step object (preallocated buffers), called twice: the second call must not
    # be disturbed by what the first one left in the buffers
    step = sharded.ShardedStep(B, N, D, Ql.dtype, Ql.device, kernels=OracleKernels())
    step.run(Ql, Pl, posl, TAU)
    loss, lse, dQ, dP = step.run(Ql, Pl, posl, TAU, measure=True)
    torch.save(dict(loss=float(loss), lse=lse.clone(), dQ=dQ.clone(), dP=dP.clone(), q=(q0, b),
                    p=(p0, n), timings=step.timings), os.path.join(out_dir, f"r{rank}.pt"))
    # an even split takes the path without padded blocks: 36 queries, 74 passages
    even = inputs_even()
    (e0, eb), (f0, fn_) = sharded.row_ranges(36, world)[rank], sharded.row_ranges(74, world)[rank]
    out = sharded.sharded_build_cache(torch.from_numpy(even.Q[e0:e0 + eb].copy()),
                                      torch.from_numpy(even.P[f0:f0 + fn_].copy()),
                                      torch.from_numpy(even.pos_idx[e0:e0 + eb].copy()), TAU, 36, 74,
                                      kernels=OracleKernels())
    torch.save(dict(loss=float(out[0]), dQ=out[2].clone(), dP=out[3].clone()),
               os.path.join(out_dir, f"e{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_two_ranks_reproduce_the_full_batch(tmp_path, oracle):
    world, port = 2, 29600 + os.getpid() % 1000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(tmp_path / f"r{k}.pt") for k in range(world)]
    prob = _problem()
    ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, TAU, 0)
    assert r[0]["q"] == (0, 19) and r[1]["q"] == (19, 18)
    assert r[0]["p"] == (0, 38) and r[1]["p"] == (38, 37)
    for k in range(world):
        assert abs(r[k]["loss"] - ref["loss"]) <= 1e-5 * abs(ref["loss"])   # same on every rank
        np.testing.assert_allclose(r[k]["lse"].numpy(), ref["row_lse"], rtol=1e-6)
    dQ = torch.cat([r[0]["dQ"], r[1]["dQ"]]).numpy()
    dP = torch.cat([r[0]["dP"], r[1]["dP"]]).numpy()
    assert np.abs(dQ - ref["dQ"]).max() <= 1e-6 * np.abs(ref["dQ"]).max()
    # dP on each rank used the exchanged float32 row_lse of the other rank's queries
    assert np.abs(dP - ref["dP"]).max() <= 1e-5 * np.abs(ref["dP"]).max()
    assert set(r[0]["timings"]) == {"gather_reps_s", "fwd_dq_s", "lse_and_loss_s", "dp_s"}
    e = [torch.load(tmp_path / f"e{k}.pt") for k in range(world)]
    even = inputs_even()
    eref = oracle.build_cache(even.Q, even.P, even.pos_idx, TAU, 0)
    assert abs(e[0]["loss"] - eref["loss"]) <= 1e-5 * abs(eref["loss"])
    edQ = torch.cat([e[0]["dQ"], e[1]["dQ"]]).numpy()
    edP = torch.cat([e[0]["dP"], e[1]["dP"]]).numpy()
    assert np.abs(edQ - eref["dQ"]).max() <= 1e-6 * np.abs(eref["dQ"]).max()
    assert np.abs(edP - eref["dP"]).max() <= 1e-5 * np.abs(eref["dP"]).max()


def test_row_ranges_cover_everything_once():
    from paper_2101_06983_b200 import sharded
    for total, world in ((37, 2), (8, 8), (5, 3), (4096, 7), (3, 4)):
        rr = sharded.row_ranges(total, world)
        assert len(rr) == world and rr[0][0] == 0
        assert all(rr[i][0] + rr[i][1] == rr[i + 1][0] for i in range(world - 1))
        assert rr[-1][0] + rr[-1][1] == total
        assert max(c for _, c in rr) - min(c for _, c in rr) <= 1


def test_single_process_needs_no_group():
    from paper_2101_06983_b200 import sharded
    x = torch.arange(12.0).reshape(4, 3)
    assert sharded.gather_rows(x, [4]) is x
