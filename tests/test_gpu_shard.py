"""Section 3.4 on one GPU: the rank-local calls gc_shard_fwd_dq / gc_shard_dp are run for every
rank of an emulated world in turn (ragged row ranges), their outputs are concatenated, and the
result is compared with the CPU oracle's full-batch loss and gradients, element by element."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs, sharded

from gpu_util import TOL, grad_err, grad_floor, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


CASES = [
    # B, N, d, dtype, world
    (50, 90, 40, "f32", 3),        # FMA-tile plan
    (300, 610, 128, "bf16", 2),    # narrow rows, fixed row scale
    (700, 1300, 768, "bf16", 3),   # four-CTA sweeps per rank
    (250, 520, 768, "bf16", 2),    # 125 queries per rank: one x tile, online-maximum sweep
    (130, 260, 1024, "bf16", 4),
]


@pytest.mark.parametrize("B,N,d,dtype,world", CASES)
def test_ranks_together_reproduce_the_full_batch(binding, oracle, B, N, d, dtype, world):
    prob = inputs.random_problem(B, N, d, dtype, seed=B + N, tau=0.5, scale=d ** -0.5)
    ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
    Q, P, pos = to_device(prob)
    row_lse = torch.zeros(B, device="cuda")
    dQ = torch.empty(B, d, device="cuda")
    dP = torch.empty(N, d, device="cuda")
    loss = torch.zeros(1, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    part = torch.zeros(1, device="cuda")
    q_ranges, p_ranges = sharded.row_ranges(B, world), sharded.row_ranges(N, world)
    for q0, b in q_ranges:
        binding.gc_shard_fwd_dq(Q, P, pos, prob.tau, q0, b, part, row_lse, dQ[q0:q0 + b],
                                dev_status=status)
        loss += part
    for p0, n in p_ranges:
        binding.gc_shard_dp(Q, P, pos, prob.tau, row_lse, p0, n, dP[p0:p0 + n], dev_status=status)
    torch.cuda.synchronize()
    tol = TOL[dtype]
    assert int(status.item()) == 0
    assert abs(loss.item() - ref["loss"]) <= tol["loss"] * abs(ref["loss"])
    lse = row_lse.cpu().numpy().astype(np.float64)
    assert np.abs(lse - ref["row_lse"]).max() <= tol["lse"] * max(1.0, np.abs(ref["row_lse"]).max())
    floor = grad_floor(prob)
    assert grad_err(dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"]
    assert grad_err(dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"]


MASKED = [
    # rows (Q = P = the same rows), d, dtype, world: the self mask with shared rows, as in the
    # two-view workload; the masked pair of a rank's row lies wherever that row sits in the batch
    (60, 40, "f32", 3),
    (300, 128, "bf16", 2),
    (520, 768, "bf16", 3),
    (1000, 128, "bf16", 4),
]


@pytest.mark.parametrize("n,d,dtype,world", MASKED)
def test_self_mask_follows_the_rank_ranges(binding, oracle, n, d, dtype, world):
    prob = inputs.random_problem(n, n, d, dtype, seed=n + d, tau=0.2, mask_mode=inputs.MASK_SELF,
                                 scale=d ** -0.5, shared=True)
    ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
    Q, P, pos = to_device(prob)
    row_lse = torch.zeros(n, device="cuda")
    dQ = torch.empty(n, d, device="cuda")
    dP = torch.empty(n, d, device="cuda")
    loss = torch.zeros(1, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    part = torch.zeros(1, device="cuda")
    for q0, b in sharded.row_ranges(n, world):
        binding.gc_shard_fwd_dq(Q, P, pos, prob.tau, q0, b, part, row_lse, dQ[q0:q0 + b],
                                dev_status=status, mask_mode=prob.mask_mode)
        loss += part
    for p0, m in sharded.row_ranges(n, world):
        binding.gc_shard_dp(Q, P, pos, prob.tau, row_lse, p0, m, dP[p0:p0 + m], dev_status=status,
                            mask_mode=prob.mask_mode)
    torch.cuda.synchronize()
    tol = TOL[dtype]
    assert int(status.item()) == 0
    assert abs(loss.item() - ref["loss"]) <= tol["loss"] * abs(ref["loss"])
    lse = row_lse.cpu().numpy().astype(np.float64)
    assert np.abs(lse - ref["row_lse"]).max() <= tol["lse"] * max(1.0, np.abs(ref["row_lse"]).max())
    floor = grad_floor(prob)
    assert grad_err(dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"]
    assert grad_err(dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"]


def test_sharded_step_object_on_one_gpu(binding, oracle):
    """`sharded.ShardedStep` (preallocated buffers, library kernels) as a world of one rank, twice
    in a row on the same buffers."""
    prob = inputs.random_problem(300, 520, 768, "bf16", seed=12, tau=0.5, scale=768 ** -0.5)
    ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
    Q, P, pos = to_device(prob)
    step = sharded.ShardedStep(prob.B, prob.N, prob.d, Q.dtype, Q.device)
    for _ in range(2):
        loss, lse, dQ, dP = step.run(Q, P, pos, prob.tau, measure=True)
        torch.cuda.synchronize()
        assert abs(loss.item() - ref["loss"]) <= TOL["bf16"]["loss"] * abs(ref["loss"])
        assert grad_err(dQ.cpu().numpy(), ref["dQ"]) <= TOL["bf16"]["grad"]
        assert grad_err(dP.cpu().numpy(), ref["dP"]) <= TOL["bf16"]["grad"]
    assert set(step.timings) == {"gather_reps_s", "fwd_dq_s", "lse_and_loss_s", "dp_s"}


def test_one_rank_is_the_whole_batch(binding, sweeps_only):
    """world = 1: the two calls together are gc_loss_fwd + gc_loss_bwd on the same kernels (the
    rank-local calls always run the sweeps, so the whole-batch call is kept on them too)."""
    prob = inputs.random_problem(140, 270, 64, "bf16", seed=5, tau=0.7, scale=0.125)
    Q, P, pos = to_device(prob)
    a = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    row_lse = torch.zeros(prob.B, device="cuda")
    dQ = torch.empty_like(a.dQ)
    dP = torch.empty_like(a.dP)
    part = torch.zeros(1, device="cuda")
    binding.gc_shard_fwd_dq(Q, P, pos, prob.tau, 0, prob.B, part, row_lse, dQ)
    binding.gc_shard_dp(Q, P, pos, prob.tau, row_lse, 0, prob.N, dP)
    torch.cuda.synchronize()
    assert torch.equal(row_lse, a.row_lse) and torch.equal(part, a.loss)
    assert torch.equal(dQ, a.dQ)
    assert grad_err(dP.cpu().numpy(), a.dP.cpu().numpy()) <= 1e-2


def test_refusals(binding):
    prob = inputs.random_problem(40, 80, 64, "bf16", seed=1)
    Q, P, pos = to_device(prob)
    f = dict(device="cuda")
    part, lse = torch.zeros(1, **f), torch.zeros(40, **f)
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_shard_fwd_dq(Q, P, pos, 1.0, 30, 20, part, lse, torch.empty(20, 64, **f))
    assert e.value.status == 2                                 # range past the last query
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_shard_dp(Q, P, pos, 1.0, lse, -1, 10, torch.empty(10, 64, **f))
    assert e.value.status == 2
    assert binding.gc_shard_workspace_bytes(40, 80, 64, binding.GC_BF16, 41, 10) == 0
