"""Seeded random shapes through every bf16 plan (narrow rows, paired wide rows, four-CTA sweeps):
gc_build_cache, the separate forward + backward calls and, for the unmasked loss, the rank-local
calls of an emulated world, each against the CPU oracle's full batch, element by element."""
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


def _cases(seed, count):
    rng = np.random.default_rng(seed)
    for it in range(count):
        d = int(rng.choice([64, 128, 192, 256, 320, 512, 640, 768, 1024]))
        B, N = int(rng.integers(1, 1400)), int(rng.integers(2, 1400))
        mask = int(rng.integers(0, 2))
        shared = bool(mask and rng.integers(0, 2))
        if shared:
            N = B = max(B, 2)
        tau = float(rng.choice([1.0, 0.5, 0.1, 0.05]))
        yield it, B, N, d, mask, shared, tau, int(rng.integers(2, 4))


@pytest.mark.parametrize("seed", [7, 11])
def test_random_shapes_match_the_oracle(binding, oracle, seed):
    tol = TOL["bf16"]
    for it, B, N, d, mask, shared, tau, world in _cases(seed, 24):
        prob = inputs.random_problem(B, N, d, "bf16", seed=1000 * seed + it, tau=tau,
                                     scale=d ** -0.5, mask_mode=mask, shared=shared)
        ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
        floor = grad_floor(prob)
        what = f"case {it}: B={B} N={N} d={d} mask={mask} tau={tau}"
        loss_scale = max(abs(ref["loss"]), 1e-3 * float(np.abs(ref["row_lse"]).mean()), 1e-6)
        Q, P, pos = to_device(prob)

        out = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
        sep = binding.Outputs(B, N, d, binding.GC_BF16)
        binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, sep.loss, sep.row_lse,
                            sep.pos_logit, sep.ws, sep.dev_status)
        binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, sep.row_lse, sep.dQ, sep.dP,
                            sep.ws, sep.dev_status)
        torch.cuda.synchronize()
        for o in (out, sep):
            assert int(o.dev_status.item()) == 0, what
            assert abs(o.loss.item() - ref["loss"]) <= tol["loss"] * loss_scale, what
            assert grad_err(o.dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"], what
            assert grad_err(o.dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"], what

        if mask == 0 and B >= 3 and N >= 3:
            lse = torch.zeros(B, device="cuda")
            dQ = torch.empty(B, d, device="cuda")
            dP = torch.empty(N, d, device="cuda")
            part = torch.zeros(1, device="cuda")
            loss = 0.0
            for q0, c in sharded.row_ranges(B, world):
                binding.gc_shard_fwd_dq(Q, P, pos, prob.tau, q0, c, part, lse, dQ[q0:q0 + c])
                loss += part.item()
            for p0, c in sharded.row_ranges(N, world):
                binding.gc_shard_dp(Q, P, pos, prob.tau, lse, p0, c, dP[p0:p0 + c])
            torch.cuda.synchronize()
            assert abs(loss - ref["loss"]) <= tol["loss"] * loss_scale, what
            assert grad_err(dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"], what
            assert grad_err(dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"], what
