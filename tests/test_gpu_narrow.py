"""GPU parity of the narrow-row gradient sweeps (bf16 rows of 64 or 128 values: S tiles and W
tiles side by side in tensor memory, each streamed tile loaded once) against the CPU oracle:
several x tiles and parts of the streamed range, ragged tails, the self mask, the separate
forward / backward calls, and inputs that leave the range of the fixed row scale."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import TOL, check_against_oracle, grad_err, run_build, to_device
from test_gpu_parity import _oracle_full

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


# B, N, d: more CTAs than the tile-pair plan takes, so the sweeps run; odd tile counts per part
SHAPES = [(1500, 2500, 64), (2100, 1900, 128), (3000, 777, 128), (9000, 129, 64), (130, 20000, 128)]


@pytest.mark.parametrize("B,N,d", SHAPES)
def test_build_cache(binding, oracle, B, N, d):
    assert binding.gc_plan_name(binding.GC_OP_BUILD, B, N, d, binding.GC_BF16) == "tcgen05"
    prob = inputs.random_problem(B, N, d, "bf16", seed=B + N + d, tau=0.3, scale=d ** -0.5)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("n,d,tau", [(2100, 128, 0.1), (1700, 64, 0.5)])
def test_self_mask_shared_rows(binding, oracle, n, d, tau):
    prob = inputs.random_problem(n, n, d, "bf16", seed=n, tau=tau, mask_mode=inputs.MASK_SELF,
                                 scale=d ** -0.5, shared=True)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))
    # the masked pair contributes nothing: dP of a row does not contain its own query's weight
    assert int(out.dev_status.item()) == 0


@pytest.mark.parametrize("d", [64, 128])
def test_forward_then_backward(binding, oracle, d, sweeps_only):
    """gc_loss_fwd + gc_loss_bwd (dQ and dP sweeps with a given row_lse) against the oracle, on a
    shape small enough that only the switch keeps it on the sweep kernels, and on a large one."""
    for B, N in ((150, 333), (1900, 2300)):
        prob = inputs.random_problem(B, N, d, "bf16", seed=B + d, tau=0.7, scale=d ** -0.5)
        Q, P, pos = to_device(prob)
        out = binding.Outputs(B, N, d, binding.GC_BF16)
        binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse,
                            out.pos_logit, out.ws, out.dev_status)
        binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, out.row_lse, out.dQ, out.dP,
                            out.ws, out.dev_status)
        torch.cuda.synchronize()
        check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("d", [64, 128])
def test_logits_far_above_the_positive(binding, oracle, d):
    """Row sums beyond what the positive logit as a fixed scale allows: the call must deliver the
    result of the sweeps that track the running maximum."""
    prob = inputs.random_problem(1800, 2200, d, "bf16", seed=21, tau=0.01, scale=1.0)
    ref = _oracle_full(oracle, prob)
    assert np.max(ref["row_lse"] - ref["pos_logit"]) > 500.0       # natural-log units
    out = run_build(prob)
    check_against_oracle(prob, out, ref)


def test_twice_is_bit_identical(binding):
    prob = inputs.random_problem(2100, 1900, 128, "bf16", seed=3, tau=0.2, scale=0.1)
    a = run_build(prob)
    b = run_build(prob)
    for name in ("loss", "row_lse", "pos_logit", "dQ", "dP"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    assert grad_err(a.dQ.cpu().numpy(), b.dQ.cpu().numpy()) == 0.0
    assert TOL["bf16"]["grad"] > 0
