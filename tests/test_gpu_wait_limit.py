"""The bounded device wait gives up cleanly: a barrier that nothing arrives on makes the wait
helper of the tensor-core kernels run out of its (here: one millisecond) limit, the kernel reports
GC_DEV_WAIT_LIMIT through dev_status and returns, and the next ordinary call works.  Nothing
faults, traps or spins without bound."""
import pytest
import torch

from paper_2101_06983_b200 import inputs

pytestmark = pytest.mark.gpu


def test_wait_runs_out_sets_the_status_bit_and_the_context_stays_usable(oracle):
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding
    from gpu_util import check_against_oracle, run_build
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    limit_ns = 1_000_000
    binding.gc_selftest_wait_limit(limit_ns, status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.GC_DEV_WAIT_LIMIT
    assert limit_ns <= int(waited.item()) < 50 * limit_ns       # gave up soon after the limit
    # limits outside the allowed range are refused on the host
    with pytest.raises(binding.GradCacheError):
        binding.gc_selftest_wait_limit(10 ** 9, status)
    # the context is intact: an ordinary tensor-core call right after it matches the oracle
    prob = inputs.config(1)
    out = run_build(prob)
    check_against_oracle(prob, out, oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau,
                                                       prob.mask_mode))
