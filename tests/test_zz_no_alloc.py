"""gc_loss_fwd_static: the forward call whose scratch is a fixed array inside the library, for
callers that have no way to hand the library a workspace (a host framework that owns all device
memory, or a hot loop that must not touch an allocator).

Collected last on purpose (file name): a run that stops at the first failure has then already
exercised every other test.  Each case calls the entry point through the C ABI twice in a row -
the second call finds the array full of the first call's values - and compares with gc_loss_fwd
given an ordinary workspace.  Both run the same kernels, so the results must agree bit for bit,
which is well inside the tolerances the parity tests use; the CPU oracle is compared as well, at
the tolerances of the parity tests, so that the check does not rest on the CUDA path alone."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


def _problems():
    yield inputs.config(1)                                               # tensor-core plan
    yield inputs.config(0)                                               # fp32 plan
    yield inputs.random_problem(300, 777, 128, "bf16", seed=3, tau=0.2, scale=0.3,
                                mask_mode=inputs.MASK_SELF)
    yield inputs.random_problem(129, 130, 40, "f32", seed=4, tau=0.5, scale=0.5)


def test_static_scratch_forward_matches_workspace_forward(binding, oracle):
    from gpu_util import TOL
    for prob in _problems():
        want = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode,
                                  grads=False)
        tol = TOL[prob.dtype]
        Q, P, pos = binding.problem_tensors(prob)
        code = binding._dtype_code(Q)
        assert binding.gc_static_scratch_need(prob.B, prob.N, prob.d, code) \
            <= binding.GC_STATIC_SCRATCH_BYTES
        ref = binding.Outputs(prob.B, prob.N, prob.d, code)
        binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, ref.loss, ref.row_lse,
                            ref.pos_logit, ref.ws, ref.dev_status)
        torch.cuda.synchronize()
        for call in range(2):
            loss = torch.full((1,), float("nan"), device="cuda")
            lse = torch.full((prob.B,), float("nan"), device="cuda")
            pl = torch.full((prob.B,), float("nan"), device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            before = torch.cuda.memory_allocated()
            binding.gc_loss_fwd_static(Q, P, pos, prob.tau, prob.mask_mode, loss, lse, pl, status)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before          # torch's pool untouched
            assert int(status.item()) == 0
            assert torch.equal(loss, ref.loss), (prob.name, call)
            assert torch.equal(lse, ref.row_lse), (prob.name, call)
            assert torch.equal(pl, ref.pos_logit), (prob.name, call)
            torch.testing.assert_close(loss, ref.loss, rtol=1e-5, atol=0)
            assert abs(loss.item() - want["loss"]) <= tol["loss"] * abs(want["loss"])
            got_lse = lse.cpu().numpy().astype(np.float64)
            assert np.abs(got_lse - want["row_lse"]).max() \
                <= tol["lse"] * max(1.0, np.abs(want["row_lse"]).max())
            got_pl = pl.cpu().numpy().astype(np.float64)
            assert np.abs(got_pl - want["pos_logit"]).max() \
                <= tol["lse"] * max(1.0, np.abs(want["pos_logit"]).max())


def test_static_scratch_refuses_oversized_problems(binding):
    """A batch whose forward scratch exceeds the built-in array is refused on the host, before
    any launch, with the dedicated status."""
    B, N, d = 1 << 20, 64, 64
    assert binding.gc_static_scratch_need(B, N, d, binding.GC_BF16) > binding.GC_STATIC_SCRATCH_BYTES
    Q = torch.zeros(8, d, dtype=torch.bfloat16, device="cuda")
    rc = binding._lib.gc_loss_fwd_static(Q.data_ptr(), d, Q.data_ptr(), d, Q.data_ptr(), B, N, d,
                                         1.0, 0, binding.GC_BF16, Q.data_ptr(), Q.data_ptr(),
                                         None, None, None)
    assert rc == 9
    assert "scratch" in binding.status_string(rc)
