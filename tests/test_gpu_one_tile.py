"""GPU parity of the one-launch plan for batches of a single tile (B <= 128; N <= 256 for bf16,
N <= 128 for fp32 inputs, which run on the tensor cores as three bf16 terms): loss, row_lse,
pos_logit, dQ and dP element by element against the CPU oracle at the tolerances of the other
parity tests, through gc_build_cache and through gc_loss_fwd + gc_loss_bwd."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import check_against_oracle, run_build, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


def _oracle_full(oracle, prob):
    return oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)


# B, N, d: one and several column slices, ragged last slice (d not a multiple of 64), rows and
# columns short of the tile, a single passage, the largest tile of each dtype
SHAPES_BF16 = [(1, 1, 8), (1, 2, 64), (7, 3, 24), (64, 128, 64), (100, 200, 320), (128, 256, 768),
               (128, 129, 72), (33, 256, 200), (128, 64, 1024), (17, 250, 520)]
SHAPES_F32 = [(1, 1, 8), (1, 2, 64), (7, 3, 24), (64, 128, 768), (100, 90, 320), (128, 128, 768),
              (128, 65, 72), (33, 128, 200), (128, 64, 1024), (17, 120, 520)]


def _cases():
    for s in SHAPES_BF16:
        yield ("bf16",) + s
    for s in SHAPES_F32:
        yield ("f32",) + s


@pytest.mark.parametrize("dtype,B,N,d", list(_cases()))
def test_build_matches_oracle(binding, oracle, dtype, B, N, d):
    code = binding.GC_BF16 if dtype == "bf16" else binding.GC_F32
    assert binding.gc_plan_name(binding.GC_OP_BUILD, B, N, d, code) == "tcgen05-one-tile"
    assert binding.gc_kernel_launches(binding.GC_OP_BUILD, B, N, d, code) == 1
    prob = inputs.random_problem(B, N, d, dtype, seed=B * 1000 + N + d, tau=0.5, scale=0.5)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))
    # twice the same bits
    again = run_build(prob)
    assert torch.equal(out.dQ, again.dQ) and torch.equal(out.dP, again.dP)
    assert torch.equal(out.loss, again.loss)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("n,d,tau", [(128, 64, 0.1), (96, 768, 1.0), (50, 136, 0.05)])
def test_self_mask(binding, oracle, n, d, tau, dtype):
    prob = inputs.random_problem(n, n, d, dtype, seed=n + d, tau=tau, mask_mode=inputs.MASK_SELF,
                                 scale=d ** -0.5, shared=True)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("dtype,B,N,d", [("bf16", 128, 256, 768), ("f32", 64, 128, 768),
                                         ("bf16", 90, 131, 136), ("f32", 77, 100, 264)])
def test_forward_then_backward(binding, oracle, dtype, B, N, d):
    """gc_loss_fwd (one CTA) and gc_loss_bwd (row_lse given) take the same kernel."""
    prob = inputs.random_problem(B, N, d, dtype, seed=5 * B + N, tau=0.3, scale=d ** -0.5)
    ref = _oracle_full(oracle, prob)
    Q, P, pos = to_device(prob)
    code = binding._dtype_code(Q)
    b = binding.Outputs(prob.B, prob.N, prob.d, code)
    b.dQ.fill_(float("nan"))
    b.dP.fill_(float("nan"))
    binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, b.loss, b.row_lse, b.pos_logit, b.ws,
                        b.dev_status)
    binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, b.row_lse, b.dQ, b.dP, b.ws,
                        b.dev_status)
    torch.cuda.synchronize()
    check_against_oracle(prob, b, ref)


def test_padded_leading_dimensions_and_untouched_padding(binding, oracle):
    B, N, d = 100, 200, 200
    prob = inputs.random_problem(B, N, d, "bf16", seed=9, tau=0.7, scale=0.3)
    ref = _oracle_full(oracle, prob)
    Q, P, pos = to_device(prob)
    bigQ = torch.zeros(B, d + 24, dtype=torch.bfloat16, device="cuda")
    bigP = torch.zeros(N, d + 8, dtype=torch.bfloat16, device="cuda")
    bigQ[:, :d], bigP[:, :d] = Q, P
    code = binding.GC_BF16
    out = binding.Outputs(B, N, d, code)
    big_dq = torch.full((B, d + 12), 5.0, device="cuda")
    big_dp = torch.full((N, d + 4), 5.0, device="cuda")
    binding.gc_build_cache(bigQ[:, :d], bigP[:, :d], pos, prob.tau, prob.mask_mode, out.loss,
                           out.row_lse, big_dq[:, :d], big_dp[:, :d], out.pos_logit, out.ws,
                           out.dev_status)
    torch.cuda.synchronize()
    out.dQ, out.dP = big_dq[:, :d].contiguous(), big_dp[:, :d].contiguous()
    check_against_oracle(prob, out, ref)
    assert bool((big_dq[:, d:] == 5.0).all()) and bool((big_dp[:, d:] == 5.0).all())


def test_bad_positive_indices_raise_the_device_flags(binding):
    prob = inputs.random_problem(40, 60, 64, "bf16", seed=3, tau=1.0, scale=0.2)
    Q, P, pos = to_device(prob)
    bad = pos.clone()
    bad[7] = 60                                    # out of range
    out = binding.build_cache(Q, P, bad, prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) & 1           # GC_DEV_POS_RANGE
    assert bool(torch.isfinite(out.dQ).all()) and bool(torch.isfinite(out.dP).all())


# fp32 batches of a few tiles: the same kernel once per tile pair and column slice
TILED_F32 = [(129, 257, 72), (130, 130, 128), (200, 513, 192), (257, 1, 64), (65, 300, 768),
             (300, 200, 320), (140, 270, 448), (129, 300, 1024), (260, 131, 1536), (70, 140, 4096),
             (1000, 900, 64), (128, 129, 8), (129, 128, 8), (1100, 2300, 136), (2100, 1500, 64)]


@pytest.mark.parametrize("B,N,d", TILED_F32)
def test_fp32_batches_of_a_few_tiles(binding, oracle, B, N, d):
    assert binding.gc_plan_name(binding.GC_OP_BUILD, B, N, d, binding.GC_F32) == "tcgen05-tiles"
    prob = inputs.random_problem(B, N, d, "f32", seed=B * 1000 + N, tau=0.5, scale=0.5)
    ref = _oracle_full(oracle, prob)
    out = run_build(prob)
    check_against_oracle(prob, out, ref)
    again = run_build(prob)
    assert torch.equal(out.dQ, again.dQ) and torch.equal(out.dP, again.dP)
    # forward and backward as separate calls
    Q, P, pos = to_device(prob)
    b = binding.Outputs(prob.B, prob.N, prob.d, binding.GC_F32)
    b.dQ.fill_(float("nan"))
    b.dP.fill_(float("nan"))
    binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, b.loss, b.row_lse, b.pos_logit, b.ws,
                        b.dev_status)
    binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, b.row_lse, b.dQ, b.dP, b.ws,
                        b.dev_status)
    torch.cuda.synchronize()
    check_against_oracle(prob, b, ref)


@pytest.mark.parametrize("n,d,tau", [(130, 64, 0.1), (257, 128, 0.1), (400, 72, 0.5)])
def test_fp32_tiles_self_mask(binding, oracle, n, d, tau):
    prob = inputs.random_problem(n, n, d, "f32", seed=n, tau=tau, mask_mode=inputs.MASK_SELF,
                                 scale=d ** -0.5, shared=True)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


# bf16 rows that are not whole 64-column chunks: a few tiles per batch run on the tensor cores too
TILED_BF16 = [(129, 257, 72), (300, 520, 200), (200, 513, 136), (130, 130, 520), (1000, 1000, 40),
              (257, 1, 8), (129, 300, 1000)]


@pytest.mark.parametrize("B,N,d", TILED_BF16)
def test_bf16_odd_widths_in_a_few_tiles(binding, oracle, B, N, d):
    assert binding.gc_plan_name(binding.GC_OP_BUILD, B, N, d, binding.GC_BF16) == "tcgen05-tiles"
    prob = inputs.random_problem(B, N, d, "bf16", seed=B + N + d, tau=0.5, scale=d ** -0.5)
    ref = _oracle_full(oracle, prob)
    out = run_build(prob)
    check_against_oracle(prob, out, ref)
    Q, P, pos = to_device(prob)
    b = binding.Outputs(prob.B, prob.N, prob.d, binding.GC_BF16)
    binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, b.loss, b.row_lse, b.pos_logit, b.ws,
                        b.dev_status)
    binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, b.row_lse, b.dQ, b.dP, b.ws,
                        b.dev_status)
    torch.cuda.synchronize()
    check_against_oracle(prob, b, ref)
