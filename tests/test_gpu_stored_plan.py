"""GPU parity of gc_build_cache_stored, the comparison plan that keeps the B x N bf16 weights in
the workspace and forms the gradients with two GEMMs, against the CPU oracle and against
gc_build_cache on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import TOL, check_against_oracle, grad_err, rel_err_scalar, to_device
from test_gpu_parity import _check_properties, _check_sampled, _oracle_full

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


def run_stored(binding, prob):
    Q, P, pos = to_device(prob)
    out = binding.Outputs(prob.B, prob.N, prob.d, binding.GC_BF16, op=binding.GC_OP_BUILD_STORED)
    binding.gc_build_cache_stored(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse,
                                  out.dQ, out.dP, out.pos_logit, out.ws, out.dev_status)
    torch.cuda.synchronize()
    return out


SHAPES = [
    # B, N, d: one tile, ragged tails, odd tile counts, every column-part layout
    (1, 2, 64), (1, 1, 64), (7, 2, 128), (64, 128, 64), (129, 257, 128), (130, 130, 192),
    (200, 513, 256), (257, 1, 64), (65, 300, 768), (300, 200, 320), (140, 270, 448),
    (150, 260, 576), (129, 300, 1024), (260, 131, 1536), (70, 140, 4096), (385, 640, 768),
]


@pytest.mark.parametrize("B,N,d", SHAPES)
def test_small_shapes(binding, oracle, B, N, d):
    prob = inputs.random_problem(B, N, d, "bf16", seed=B * 1000 + N, tau=0.5, scale=0.5)
    out = run_stored(binding, prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("n,d,tau", [(130, 64, 0.1), (257, 128, 0.1), (96, 768, 1.0)])
def test_self_mask_shared_rows(binding, oracle, n, d, tau):
    prob = inputs.random_problem(n, n, d, "bf16", seed=n, tau=tau, mask_mode=inputs.MASK_SELF,
                                 scale=d ** -0.5, shared=True)
    out = run_stored(binding, prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


def test_many_queries_share_few_positives(binding, oracle):
    """The positive-column terms of dP are summed per passage in query order: 1500 queries on
    5 positives (more matches per passage than one scan block of 1024 queries holds), twice,
    bit for bit, and against the oracle."""
    prob = inputs.random_problem(1500, 700, 128, "bf16", seed=5, tau=0.8, scale=0.2)
    pos = (np.arange(prob.B) % 5 * 131 + 3).astype(np.int32)
    prob = dataclasses.replace(prob, pos_idx=pos)
    a = run_stored(binding, prob)
    b = run_stored(binding, prob)
    check_against_oracle(prob, a, _oracle_full(oracle, prob))
    assert torch.equal(a.dP, b.dP) and torch.equal(a.dQ, b.dQ)


@pytest.mark.parametrize("index", [1, 3])
def test_config_full(binding, oracle, index):
    prob = inputs.config(index)
    out = run_stored(binding, prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


def test_config2_headline_full_size(binding, oracle):
    prob = inputs.config(2)
    Q, P, pos = to_device(prob)
    out = run_stored(binding, prob)
    assert int(out.dev_status.item()) == 0
    fwd = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode, grads=False)
    assert rel_err_scalar(out.loss.item(), fwd["loss"]) <= TOL["bf16"]["loss"]
    lse = out.row_lse.cpu().numpy().astype(np.float64)
    assert np.abs(lse - fwd["row_lse"]).max() <= 1e-4 * np.abs(fwd["row_lse"]).max()
    _check_sampled(oracle, prob, out, 96, 48, full_lse=fwd["row_lse"], seed=2)
    _check_properties(prob, out, Q, P)


def test_config4_sampled(binding, oracle):
    prob = inputs.config(4)
    need = binding.gc_workspace_bytes(binding.GC_OP_BUILD_STORED, prob.B, prob.N, prob.d,
                                      binding.GC_BF16)
    assert need >= 2 * prob.B * prob.N                     # this plan does keep the weights
    Q, P, pos = to_device(prob)
    out = run_stored(binding, prob)
    assert int(out.dev_status.item()) == 0
    _check_sampled(oracle, prob, out, 40, 0, seed=4)
    # The scaled queries Q' are rounded to bf16 once per element, an error all passages share, so
    # the column sums of dP cancel less completely than with independently rounded weights: the
    # residue of a column is about 2^-9 |Q_ik| sqrt(B) / (B tau), a few times the 4 units above.
    _check_properties(prob, out, Q, P, units=16)


def test_out_of_range_logits_fall_back_to_recomputing(binding, oracle, sweeps_only):
    """Logits far above a row's positive logit (here by thousands of powers of two) cannot be
    stored relative to it; the call must then deliver exactly what gc_build_cache delivers.  On
    an ordinary input the two routes differ in rounding, which shows the flag is what switches."""
    hot = inputs.random_problem(200, 300, 128, "bf16", seed=21, tau=0.01, scale=1.0)
    ref = _oracle_full(oracle, hot)
    assert np.max(ref["row_lse"] - ref["pos_logit"]) > 500.0       # natural-log units
    a = run_stored(binding, hot)
    Q, P, pos = to_device(hot)
    b = binding.build_cache(Q, P, pos, hot.tau, hot.mask_mode)
    torch.cuda.synchronize()
    for name in ("loss", "row_lse", "pos_logit", "dQ", "dP"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    check_against_oracle(hot, a, ref)
    mild = inputs.random_problem(200, 300, 128, "bf16", seed=21, tau=1.0, scale=0.1)
    a = run_stored(binding, mild)
    Q, P, pos = to_device(mild)
    b = binding.build_cache(Q, P, pos, mild.tau, mild.mask_mode)
    torch.cuda.synchronize()
    assert not torch.equal(a.dP, b.dP)
    assert grad_err(a.dP.cpu().numpy(), b.dP.cpu().numpy()) <= 1e-2


def test_bad_positives_are_flagged_not_fatal(binding, oracle):
    prob = inputs.random_problem(150, 200, 128, "bf16", seed=8, tau=0.9, scale=0.2)
    pos = prob.pos_idx.copy()
    pos[3] = -1
    pos[77] = prob.N
    bad = dataclasses.replace(prob, pos_idx=pos)
    out = run_stored(binding, bad)
    assert int(out.dev_status.item()) & binding.GC_DEV_POS_RANGE
    good = np.ones(prob.B, bool)
    good[[3, 77]] = False
    ref = oracle.query_rows(prob.Q, prob.P, prob.pos_idx, np.flatnonzero(good), prob.tau,
                            prob.mask_mode)
    lse = out.row_lse.cpu().numpy().astype(np.float64)[good]
    assert np.abs(lse - ref["row_lse"]).max() <= TOL["bf16"]["lse"] * np.abs(ref["row_lse"]).max()
    assert grad_err(out.dQ.cpu().numpy()[good], ref["dQ"]) <= TOL["bf16"]["grad"]
    assert bool(torch.isfinite(out.dQ).all()) and bool(torch.isfinite(out.dP).all())


def test_refuses_what_it_cannot_store(binding):
    prob = inputs.random_problem(16, 32, 64, "f32", seed=1)
    Q, P, pos = to_device(prob)
    out = binding.Outputs(16, 32, 64, binding.GC_F32)
    with pytest.raises(binding.GradCacheError) as err:
        binding.gc_build_cache_stored(Q, P, pos, 1.0, 0, out.loss, out.row_lse, out.dQ, out.dP,
                                      out.pos_logit, out.ws, out.dev_status)
    assert err.value.status == 9
