"""gc_build_cache captured into a CUDA graph: the call is asynchronous on the caller's stream, its
side-stream work is forked from and joined back into that stream, and nothing in it touches the
host allocator or synchronises, so one call can be captured once and replayed.  The replay must
give the eager call's results bit for bit (and those are checked against the oracle), for every
plan."""
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import check_against_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


CASES = [
    # B, N, d, dtype, mask: one launch, tile pairs, four-CTA sweeps, narrow-row sweeps, paired wide
    # rows, FMA tiles
    (128, 256, 768, "bf16", 0), (64, 128, 768, "f32", 0), (300, 520, 640, "bf16", 0),
    (1030, 1300, 768, "bf16", 0), (2100, 2100, 128, "bf16", 1), (700, 1400, 320, "bf16", 0),
    (150, 140, 36, "f32", 0),
]


@pytest.mark.parametrize("B,N,d,dtype,mask", CASES)
def test_graph_replay_equals_the_eager_call(binding, oracle, B, N, d, dtype, mask):
    prob = inputs.random_problem(B, N, d, dtype, seed=B + d, tau=0.5, scale=d ** -0.5,
                                 mask_mode=mask, shared=bool(mask))
    Q, P, pos = binding.problem_tensors(prob)
    out = binding.Outputs(prob.B, prob.N, prob.d, binding._dtype_code(Q))

    def step():
        binding.gc_build_cache(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse, out.dQ,
                               out.dP, out.pos_logit, out.ws, out.dev_status)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        step()
    torch.cuda.synchronize()
    ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
    check_against_oracle(prob, out, ref)
    eager = [t.clone() for t in (out.loss, out.row_lse, out.pos_logit, out.dQ, out.dP)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        step()
    for _ in range(2):
        for t in (out.loss, out.row_lse, out.pos_logit, out.dQ, out.dP):
            t.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        for got, want in zip((out.loss, out.row_lse, out.pos_logit, out.dQ, out.dP), eager):
            assert torch.equal(got, want)
    assert int(out.dev_status.item()) == 0
