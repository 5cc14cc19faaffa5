"""GPU parity of gc_cache_apply (Step 3 for a linear encoder, Eq. 8-9) against the CPU oracle:
dW (+)= U^T X, element by element, over shapes that span several tiles with ragged tails, with
sub-batch accumulation, padded leading dimensions, and end to end behind gc_build_cache."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import grad_err

pytestmark = pytest.mark.gpu

# U is used as two bf16 terms (exact to 2^-17 |u|), X is exact, accumulation is fp32: the result
# is fp32-class, and the fp32 gradient tolerance of the other parity tests applies.
TOL_APPLY = 1e-4


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


def _bf16_tensor(bits, device="cuda"):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(device)


SHAPES = [
    # rows, d, d_in
    (1, 8, 64), (77, 64, 64), (128, 128, 128), (300, 200, 192), (129, 768, 768),
    (1024, 768, 768), (515, 136, 1024), (640, 1536, 320), (4096, 768, 768),
]


@pytest.mark.parametrize("rows,d,d_in", SHAPES)
def test_matches_oracle(binding, oracle, rows, d, d_in):
    U = inputs.cache_rows(rows, d, seed=rows + d)
    xbits, X = inputs.encoder_inputs(rows, d_in, seed=rows + d_in)
    ref = oracle.cache_apply(U, X)
    dU, dX = torch.from_numpy(U).cuda(), _bf16_tensor(xbits)
    dW = torch.full((d, d_in), 7.0, device="cuda")          # must be overwritten
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.gc_cache_apply(dU, dX, dW, False, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert grad_err(dW.cpu().numpy(), ref) <= TOL_APPLY
    # twice the same bits
    dW2 = torch.empty_like(dW)
    binding.gc_cache_apply(dU, dX, dW2, False)
    torch.cuda.synchronize()
    assert torch.equal(dW, dW2)


def test_sub_batches_accumulate_to_the_full_batch(binding, oracle):
    """Ragged sub-batches taken as row ranges of one cache, padded leading dimensions on every
    operand: the accumulated result equals the oracle's full-batch product."""
    rows, d, d_in = 1000, 256, 384
    U = inputs.cache_rows(rows, d, seed=11)
    xbits, X = inputs.encoder_inputs(rows, d_in, seed=12)
    ref = oracle.cache_apply(U, X)
    bigU = torch.zeros(rows, d + 12, device="cuda")
    bigU[:, :d] = torch.from_numpy(U).cuda()
    bigX = torch.zeros(rows, d_in + 8, dtype=torch.bfloat16, device="cuda")
    bigX[:, :d_in] = _bf16_tensor(xbits)
    bigW = torch.full((d, d_in + 4), -3.0, device="cuda")
    dW = bigW[:, :d_in]
    lo, first = 0, True
    for n in (1, 130, 257, 512, 100):
        binding.gc_cache_apply(bigU[lo:lo + n, :d], bigX[lo:lo + n, :d_in], dW, not first)
        lo, first = lo + n, False
    torch.cuda.synchronize()
    assert lo == rows
    assert grad_err(dW.cpu().numpy(), ref) <= TOL_APPLY
    assert bool((bigW[:, d_in:] == -3.0).all())             # padding untouched


def test_step2_then_step3_gives_the_full_batch_parameter_gradient(binding, oracle):
    """Eq. 8-9 on the device: representations of two linear encoders, gc_build_cache, then
    gc_cache_apply over sub-batches.  The result is compared with the oracle's Step 2 + Step 3
    on the same bf16 representations, within the bf16 gradient tolerance of the cache."""
    B, N, d, d_in, tau = 384, 768, 768, 256, 0.5
    sbits, Xs = inputs.encoder_inputs(B, d_in, seed=21)
    tbits, Xt = inputs.encoder_inputs(N, d_in, seed=22)
    _, Wf = inputs.encoder_inputs(d, d_in, seed=23, sigma=d_in ** -0.5 * 0.6)
    _, Wg = inputs.encoder_inputs(d, d_in, seed=24, sigma=d_in ** -0.5 * 0.6)
    # encoder outputs are inputs of the path under test: formed on the host, rounded to bf16
    qbits, Q = inputs.bf16_round((Xs.astype(np.float64) @ Wf.astype(np.float64).T).astype(np.float32))
    pbits, P = inputs.bf16_round((Xt.astype(np.float64) @ Wg.astype(np.float64).T).astype(np.float32))
    pos = (2 * np.arange(B)).astype(np.int32)
    ref = oracle.build_cache(Q, P, pos, tau, 0)
    ref_Wf = oracle.cache_apply(ref["dQ"], Xs)
    ref_Wg = oracle.cache_apply(ref["dP"], Xt)

    out = binding.build_cache(_bf16_tensor(qbits), _bf16_tensor(pbits),
                              torch.from_numpy(pos).cuda(), tau, 0)
    dXs, dXt = _bf16_tensor(sbits), _bf16_tensor(tbits)
    gWf = torch.empty(d, d_in, device="cuda")
    gWg = torch.empty(d, d_in, device="cuda")
    for lo in range(0, B, 128):
        binding.gc_cache_apply(out.dQ[lo:lo + 128], dXs[lo:lo + 128], gWf, lo > 0)
    for lo in range(0, N, 192):
        binding.gc_cache_apply(out.dP[lo:lo + 192], dXt[lo:lo + 192], gWg, lo > 0)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == 0
    assert grad_err(gWf.cpu().numpy(), ref_Wf) <= 2e-2
    assert grad_err(gWg.cpu().numpy(), ref_Wg) <= 2e-2
    # Step 3 alone, fed the device's own cache, is fp32-class
    own = oracle.cache_apply(out.dQ.cpu().numpy(), Xs)
    assert grad_err(gWf.cpu().numpy(), own) <= TOL_APPLY


def test_refusals(binding):
    U = torch.zeros(16, 64, device="cuda")
    X = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, 64, device="cuda")
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_cache_apply(U, X.float(), W, False)
    assert e.value.status == 3                                # GC_ERR_DTYPE
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_cache_apply(U, torch.zeros(16, 96, dtype=torch.bfloat16, device="cuda"),
                               torch.zeros(64, 96, device="cuda"), False)
    assert e.value.status == 9                                # GC_ERR_LIMIT
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_cache_apply(U, X, W, False, ws=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6                                # GC_ERR_WORKSPACE
    assert binding.gc_cache_apply_workspace_bytes(16, 64, 96) == 0
    assert binding.gc_cache_apply_workspace_bytes(16, 64, 64) > 0
