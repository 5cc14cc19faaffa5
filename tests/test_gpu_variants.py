"""GPU parity of the loss-variant calls (Section 3.3, Step 2) against oracle.build_variant:
dL/dtau from the cache rows, and the cosine-similarity loss (unit rows in, normalisation
Jacobian out) end to end through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import TOL, grad_err, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


@pytest.mark.parametrize("B,N,d,dtype,tau,mask", [
    (64, 128, 768, "f32", 1.0, 0), (130, 257, 72, "f32", 0.3, 0), (128, 256, 768, "bf16", 1.0, 0),
    (300, 300, 128, "bf16", 0.2, 1), (700, 1300, 768, "bf16", 0.5, 0),
])
def test_dtau_from_the_cache(binding, oracle, B, N, d, dtype, tau, mask):
    prob = inputs.random_problem(B, N, d, dtype, seed=B + d, tau=tau, scale=d ** -0.5,
                                 mask_mode=mask, shared=bool(mask))
    Q, P, pos = to_device(prob)
    out = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    dtau = torch.full((1,), float("nan"), device="cuda")
    binding.gc_dtau(Q, out.dQ, prob.tau, dtau)
    again = torch.zeros(1, device="cuda")
    binding.gc_dtau(Q, out.dQ, prob.tau, again)
    torch.cuda.synchronize()
    ref = oracle.build_variant(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
    # dL/dtau is a sum of B terms of either sign: the error is measured against their magnitude
    scale = float(np.abs((prob.Q * ref["dQ"]).sum(axis=1)).sum() / prob.tau)
    assert abs(dtau.item() - ref["dtau"]) <= TOL[dtype]["grad"] * max(scale, 1e-30)
    assert torch.equal(dtau, again)                          # fixed reduction order


@pytest.mark.parametrize("B,N,d,dtype,tau", [
    (64, 128, 768, "f32", 1.0), (129, 300, 64, "f32", 0.1), (128, 256, 768, "bf16", 1.0),
    (600, 1100, 768, "bf16", 0.5), (300, 520, 128, "bf16", 0.5),
])
def test_cosine_loss_end_to_end(binding, oracle, B, N, d, dtype, tau):
    """Rows of widely different lengths: normalise, Step 2 on the unit rows, Jacobian."""
    prob = inputs.random_problem(B, N, d, dtype, seed=B + N + d, tau=tau, scale=1.0)
    rng = np.random.default_rng(3)
    prob_Q = prob.Q * rng.uniform(0.2, 5.0, size=(B, 1)).astype(prob.Q.dtype)
    prob_P = prob.P * rng.uniform(0.2, 5.0, size=(N, 1)).astype(prob.P.dtype)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    Q = torch.from_numpy(prob_Q.astype(np.float32)).cuda().to(tdt)
    P = torch.from_numpy(prob_P.astype(np.float32)).cuda().to(tdt)
    pos = torch.from_numpy(prob.pos_idx).cuda()
    # the instance is what the device holds (bf16-rounded where the dtype is bf16)
    Qh, Ph = Q.float().cpu().numpy().astype(np.float64), P.float().cpu().numpy().astype(np.float64)
    ref = oracle.build_variant(Qh, Ph, prob.pos_idx, tau, 0, cosine=True)

    Qn, Pn = torch.empty_like(Q), torch.empty_like(P)
    iq, ip = torch.empty(B, device="cuda"), torch.empty(N, device="cuda")
    binding.gc_row_normalize(Q, Qn, iq)
    binding.gc_row_normalize(P, Pn, ip)
    out = binding.build_cache(Qn, Pn, pos, tau, 0)
    dtau = torch.zeros(1, device="cuda")
    binding.gc_dtau(Qn, out.dQ, tau, dtau)
    dQ, dP = torch.empty_like(out.dQ), out.dP                  # one out of place, one in place
    binding.gc_cosine_bwd(Q, iq, out.dQ, dQ)
    binding.gc_cosine_bwd(P, ip, out.dP, dP)
    torch.cuda.synchronize()

    np.testing.assert_allclose(iq.cpu().numpy(), 1.0 / np.linalg.norm(Qh, axis=1), rtol=2e-6)
    unit = Qh / np.linalg.norm(Qh, axis=1, keepdims=True)
    tol_unit = 2.0 ** -8 if dtype == "bf16" else 1e-6
    assert np.abs(Qn.float().cpu().numpy() - unit).max() <= tol_unit
    # bf16: the unit rows are rounded to bf16 before the sweeps see them, which moves every logit
    # by at most 2 * 2^-9 / tau on top of the usual bf16 tolerances
    extra = 2.0 ** -8 / tau if dtype == "bf16" else 0.0
    tol = TOL[dtype]
    assert int(out.dev_status.item()) == 0
    assert abs(out.loss.item() - ref["loss"]) <= (tol["loss"] + extra) * abs(ref["loss"])
    assert grad_err(dQ.cpu().numpy(), ref["dQ"]) <= tol["grad"] + extra
    assert grad_err(dP.cpu().numpy(), ref["dP"]) <= tol["grad"] + extra
    scale = float(np.abs((unit * (ref["dQ"] * np.linalg.norm(Qh, axis=1, keepdims=True))).sum(axis=1)).sum())
    big = float(np.abs(ref["dQ"] * np.linalg.norm(Qh, axis=1, keepdims=True)).sum()) / tau
    assert abs(dtau.item() - ref["dtau"]) <= (tol["grad"] + extra) * max(big, scale)
    # the gradients have no component along their rows (tangent to the sphere)
    along = (Q.float() * dQ).sum(dim=1).abs().max().item()
    assert along <= 1e-3 * float(np.abs(ref["dQ"]).max()) * float(np.abs(Qh).max()) * d ** 0.5


def test_variant_calls_refuse_bad_arguments(binding):
    X = torch.zeros(4, 12, device="cuda")
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_row_normalize(X, torch.empty_like(X), torch.empty(4, device="cuda"))
    assert e.value.status == 9                                   # d not a multiple of 8
    Q = torch.zeros(4, 16, device="cuda")
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_dtau(Q, torch.zeros(4, 16, device="cuda"), 0.0, torch.zeros(1, device="cuda"))
    assert e.value.status == 2


def _positive_lists(B, N, rng, mask_mode, max_pos=4):
    """Between one and max_pos distinct positives per query, none on the masked diagonal; some
    passages are the positive of several queries."""
    lists = []
    for i in range(B):
        k = int(rng.integers(1, max_pos + 1))
        allowed = np.array([j for j in range(N) if not (mask_mode and j == i)])
        lists.append([int(v) for v in rng.choice(allowed, size=min(k, len(allowed)), replace=False)])
    return lists


@pytest.mark.parametrize("B,N,d,dtype,tau,mask", [
    (64, 128, 768, "f32", 1.0, 0), (100, 57, 72, "f32", 0.3, 0), (128, 256, 768, "bf16", 1.0, 0),
    (300, 300, 128, "bf16", 0.2, 1), (520, 900, 768, "bf16", 0.5, 0), (200, 200, 64, "f32", 0.5, 1),
])
def test_several_positives_per_query(binding, oracle, B, N, d, dtype, tau, mask):
    prob = inputs.random_problem(B, N, d, dtype, seed=B + 3 * d, tau=tau, scale=d ** -0.5,
                                 mask_mode=mask, shared=bool(mask))
    rng = np.random.default_rng(B + N)
    lists = _positive_lists(B, N, rng, mask)
    ref = oracle.build_variant(prob.Q, prob.P, lists, prob.tau, prob.mask_mode)
    Q, P, _ = to_device(prob)
    ptr = np.zeros(B + 1, np.int32)
    ptr[1:] = np.cumsum([len(r) for r in lists])
    flat = np.array([v for r in lists for v in r], np.int32)
    pos_ptr, pos_list = torch.from_numpy(ptr).cuda(), torch.from_numpy(flat).cuda()
    f = dict(dtype=torch.float32, device="cuda")
    outs = []
    for _ in range(2):
        loss, lse = torch.zeros(1, **f), torch.empty(B, **f)
        dQ, dP = torch.full((B, d), float("nan"), **f), torch.full((N, d), float("nan"), **f)
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.gc_build_cache_multi_pos(Q, P, pos_ptr, pos_list, prob.tau, prob.mask_mode, loss,
                                         lse, dQ, dP, dev_status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        outs.append((loss, dQ, dP))
    loss, dQ, dP = outs[0]
    tol = TOL[dtype]
    assert abs(loss.item() - ref["loss"]) <= tol["loss"] * max(abs(ref["loss"]), 1e-6)
    floor = 1e-2 * max(float(np.abs(prob.Q).max()), float(np.abs(prob.P).max())) / (B * tau)
    assert grad_err(dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"]
    assert grad_err(dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"]
    assert torch.equal(dQ, outs[1][1]) and torch.equal(dP, outs[1][2])      # reproducible
    assert torch.equal(loss, outs[1][0])


def test_one_positive_per_query_is_the_plain_call(binding):
    prob = inputs.random_problem(150, 260, 128, "bf16", seed=8, tau=0.4, scale=0.1)
    Q, P, pos = to_device(prob)
    plain = binding.build_cache(Q, P, pos, prob.tau, 0)
    B, N, d = prob.B, prob.N, prob.d
    f = dict(dtype=torch.float32, device="cuda")
    loss, lse, dQ, dP = torch.zeros(1, **f), torch.empty(B, **f), torch.empty(B, d, **f), torch.empty(N, d, **f)
    ptr = torch.arange(B + 1, dtype=torch.int32, device="cuda")
    binding.gc_build_cache_multi_pos(Q, P, ptr, pos, prob.tau, 0, loss, lse, dQ, dP)
    torch.cuda.synchronize()
    assert torch.equal(loss, plain.loss) and torch.equal(dQ, plain.dQ) and torch.equal(dP, plain.dP)


def test_bad_positive_lists_raise_the_device_flags(binding):
    prob = inputs.random_problem(40, 60, 64, "bf16", seed=3, tau=1.0, scale=0.2)
    Q, P, pos = to_device(prob)
    B, N, d = prob.B, prob.N, prob.d
    f = dict(dtype=torch.float32, device="cuda")
    loss, lse, dQ, dP = torch.zeros(1, **f), torch.empty(B, **f), torch.empty(B, d, **f), torch.empty(N, d, **f)
    ptr = torch.arange(B + 1, dtype=torch.int32, device="cuda")
    ptr[5] = ptr[4]                                 # query 4 has no positive
    bad = pos.clone()
    bad[9] = N + 3                                  # out of range
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.gc_build_cache_multi_pos(Q, P, ptr, bad, prob.tau, 0, loss, lse, dQ, dP, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & 1                       # GC_DEV_POS_RANGE
    assert bool(torch.isfinite(dQ).all()) and bool(torch.isfinite(dP).all())


@pytest.mark.parametrize("B,N,d,dtype,tau", [
    (64, 128, 768, "f32", 1.0), (100, 100, 72, "f32", 0.3), (128, 256, 768, "bf16", 1.0),
    (300, 450, 128, "bf16", 0.2), (520, 900, 768, "bf16", 0.5), (77, 77, 64, "f32", 0.5),
])
def test_two_direction_loss(binding, oracle, B, N, d, dtype, tau):
    prob = inputs.random_problem(B, N, d, dtype, seed=2 * B + d, tau=tau, scale=d ** -0.5)
    pos_np = prob.pos_idx.copy()
    pos_np[B // 2] = pos_np[0]                      # two queries share a positive passage
    ref = oracle.build_variant(prob.Q, prob.P, pos_np, prob.tau, 0, two_direction=True)
    Q, P, _ = to_device(prob)
    pos = torch.from_numpy(pos_np).cuda()
    f = dict(dtype=torch.float32, device="cuda")
    outs = []
    for _ in range(2):
        loss, lse = torch.zeros(1, **f), torch.empty(B, **f)
        dQ, dP = torch.full((B, d), float("nan"), **f), torch.full((N, d), float("nan"), **f)
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.gc_build_cache_two_direction(Q, P, pos, prob.tau, loss, lse, dQ, dP, dev_status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        outs.append((loss, dQ, dP))
    loss, dQ, dP = outs[0]
    tol = TOL[dtype]
    assert abs(loss.item() - ref["loss"]) <= tol["loss"] * max(abs(ref["loss"]), 1e-6)
    floor = 1e-2 * max(float(np.abs(prob.Q).max()), float(np.abs(prob.P).max())) / (B * tau)
    assert grad_err(dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"]
    assert grad_err(dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"]
    assert torch.equal(dQ, outs[1][1]) and torch.equal(dP, outs[1][2])
