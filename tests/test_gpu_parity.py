"""GPU parity: the CUDA library (called through its C ABI) against the CPU oracle on the same
seeded inputs, element by element at sizes the oracle finishes in seconds, and by sampled rows
and size-independent properties at the full workload sizes."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import TOL, check_against_oracle, grad_err, rel_err_scalar, run_build, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


def _oracle_full(oracle, prob):
    return oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)


# ---- element-by-element parity on small and ragged shapes ---------------------------------------
SHAPES = [
    # B, N, d
    (1, 2, 4), (1, 1, 8), (7, 2, 12), (64, 128, 64), (129, 257, 72), (130, 130, 128),
    (200, 513, 192), (257, 1, 64), (65, 300, 768), (300, 200, 320), (140, 270, 448),
    (150, 260, 576), (129, 300, 1024), (260, 131, 1536), (70, 140, 4096),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,N,d", SHAPES)
def test_small_shapes(binding, oracle, B, N, d, dtype, plan_mode):
    if dtype == "bf16" and d % 8:
        d = (d + 7) // 8 * 8            # rows must start on 16-byte boundaries
    prob = inputs.random_problem(B, N, d, dtype, seed=B * 1000 + N, tau=0.5, scale=0.5)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,d,tau", [(130, 64, 0.1), (257, 128, 0.1), (96, 768, 1.0)])
def test_self_mask_shared_rows(binding, oracle, n, d, tau, dtype, plan_mode):
    prob = inputs.random_problem(n, n, d, dtype, seed=n, tau=tau, mask_mode=inputs.MASK_SELF,
                                 scale=d ** -0.5, shared=True)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


# Rows of two column halves (d = 512, 640, 768) with more than one x tile run as clusters of four
# CTAs whose two pairs alternate over the streamed tiles: 1, 2, 3 and more tiles per cluster, odd
# and even counts, an odd number of x tiles, split streamed ranges, both mask modes.
QUAD_SHAPES = [
    (130, 100, 768), (200, 200, 768), (257, 330, 512), (300, 520, 640), (385, 900, 768),
    (520, 260, 512), (1030, 1300, 768), (2100, 3000, 640),
]


@pytest.mark.parametrize("B,N,d", QUAD_SHAPES)
def test_four_cta_cluster_sweeps(binding, oracle, B, N, d, plan_mode):
    prob = inputs.random_problem(B, N, d, "bf16", seed=B + N + d, tau=0.3, scale=d ** -0.5)
    out = run_build(prob)
    ref = _oracle_full(oracle, prob)
    check_against_oracle(prob, out, ref)
    # the same kernels with a given row_lse (gc_loss_bwd), from the forward call's lse
    Q, P, pos = to_device(prob)
    b = binding.Outputs(prob.B, prob.N, prob.d, binding.GC_BF16)
    binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, b.loss, b.row_lse, b.pos_logit, b.ws,
                        b.dev_status)
    binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, b.row_lse, b.dQ, b.dP, b.ws,
                        b.dev_status)
    torch.cuda.synchronize()
    check_against_oracle(prob, b, ref)


def test_four_cta_cluster_sweeps_self_mask(binding, oracle, plan_mode):
    prob = inputs.random_problem(700, 700, 768, "bf16", seed=77, tau=0.2,
                                 mask_mode=inputs.MASK_SELF, scale=768 ** -0.5, shared=True)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("B,N", [(300, 45000), (45000, 300)])
def test_streamed_matrix_larger_than_l2_uses_cta_pairs(binding, oracle, B, N):
    """When the streamed matrix (P for the forward/dQ sweeps, Q for the dP sweep) exceeds 64 MB
    the wide-row kernels run as CTA pairs that share every streamed chunk.  Both orientations,
    with an odd number of 128-row tiles on the stationary side (3), against the full oracle."""
    prob = inputs.random_problem(B, N, 768, "bf16", seed=B + N, tau=0.5, scale=768 ** -0.5)
    Q, P, pos = to_device(prob)
    out = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    ref = _oracle_full(oracle, prob)
    check_against_oracle(prob, out, ref)
    # the stand-alone forward and backward calls take the same paired kernels
    b = binding.Outputs(prob.B, prob.N, prob.d, binding.GC_BF16)
    binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, b.loss, b.row_lse, b.pos_logit, b.ws,
                        b.dev_status)
    binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, b.row_lse, b.dQ, b.dP, b.ws,
                        b.dev_status)
    torch.cuda.synchronize()
    check_against_oracle(prob, b, ref)


def test_fwd_then_bwd_equals_build(binding, oracle, plan_mode):
    """The separate forward and backward calls reproduce gc_build_cache: bit for bit where both
    run the same kernels (fp32 inputs), within rounding where gc_build_cache fuses the forward
    into the dQ sweep (bf16 rows)."""
    for dtype, d in (("f32", 96), ("bf16", 128), ("bf16", 768)):
        prob = inputs.random_problem(150, 333, d, dtype, seed=9, tau=0.7, scale=d ** -0.5)
        Q, P, pos = to_device(prob)
        a = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
        b = binding.Outputs(prob.B, prob.N, prob.d, binding._dtype_code(Q))
        binding.gc_loss_fwd(Q, P, pos, prob.tau, prob.mask_mode, b.loss, b.row_lse, b.pos_logit,
                            b.ws, b.dev_status)
        binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, b.row_lse, b.dQ, b.dP, b.ws,
                            b.dev_status)
        torch.cuda.synchronize()
        if dtype == "bf16":
            assert torch.equal(a.pos_logit, b.pos_logit)
            torch.testing.assert_close(a.loss, b.loss, rtol=1e-5, atol=0)
            torch.testing.assert_close(a.row_lse, b.row_lse, rtol=1e-5, atol=1e-5)
            assert grad_err(a.dQ.cpu().numpy(), b.dQ.cpu().numpy()) <= 1e-2
            assert grad_err(a.dP.cpu().numpy(), b.dP.cpu().numpy()) <= 1e-2
        else:
            for name in ("loss", "row_lse", "pos_logit", "dQ", "dP"):
                assert torch.equal(getattr(a, name), getattr(b, name)), name
        # either gradient may be skipped
        c = binding.Outputs(prob.B, prob.N, prob.d, binding._dtype_code(Q))
        c.dQ.fill_(7.0)
        binding.gc_loss_bwd(Q, P, pos, prob.tau, prob.mask_mode, a.row_lse, None, c.dP, c.ws)
        torch.cuda.synchronize()
        assert torch.equal(c.dP, a.dP) and bool((c.dQ == 7.0).all())


def test_strided_rows(binding, oracle, plan_mode):
    """Leading dimensions larger than d on inputs and outputs."""
    prob = inputs.random_problem(70, 140, 64, "f32", seed=4, tau=1.0, scale=0.3)
    Qb = torch.zeros(70, 80, device="cuda")
    Pb = torch.zeros(140, 96, device="cuda")
    Qb[:, :64] = torch.from_numpy(prob.Q)
    Pb[:, :64] = torch.from_numpy(prob.P)
    pos = torch.from_numpy(prob.pos_idx).cuda()
    out = binding.Outputs(70, 140, 64, binding.GC_F32)
    dQb = torch.full((70, 72), 3.0, device="cuda")
    dPb = torch.full((140, 68), 3.0, device="cuda")
    binding.gc_build_cache(Qb[:, :64], Pb[:, :64], pos, 1.0, 0, out.loss, out.row_lse,
                           dQb[:, :64], dPb[:, :64], out.pos_logit, out.ws, out.dev_status)
    torch.cuda.synchronize()
    ref = _oracle_full(oracle, prob)
    assert grad_err(dQb[:, :64].cpu().numpy(), ref["dQ"]) <= 1e-4
    assert grad_err(dPb[:, :64].cpu().numpy(), ref["dP"]) <= 1e-4
    assert bool((dQb[:, 64:] == 3.0).all()) and bool((dPb[:, 64:] == 3.0).all())


# ---- the named workloads ------------------------------------------------------------------------
@pytest.mark.parametrize("index", [0, 1])
def test_config_small(binding, oracle, index, plan_mode):
    prob = inputs.config(index)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


def test_config3_symmetric_full(binding, oracle):
    prob = inputs.config(3)
    assert binding.gc_plan_name(binding.GC_OP_BUILD, prob.B, prob.N, prob.d, binding.GC_BF16) \
        == "tcgen05"
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


def _check_sampled(oracle, prob, out, n_q, n_p, full_lse=None, seed=0):
    """Sampled rows against the oracle.  dP rows need lse for every query from the oracle; they
    are checked only when `full_lse` (oracle values) is supplied."""
    tol = TOL[prob.dtype]
    rng = np.random.default_rng(seed)
    rows = np.unique(np.r_[0, prob.B - 1, rng.integers(0, prob.B, n_q)]).astype(np.int64)
    ref = oracle.query_rows(prob.Q, prob.P, prob.pos_idx, rows, prob.tau, prob.mask_mode)
    lse = out.row_lse.cpu().numpy().astype(np.float64)[rows]
    assert np.abs(lse - ref["row_lse"]).max() <= tol["lse"] * np.abs(ref["row_lse"]).max()
    pl = out.pos_logit.cpu().numpy().astype(np.float64)[rows]
    assert np.abs(pl - ref["pos_logit"]).max() <= tol["lse"] * max(1.0, np.abs(ref["pos_logit"]).max())
    dq = out.dQ[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert grad_err(dq, ref["dQ"]) <= tol["grad"]
    if full_lse is not None:
        prow = np.unique(np.r_[0, prob.N - 1, rng.integers(0, prob.N, n_p)]).astype(np.int64)
        dp_ref = oracle.passage_rows(prob.Q, prob.P, prob.pos_idx, full_lse, prow, prob.tau,
                                     prob.mask_mode)
        dp = out.dP[torch.from_numpy(prow).cuda()].cpu().numpy()
        assert grad_err(dp, dp_ref) <= tol["grad"]


def _check_properties(prob, out, Q, P, units=4):
    """Identities that hold at any size: sum_j dP_j = 0 and sum <Q, dQ> = sum <P, dP>."""
    dP64 = out.dP.double()
    scale = float(dP64.abs().max())
    col = dP64.sum(dim=0).abs().max().item()
    assert col <= 2e-2 * scale * units                   # bf16 weights: a few rounding units
    a = (Q.double() * out.dQ.double()).sum().item()
    b = (P.double() * dP64).sum().item()
    norm = (Q.double().abs() * out.dQ.double().abs()).sum().item()
    assert abs(a - b) <= 2e-2 * norm
    assert bool(torch.isfinite(out.dQ).all()) and bool(torch.isfinite(out.dP).all())


def test_config2_headline_full_size(binding, oracle):
    """Headline workload, every element of the loss, row_lse, pos_logit, dQ and dP against the full
    oracle (a few seconds on the host)."""
    prob = inputs.config(2)
    assert binding.gc_plan_name(binding.GC_OP_BUILD, prob.B, prob.N, prob.d, binding.GC_BF16) \
        == "tcgen05"
    Q, P, pos = to_device(prob)
    out = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    ref = _oracle_full(oracle, prob)
    check_against_oracle(prob, out, ref)
    lse = out.row_lse.cpu().numpy().astype(np.float64)
    assert np.abs(lse - ref["row_lse"]).max() <= 1e-4 * np.abs(ref["row_lse"]).max()
    _check_properties(prob, out, Q, P)


def test_config4_extreme_batch_never_stores_S(binding, oracle):
    prob = inputs.config(4)
    code = binding.GC_BF16
    need = binding.gc_workspace_bytes(binding.GC_OP_BUILD, prob.B, prob.N, prob.d, code)
    assert need < prob.B * prob.N // 4                   # nowhere near one value per logit
    Q, P, pos = to_device(prob)
    torch.cuda.reset_peak_memory_stats()
    before = torch.cuda.memory_allocated()
    out = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    grown = torch.cuda.max_memory_allocated() - before
    assert grown < 2 * ((prob.B + prob.N) * prob.d * 4) + need + (64 << 20)
    assert int(out.dev_status.item()) == 0
    # 256 sampled query rows (lse, positive logit, dQ) against the oracle.  Rows of dP need the
    # logsumexp of all 65536 queries, which the oracle would take minutes to produce; the library's
    # row_lse stands in for it here, after the sampled rows of it have just matched the oracle.
    _check_sampled(oracle, prob, out, 256, 0, seed=4)
    gpu_lse = out.row_lse.cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(44)
    prow = np.unique(np.r_[0, 1, prob.N - 1, rng.integers(0, prob.N, 64)]).astype(np.int64)
    assert prow.size >= 64
    dp_ref = oracle.passage_rows(prob.Q, prob.P, prob.pos_idx, gpu_lse, prow, prob.tau,
                                 prob.mask_mode)
    dp = out.dP[torch.from_numpy(prow).cuda()].cpu().numpy()
    assert grad_err(dp, dp_ref) <= TOL["bf16"]["grad"]
    _check_properties(prob, out, Q, P)
    # the loss is the mean of (lse - positive logit); spot rows already match the oracle
    lse = out.row_lse.double()
    pl = out.pos_logit.double()
    assert abs((lse - pl).mean().item() - out.loss.item()) <= 1e-5 * abs(out.loss.item())


# ---- bit-exact index and mask behaviour ------------------------------------------------------------
@pytest.mark.parametrize("dtype,d", [("f32", 64), ("bf16", 64), ("bf16", 768)])
def test_positive_gather_is_bit_exact(binding, dtype, d, plan_mode):
    """Q_i = e_0 and P_j[0] = code(j), all other entries 0: S_ij = code(j) exactly, so
    pos_logit[i] must equal code(pos_idx[i]) bit for bit wherever the positive sits."""
    B, N = 300, 1000
    code = (np.arange(N) % 251 + 1).astype(np.float32) / 256.0      # exact in bf16
    Qn = np.zeros((B, d), np.float32)
    Qn[:, 0] = 1.0
    Pn = np.zeros((N, d), np.float32)
    Pn[:, 0] = code
    rng = np.random.default_rng(0)
    edges = [0, N - 1]
    for t in (32, 64, 128, 256):
        edges += [t - 1, t, t + 1, N - t, 2 * t - 1, 2 * t]
    pos = rng.integers(0, N, B)
    pos[:len(edges)] = edges
    pos[-5:] = pos[0]                                                # duplicates
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    Q = torch.from_numpy(Qn).to(tdt).cuda()
    P = torch.from_numpy(Pn).to(tdt).cuda()
    out = binding.build_cache(Q, P, torch.from_numpy(pos.astype(np.int32)).cuda(), 1.0, 0)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == 0
    got = out.pos_logit.cpu().numpy()
    assert np.array_equal(got.view(np.uint32), code[pos].view(np.uint32))


@pytest.mark.parametrize("dtype,d", [("f32", 320), ("bf16", 320), ("bf16", 768)])
def test_self_mask_is_exact_zero(binding, dtype, d, plan_mode):
    """Row i has a private coordinate c_i = i.  dP_i[c_i] = G_ii Q_i[c_i] / tau must be exactly
    +0 under the self mask, and is non-zero without it."""
    n = 300
    rng = np.random.default_rng(3)
    X = (rng.standard_normal((n, d)) * 0.05).astype(np.float32)
    X[:, :n] = 0.0
    X[np.arange(n), np.arange(n)] = 1.0
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    Xd = torch.from_numpy(X).to(tdt).cuda()
    pos = torch.from_numpy(((np.arange(n) + 7) % n).astype(np.int32)).cuda()
    masked = binding.build_cache(Xd, Xd, pos, 0.5, binding.GC_MASK_SELF)
    plain = binding.build_cache(Xd, Xd, pos, 0.5, binding.GC_MASK_NONE)
    torch.cuda.synchronize()
    idx = torch.arange(n, device="cuda")
    diag_m = masked.dP[idx, idx].cpu().numpy()
    assert np.array_equal(diag_m.view(np.uint32), np.zeros(n, np.uint32))     # +0.0f exactly
    assert bool((plain.dP[idx, idx] != 0).all())
    diag_q = masked.dQ[idx, idx].cpu().numpy()
    assert np.array_equal(diag_q.view(np.uint32), np.zeros(n, np.uint32))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mask_does_not_leak(binding, oracle, dtype, plan_mode):
    """Rows of norm 8 in random directions, shared between Q and P: every diagonal logit is 64
    while the off-diagonal ones stay below about 30, so a single unmasked diagonal entry would
    move that row's lse by tens.  Sizes are not multiples of any tile."""
    n, d = 333, 64
    rng = np.random.default_rng(5)
    X = rng.standard_normal((n, d))
    X = (8.0 * X / np.linalg.norm(X, axis=1, keepdims=True)).astype(np.float32)
    prob = inputs._finish("leak", X, X, ((np.arange(n) + 1) % n).astype(np.int32), 1.0,
                          inputs.MASK_SELF, dtype, shared=True)
    out = run_build(prob)
    check_against_oracle(prob, out, _oracle_full(oracle, prob))


@pytest.mark.parametrize("B,N,d,tau", [(200, 300, 128, 0.01), (300, 520, 768, 0.004)])
def test_logits_far_above_the_positive(binding, oracle, B, N, d, tau, plan_mode):
    """Rows whose largest logit lies hundreds of powers of two above their positive logit: the
    wide-row build scales its weights by the positive logit and must hand such inputs to the
    kernels that track the running row maximum."""
    prob = inputs.random_problem(B, N, d, "bf16", seed=21, tau=tau, scale=1.0)
    ref = _oracle_full(oracle, prob)
    assert np.max(ref["row_lse"] - ref["pos_logit"]) > 500.0       # natural-log units
    out = run_build(prob)
    check_against_oracle(prob, out, ref)


def test_bad_positives_are_flagged_not_fatal(binding, oracle, plan_mode):
    prob = inputs.random_problem(40, 50, 64, "f32", seed=1, tau=1.0, scale=0.3,
                                 mask_mode=inputs.MASK_SELF)
    pos = prob.pos_idx.copy()
    pos[3] = 50
    pos[4] = -1
    pos[5] = 5                                                      # the masked column
    Q, P, _ = to_device(prob)
    out = binding.build_cache(Q, P, torch.from_numpy(pos).cuda(), prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == (binding.GC_DEV_POS_RANGE | binding.GC_DEV_POS_MASKED)
    pl = out.pos_logit.cpu().numpy()
    assert pl[3] == 0 and pl[4] == 0 and pl[5] == 0
    # the flagged rows have no one-hot term: their G row sums to one instead of zero, all other
    # rows match the oracle run on the valid rows' problem
    good = np.array([i for i in range(40) if i not in (3, 4, 5)])
    ref = oracle.query_rows(prob.Q, prob.P, prob.pos_idx, good, prob.tau, prob.mask_mode)
    assert grad_err(out.dQ[torch.from_numpy(good).cuda()].cpu().numpy(), ref["dQ"]) <= 1e-4
    assert bool(torch.isfinite(out.dQ).all()) and bool(torch.isfinite(out.dP).all())
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.gc_loss_bwd(Q, P, torch.from_numpy(pos).cuda(), prob.tau, prob.mask_mode, out.row_lse,
                        out.dQ, out.dP, out.ws, st)
    assert int(st.item()) == (binding.GC_DEV_POS_RANGE | binding.GC_DEV_POS_MASKED)


@pytest.mark.parametrize("d", [128, 768])
def test_bad_positives_with_a_fixed_row_scale(binding, oracle, d, plan_mode):
    """The bf16 builds that scale each row's weights by its positive logit (narrow rows, and rows
    of two column halves): a row whose pos_idx is unusable has no positive logit to scale by; it
    is flagged, gets no one-hot term, and every other row still matches the oracle."""
    B, N = 200, 300
    prob = inputs.random_problem(B, N, d, "bf16", seed=31, tau=0.5, scale=d ** -0.5,
                                 mask_mode=inputs.MASK_SELF)
    pos = prob.pos_idx.copy()
    pos[7] = N
    pos[130] = -3
    pos[150] = 150                                                  # the masked column
    Q, P, _ = to_device(prob)
    out = binding.build_cache(Q, P, torch.from_numpy(pos).cuda(), prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == (binding.GC_DEV_POS_RANGE | binding.GC_DEV_POS_MASKED)
    pl = out.pos_logit.cpu().numpy()
    assert pl[7] == 0 and pl[130] == 0 and pl[150] == 0
    good = np.array([i for i in range(B) if i not in (7, 130, 150)])
    ref = oracle.query_rows(prob.Q, prob.P, prob.pos_idx, good, prob.tau, prob.mask_mode)
    lse = out.row_lse.cpu().numpy()[good]
    assert np.abs(lse - ref["row_lse"]).max() <= TOL["bf16"]["lse"] * np.abs(ref["row_lse"]).max()
    assert grad_err(out.dQ[torch.from_numpy(good).cuda()].cpu().numpy(), ref["dQ"]) <= TOL["bf16"]["grad"]
    assert bool(torch.isfinite(out.dQ).all()) and bool(torch.isfinite(out.dP).all())


@pytest.mark.parametrize("index", [1, 2, 3])
def test_deterministic(binding, index):
    prob = inputs.config(index)
    Q, P, pos = to_device(prob)
    a = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    b = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    for name in ("loss", "row_lse", "pos_logit", "dQ", "dP"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


def test_workspace_canaries(binding, plan_mode):
    """Nothing is written outside the reported workspace size or outside the output rows."""
    prob = inputs.config(1)
    Q, P, pos = to_device(prob)
    code = binding.GC_BF16
    need = binding.gc_workspace_bytes(binding.GC_OP_BUILD, prob.B, prob.N, prob.d, code)
    pad = 4096
    buf = torch.full((need + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
    off = (-buf.data_ptr()) % 256 + 256
    ws = buf[off:off + need]
    out = binding.Outputs(prob.B, prob.N, prob.d, code)
    binding.gc_build_cache(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse, out.dQ,
                           out.dP, out.pos_logit, ws, out.dev_status)
    torch.cuda.synchronize()
    assert bool((buf[:off] == 0xA5).all()) and bool((buf[off + need:] == 0xA5).all())


def test_per_call_kernel_timing(binding, sweeps_only):
    """gc_profile_enable(n) keeps one event set per call: n queued calls can be read afterwards,
    each with positive sweep durations; a call that was never made is refused."""
    prob = inputs.random_problem(300, 520, 768, "bf16", seed=2, tau=0.5, scale=768 ** -0.5)
    Q, P, pos = to_device(prob)
    out = binding.Outputs(prob.B, prob.N, prob.d, binding.GC_BF16)
    binding.gc_profile_enable(3)
    try:
        for _ in range(3):
            binding.gc_build_cache(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse,
                                   out.dQ, out.dP, out.pos_logit, out.ws, out.dev_status)
        torch.cuda.synchronize()
        for call in range(3):
            fwd, dq, dp = binding.gc_profile_read(call)
            assert fwd == 0.0 and 0.0 < dq < 50.0 and 0.0 < dp < 50.0      # milliseconds
        assert binding.gc_profile_read() == binding.gc_profile_read(2)
        with pytest.raises(binding.GradCacheError) as e:
            binding.gc_profile_read(3)
        assert e.value.status == 9
    finally:
        binding.gc_profile_enable(0)
    assert int(out.dev_status.item()) == 0


def _guarded(need, pad=4096):
    buf = torch.full((need + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
    off = (-buf.data_ptr()) % 256 + 256
    return buf, off, buf[off:off + need]


@pytest.mark.parametrize("B,N,d", [(300, 500, 128), (300, 520, 768), (130, 90, 1024)])
def test_workspace_canaries_of_every_bf16_plan(binding, B, N, d, plan_mode):
    """Narrow rows with a fixed row scale, four-CTA sweeps, paired wide rows: gc_build_cache,
    the rank-local calls and gc_cache_apply stay inside the workspace sizes they report."""
    prob = inputs.random_problem(B, N, d, "bf16", seed=B, tau=0.5, scale=d ** -0.5)
    Q, P, pos = to_device(prob)
    code = binding.GC_BF16
    out = binding.Outputs(B, N, d, code)
    buf, off, ws = _guarded(binding.gc_workspace_bytes(binding.GC_OP_BUILD, B, N, d, code))
    binding.gc_build_cache(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse, out.dQ,
                           out.dP, out.pos_logit, ws, out.dev_status)
    torch.cuda.synchronize()
    assert bool((buf[:off] == 0xA5).all()) and bool((buf[off + ws.numel():] == 0xA5).all())

    q0, b, p0, n = B // 3, B - B // 3, 0, N // 2
    buf, off, ws = _guarded(binding.gc_shard_workspace_bytes(B, N, d, code, b, n))
    part = torch.zeros(1, device="cuda")
    lse = out.row_lse.clone()
    binding.gc_shard_fwd_dq(Q, P, pos, prob.tau, q0, b, part, lse, out.dQ[q0:q0 + b], ws=ws)
    binding.gc_shard_dp(Q, P, pos, prob.tau, out.row_lse, p0, n, out.dP[p0:p0 + n], ws=ws)
    torch.cuda.synchronize()
    assert bool((buf[:off] == 0xA5).all()) and bool((buf[off + ws.numel():] == 0xA5).all())

    d_in = 192
    X = torch.zeros(B, d_in, dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros(d, d_in, device="cuda")
    buf, off, ws = _guarded(binding.gc_cache_apply_workspace_bytes(B, d, d_in))
    binding.gc_cache_apply(out.dQ, X, dW, False, ws=ws)
    torch.cuda.synchronize()
    assert bool((buf[:off] == 0xA5).all()) and bool((buf[off + ws.numel():] == 0xA5).all())
    assert int(out.dev_status.item()) == 0
