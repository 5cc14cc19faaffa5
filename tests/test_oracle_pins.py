"""Pins for the CPU oracle: checks against what the paper's equations and plain mathematics fix,
none of which re-use the oracle's own formulas.  A dropped term, wrong sign, wrong index,
transposed operand or misplaced temperature fails at least one of these."""
import math
import os

import numpy as np
import pytest

from paper_2101_06983_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _fd_grad(fn, X, h=1e-6):
    """Central finite differences of the scalar fn with respect to every entry of X."""
    g = np.zeros_like(X)
    it = np.nditer(X, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        old = X[idx]
        X[idx] = old + h
        fp = fn()
        X[idx] = old - h
        fm = fn()
        X[idx] = old
        g[idx] = (fp - fm) / (2 * h)
    return g


def _rand(seed, B, N, d, mask, dup=True):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, d))
    P = rng.standard_normal((N, d))
    pos = rng.integers(0, N, size=B)
    if not dup:
        pos = rng.permutation(N)[:B]
    if mask:
        for i in range(B):
            if pos[i] == i:
                pos[i] = (i + 1) % N
    return Q, P, pos.astype(np.int32)


# ---- Eq. 5-7 are the derivative of Eq. 1: central finite differences ------------------------
@pytest.mark.parametrize("tau", [1.0, 0.1])
@pytest.mark.parametrize("mask", [0, 1])
@pytest.mark.parametrize("shape", [(3, 6, 4), (4, 8, 5), (1, 2, 1), (4, 4, 3)])
def test_gradients_match_finite_differences(oracle, tau, mask, shape):
    B, N, d = shape
    Q, P, pos = _rand(11 + B + 7 * N, B, N, d, mask)
    Q *= 0.7
    P *= 0.7
    out = oracle.build_cache(Q, P, pos, tau, mask)
    gq = _fd_grad(lambda: oracle.loss_only(Q, P, pos, tau, mask), Q)
    gp = _fd_grad(lambda: oracle.loss_only(Q, P, pos, tau, mask), P)
    scale = max(np.abs(gq).max(), np.abs(gp).max())
    assert np.abs(out["dQ"] - gq).max() <= 1e-7 * max(scale, 1.0)
    assert np.abs(out["dP"] - gp).max() <= 1e-7 * max(scale, 1.0)


def test_duplicate_positives_sum_in_epsilon(oracle):
    """Eq. 7 with several k sharing r_k = j: differentiation gives the SUM of those f(s_k)."""
    B, N, d = 4, 5, 3
    Q, P, _ = _rand(5, B, N, d, 0)
    pos = np.array([2, 2, 2, 0], np.int32)
    out = oracle.build_cache(Q, P, pos, 0.5, 0)
    gp = _fd_grad(lambda: oracle.loss_only(Q, P, pos, 0.5, 0), P)
    assert np.abs(out["dP"] - gp).max() <= 1e-7


@pytest.mark.parametrize("tau", [1.0, 0.1])
def test_shared_rows_gradient_is_dq_plus_dp(oracle, tau):
    """Q and P the same rows X with the diagonal masked: dL/dX = dQ + dP."""
    n, d = 6, 4
    rng = np.random.default_rng(3)
    X = rng.standard_normal((n, d))
    X /= np.linalg.norm(X, axis=1, keepdims=True)
    pos = ((np.arange(n) + n // 2) % n).astype(np.int32)
    out = oracle.build_cache(X, X, pos, tau, 1)
    g = _fd_grad(lambda: oracle.loss_only(X, X, pos, tau, 1), X)
    assert np.abs(out["dQ"] + out["dP"] - g).max() <= 2e-7 * max(1.0, np.abs(g).max())


# ---- hand-worked rational example (tests/golden/rational_softmax.txt) ------------------------
def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "rational_softmax.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            vals[k] = [float(x) for x in v]
    return vals


def test_hand_worked_rational_example(oracle):
    g = _golden()
    ln = math.log
    Q = np.array([[ln(1), ln(2), ln(3)], [ln(4), ln(1), ln(1)]])
    P = np.eye(3)
    pos = np.array([2, 0], np.int32)
    out = oracle.build_cache(Q, P, pos, 1.0, 0)
    assert math.exp(2 * out["loss"]) == pytest.approx(g["loss_times_2_exp"][0], rel=1e-14)
    G = np.array(g["G_times_12"]).reshape(2, 3) / 12.0
    np.testing.assert_allclose(out["dQ"], G, rtol=0, atol=1e-15)
    C = np.array(g["dP_coeff_times_12"]).reshape(3, 2) / 12.0
    np.testing.assert_allclose(out["dP"], C @ Q, rtol=0, atol=1e-15)
    np.testing.assert_allclose(out["row_lse"], [ln(6), ln(6)], rtol=1e-15)
    np.testing.assert_allclose(out["pos_logit"], [ln(3), ln(4)], rtol=1e-15)


# ---- rows of softmax - onehot sum to zero (Eq. 4) ---------------------------------------------
@pytest.mark.parametrize("mask", [0, 1])
def test_rows_of_G_sum_to_zero(oracle, mask):
    """With P = I (d = N) row i of dQ * tau is row i of G, so its entries must sum to zero."""
    B, N = 7, 9
    rng = np.random.default_rng(8)
    Q = rng.standard_normal((B, N)) * 2.0
    P = np.eye(N)
    pos = ((np.arange(B) + 3) % N).astype(np.int32)
    tau = 0.3
    out = oracle.build_cache(Q, P, pos, tau, mask)
    G = out["dQ"] * tau
    assert np.abs(G.sum(axis=1)).max() <= 1e-15
    if mask:
        assert np.all(np.diag(G[:, :B]) == 0.0)   # masked pair contributes exactly nothing
    # p_ij in (0, 1): off-positive entries positive, the positive entry in (-1/B, 0)
    for i in range(B):
        assert -1.0 / B < G[i, pos[i]] < 0.0


@pytest.mark.parametrize("mask", [0, 1])
def test_gradient_identities(oracle, mask):
    """sum_j dP_j = 0 and sum_i <Q_i, dQ_i> = sum_j <P_j, dP_j> (both equal sum_ij G_ij S_ij)."""
    Q, P, pos = _rand(21, 9, 13, 6, mask)
    out = oracle.build_cache(Q, P, pos, 0.7, mask)
    assert np.abs(out["dP"].sum(axis=0)).max() <= 1e-15 * 50
    assert (Q * out["dQ"]).sum() == pytest.approx((P * out["dP"]).sum(), rel=1e-12, abs=1e-15)


# ---- closed forms ----------------------------------------------------------------------------
@pytest.mark.parametrize("tau", [1.0, 0.25])
def test_identical_representations(oracle, tau):
    """All logits equal: L = log N, dQ = 0, dP_j = (B/N - c_j) q / (B tau), c_j = #{i: r_i=j}."""
    B, N, d = 6, 10, 4
    q = np.array([0.3, -0.2, 0.5, 0.1])
    Q = np.tile(q, (B, 1))
    P = np.tile(q, (N, 1))
    pos = np.array([0, 0, 3, 4, 9, 9], np.int32)
    out = oracle.build_cache(Q, P, pos, tau, 0)
    assert out["loss"] == pytest.approx(math.log(N), rel=1e-14)
    assert np.abs(out["dQ"]).max() <= 1e-16
    c = np.bincount(pos, minlength=N)
    expect = ((B / N - c) / (B * tau))[:, None] * q[None, :]
    np.testing.assert_allclose(out["dP"], expect, rtol=0, atol=1e-15)
    # self mask: one column fewer in every denominator
    pos_m = np.array([1, 0, 3, 4, 9, 9], np.int32)
    out_m = oracle.build_cache(np.tile(q, (N, 1)), P, np.r_[pos_m, [0, 0, 0, 0]].astype(np.int32),
                               tau, 1)
    assert out_m["loss"] == pytest.approx(math.log(N - 1), rel=1e-14)


def test_one_query_two_passages_is_logistic_loss(oracle):
    """B=1, N=2, d=1: L = log(1 + exp((s_neg - s_pos))) with the sigmoid as derivative."""
    q, p_pos, p_neg, tau = 0.7, 1.3, -0.4, 0.5
    out = oracle.build_cache(np.array([[q]]), np.array([[p_pos], [p_neg]]),
                             np.array([0], np.int32), tau, 0)
    z = (q * p_neg - q * p_pos) / tau
    assert out["loss"] == pytest.approx(math.log1p(math.exp(z)), rel=1e-14)
    sig = 1.0 / (1.0 + math.exp(-z))
    assert out["dQ"][0, 0] == pytest.approx(sig * (p_neg - p_pos) / tau, rel=1e-13)
    assert out["dP"][0, 0] == pytest.approx(-sig * q / tau, rel=1e-13)
    assert out["dP"][1, 0] == pytest.approx(sig * q / tau, rel=1e-13)


# ---- symmetries ------------------------------------------------------------------------------
def test_scale_and_permutation_symmetry(oracle):
    Q, P, pos = _rand(4, 5, 8, 3, 0)
    a = oracle.build_cache(Q, P, pos, 0.5, 0)
    b = oracle.build_cache(4.0 * Q, P, pos, 2.0, 0)       # L(cQ, P, c tau) = L(Q, P, tau)
    assert b["loss"] == pytest.approx(a["loss"], rel=1e-13)
    np.testing.assert_allclose(b["dP"], a["dP"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(b["dQ"] * 4.0, a["dQ"], rtol=1e-12, atol=1e-15)
    perm = np.random.default_rng(1).permutation(8)         # new row k holds old row perm[k]
    inv = np.argsort(perm)
    c = oracle.build_cache(Q, P[perm], inv[pos].astype(np.int32), 0.5, 0)
    assert c["loss"] == pytest.approx(a["loss"], rel=1e-13)
    np.testing.assert_allclose(c["dQ"], a["dQ"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(c["dP"], a["dP"][perm], rtol=1e-12, atol=1e-15)


# ---- library special case: float64 cross-entropy with autograd -------------------------------
@pytest.mark.parametrize("mask", [0, 1])
def test_against_autograd_cross_entropy(oracle, mask):
    torch = pytest.importorskip("torch")
    B, N, d, tau = 37, 53, 24, 0.2
    Q, P, pos = _rand(17, B, N, d, mask)
    Q *= 0.4
    P *= 0.4
    out = oracle.build_cache(Q, P, pos, tau, mask)
    q = torch.tensor(Q, dtype=torch.float64, requires_grad=True)
    p = torch.tensor(P, dtype=torch.float64, requires_grad=True)
    S = q @ p.T / tau
    if mask:
        S = S.masked_fill(torch.eye(B, N, dtype=torch.bool), float("-inf"))
    loss = torch.nn.functional.cross_entropy(S, torch.tensor(pos, dtype=torch.long))
    loss.backward()
    assert out["loss"] == pytest.approx(loss.item(), rel=1e-13)
    np.testing.assert_allclose(out["dQ"], q.grad.numpy(), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(out["dP"], p.grad.numpy(), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(out["row_lse"], torch.logsumexp(S, dim=1).detach().numpy(),
                               rtol=1e-13)
    # the row-sampled entry points agree with the same library result
    rows = np.array([0, 5, 36, 5], np.int64)
    qr = oracle.query_rows(Q, P, pos, rows, tau, mask)
    np.testing.assert_allclose(qr["dQ"], q.grad.numpy()[rows], rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(qr["pos_logit"], S.detach().numpy()[rows, pos[rows]], rtol=1e-13)
    prow = np.array([52, 0, 7], np.int64)
    full_lse = torch.logsumexp(S, dim=1).detach().numpy()
    dp = oracle.passage_rows(Q, P, pos, full_lse, prow, tau, mask)
    np.testing.assert_allclose(dp, p.grad.numpy()[prow], rtol=1e-10, atol=1e-14)


# ---- the row-sampled entry points (query_rows, passage_rows) -----------------------------------
def test_row_sampled_entry_points_on_the_hand_worked_example(oracle):
    """Same rational instance as above, read off the fixture: query_rows must give rows of G (P is
    the identity) and passage_rows the hand-derived combinations of the query rows."""
    g = _golden()
    ln = math.log
    Q = np.array([[ln(1), ln(2), ln(3)], [ln(4), ln(1), ln(1)]])
    P = np.eye(3)
    pos = np.array([2, 0], np.int32)
    G = np.array(g["G_times_12"]).reshape(2, 3) / 12.0
    C = np.array(g["dP_coeff_times_12"]).reshape(3, 2) / 12.0
    rows = np.array([1, 0, 1], np.int64)
    qr = oracle.query_rows(Q, P, pos, rows, 1.0, 0)
    np.testing.assert_allclose(qr["dQ"], G[rows], rtol=0, atol=1e-15)
    np.testing.assert_allclose(qr["row_lse"], [ln(6)] * 3, rtol=1e-15)
    np.testing.assert_allclose(qr["pos_logit"], [ln(4), ln(3), ln(4)], rtol=1e-15)
    prow = np.array([2, 0, 1, 2], np.int64)
    dp = oracle.passage_rows(Q, P, pos, np.array([ln(6), ln(6)]), prow, 1.0, 0)
    np.testing.assert_allclose(dp, (C @ Q)[prow], rtol=0, atol=1e-15)


@pytest.mark.parametrize("tau", [1.0, 0.1])
@pytest.mark.parametrize("mask", [0, 1])
def test_row_sampled_entry_points_match_finite_differences(oracle, tau, mask):
    """Rows of dQ from query_rows and rows of dP from passage_rows (fed the lse that query_rows
    itself returns for every query) against central finite differences of the loss of Eq. 1, and
    row for row against build_cache.  Rows are listed out of order and with a repeat."""
    B, N, d = 4, 8, 5
    Q, P, pos = _rand(11 + B + 7 * N, B, N, d, mask)
    Q *= 0.7
    P *= 0.7
    gq = _fd_grad(lambda: oracle.loss_only(Q, P, pos, tau, mask), Q)
    gp = _fd_grad(lambda: oracle.loss_only(Q, P, pos, tau, mask), P)
    scale = max(np.abs(gq).max(), np.abs(gp).max(), 1.0)
    all_rows = oracle.query_rows(Q, P, pos, np.arange(B, dtype=np.int64), tau, mask)
    rows = np.array([3, 0, 2, 3], np.int64)
    qr = oracle.query_rows(Q, P, pos, rows, tau, mask)
    assert np.abs(qr["dQ"] - gq[rows]).max() <= 1e-7 * scale
    prow = np.array([7, 1, 0, 4, 1], np.int64)
    dp = oracle.passage_rows(Q, P, pos, all_rows["row_lse"], prow, tau, mask)
    assert np.abs(dp - gp[prow]).max() <= 1e-7 * scale
    full = oracle.build_cache(Q, P, pos, tau, mask)
    np.testing.assert_allclose(qr["dQ"], full["dQ"][rows], rtol=0, atol=1e-14)
    np.testing.assert_allclose(qr["row_lse"], full["row_lse"][rows], rtol=0, atol=1e-14)
    np.testing.assert_allclose(qr["pos_logit"], full["pos_logit"][rows], rtol=0, atol=1e-14)
    np.testing.assert_allclose(dp, full["dP"][prow], rtol=0, atol=1e-14)


def test_row_sampled_entry_points_identical_representations(oracle):
    """All logits equal: lse = log N, dQ rows vanish, dP_j = (B/N - c_j) q / (B tau)."""
    B, N, tau = 6, 10, 0.25
    q = np.array([0.3, -0.2, 0.5, 0.1])
    Q = np.tile(q, (B, 1))
    P = np.tile(q, (N, 1))
    pos = np.array([0, 0, 3, 4, 9, 9], np.int32)
    rows = np.array([5, 0, 2], np.int64)
    qr = oracle.query_rows(Q, P, pos, rows, tau, 0)
    s = float(q @ q) / tau
    np.testing.assert_allclose(qr["row_lse"], s + math.log(N), rtol=1e-14)
    np.testing.assert_allclose(qr["pos_logit"], s, rtol=1e-14)
    assert np.abs(qr["dQ"]).max() <= 1e-16
    c = np.bincount(pos, minlength=N)
    expect = ((B / N - c) / (B * tau))[:, None] * q[None, :]
    prow = np.array([9, 0, 1, 3], np.int64)
    dp = oracle.passage_rows(Q, P, pos, np.full(B, s + math.log(N)), prow, tau, 0)
    np.testing.assert_allclose(dp, expect[prow], rtol=0, atol=1e-15)


# ---- the paper's exactness claim on a linear encoder (Eq. 2, Eq. 8-9) -------------------------
def test_cached_chunked_gradient_equals_full_batch_gradient(oracle):
    """f(s) = W_f s, g(t) = W_g t.  Full-batch dL/dW_f (by finite differences on W_f) equals the
    sum over sub-batches of (cached u_i)(ds_i)^T; per-chunk losses (gradient accumulation) do
    not reproduce it."""
    rng = np.random.default_rng(2101)
    B, N, din, d, tau = 8, 16, 5, 4, 0.5
    Xs = rng.standard_normal((B, din))
    Xt = rng.standard_normal((N, din))
    Wf = rng.standard_normal((d, din)) * 0.5
    Wg = rng.standard_normal((d, din)) * 0.5
    pos = (2 * np.arange(B)).astype(np.int32)

    def full_loss():
        return oracle.loss_only(Xs @ Wf.T, Xt @ Wg.T, pos, tau, 0)

    gWf = _fd_grad(full_loss, Wf)
    gWg = _fd_grad(full_loss, Wg)
    cache = oracle.build_cache(Xs @ Wf.T, Xt @ Wg.T, pos, tau, 0)      # Step 2
    accWf = np.zeros_like(Wf)
    for lo in range(0, B, 3):                                            # Step 3, ragged chunks
        accWf += cache["dQ"][lo:lo + 3].T @ Xs[lo:lo + 3]                # Eq. 8
    accWg = np.zeros_like(Wg)
    for lo in range(0, N, 5):
        accWg += cache["dP"][lo:lo + 5].T @ Xt[lo:lo + 5]                # Eq. 9
    np.testing.assert_allclose(accWf, cache["dQ"].T @ Xs, rtol=1e-12, atol=1e-15)
    assert np.abs(accWf - gWf).max() <= 1e-7 * max(1.0, np.abs(gWf).max())
    assert np.abs(accWg - gWg).max() <= 1e-7 * max(1.0, np.abs(gWg).max())

    # plain accumulation: each chunk of 4 queries only sees its own 8 passages
    naive = np.zeros_like(Wf)
    for c in range(2):
        qs, ps = slice(4 * c, 4 * c + 4), slice(8 * c, 8 * c + 8)
        sub = oracle.build_cache(Xs[qs] @ Wf.T, Xt[ps] @ Wg.T,
                                 (2 * np.arange(4)).astype(np.int32), tau, 0)
        naive += 0.5 * sub["dQ"].T @ Xs[qs]
    assert np.abs(naive - gWf).max() > 1e-3


# ---- magnitudes under the workload generators --------------------------------------------------
def test_generator_magnitudes(oracle):
    p = inputs.config(0)
    out = oracle.build_cache(p.Q, p.P, p.pos_idx, p.tau, p.mask_mode, grads=False)
    # positive logit ~0.8, hard negative ~0.5, the other 126 ~N(0, 1/d)
    expect = math.log(126 + math.exp(0.8) + math.exp(0.5)) - 0.8
    assert abs(out["loss"] - expect) < 0.08
    assert abs(out["pos_logit"].mean() - 0.8) < 0.05
    s = inputs.simclr_batch(256, 128, "bf16", seed=5)
    o = oracle.build_cache(s.Q, s.P, s.pos_idx, s.tau, s.mask_mode, grads=False)
    # partner cosine ~ 1/1.09, so the positive logit is ~9.2 at tau = 0.1
    assert abs(o["pos_logit"].mean() - 10.0 / 1.09) < 0.3
    assert 0.0 < o["loss"] < 2.0


def test_rejects_bad_positives(oracle):
    Q, P, pos = _rand(1, 3, 4, 2, 0)
    bad = pos.copy()
    bad[1] = 4
    with pytest.raises(ValueError):
        oracle.build_cache(Q, P, bad, 1.0, 0)
    bad[1] = 1                                   # equals the masked column of row 1
    with pytest.raises(ValueError):
        oracle.build_cache(Q, P, bad, 1.0, 1)


# ---- Step 3 for a linear encoder (Eq. 8-9): oracle.cache_apply ----------------------------------
def test_cache_apply_hand_worked_example(oracle):
    """rows = 2, d = 2, d_in = 3 with small integers: dW[a][b] = sum_i U[i][a] X[i][b], written
    out by hand (u_1 x_1^T + u_2 x_2^T); a transposed operand or swapped index changes it."""
    U = np.array([[1.0, -2.0], [3.0, 4.0]])
    X = np.array([[5.0, 0.0, -1.0], [2.0, 7.0, 1.0]])
    # u_1 x_1^T = [[5, 0, -1], [-10, 0, 2]];  u_2 x_2^T = [[6, 21, 3], [8, 28, 4]]
    want = np.array([[11.0, 21.0, 2.0], [-2.0, 28.0, 6.0]])
    got = oracle.cache_apply(U, X)
    assert got.shape == (2, 3) and np.array_equal(got, want)
    # accumulation adds in place; a second call with the rows swapped gives the same sum
    acc = want.copy()
    oracle.cache_apply(U[::-1], X[::-1], acc)
    assert np.array_equal(acc, 2 * want)


def test_cache_apply_chunks_reproduce_full_batch_parameter_gradient(oracle):
    """Eq. 8-9 through the oracle's own Step-3 routine: accumulating cache_apply over ragged
    sub-batches gives dL/dW_f and dL/dW_g of the FULL batch, checked against central finite
    differences of the full-batch loss with respect to the encoder matrices (tau != 1, so a
    dropped 1/tau or 1/B anywhere between Step 2 and Step 3 shows)."""
    rng = np.random.default_rng(68983)
    B, N, din, d, tau = 7, 14, 6, 3, 0.7
    Xs = rng.standard_normal((B, din))
    Xt = rng.standard_normal((N, din))
    Wf = rng.standard_normal((d, din)) * 0.4
    Wg = rng.standard_normal((d, din)) * 0.4
    pos = (2 * np.arange(B)).astype(np.int32)

    def full_loss():
        return oracle.loss_only(Xs @ Wf.T, Xt @ Wg.T, pos, tau, 0)

    gWf = _fd_grad(full_loss, Wf)
    gWg = _fd_grad(full_loss, Wg)
    cache = oracle.build_cache(Xs @ Wf.T, Xt @ Wg.T, pos, tau, 0)
    accWf = oracle.cache_apply(cache["dQ"][0:3], Xs[0:3])
    for lo in (3, 5):
        oracle.cache_apply(cache["dQ"][lo:lo + 2], Xs[lo:lo + 2], accWf)
    accWg = oracle.cache_apply(cache["dP"][0:9], Xt[0:9])
    oracle.cache_apply(cache["dP"][9:], Xt[9:], accWg)
    assert np.abs(accWf - gWf).max() <= 1e-7 * max(1.0, np.abs(gWf).max())
    assert np.abs(accWg - gWg).max() <= 1e-7 * max(1.0, np.abs(gWg).max())
    # one call over the whole batch is the same sum
    np.testing.assert_allclose(oracle.cache_apply(cache["dQ"], Xs), accWf, rtol=1e-12, atol=1e-15)
