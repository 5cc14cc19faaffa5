"""Pins for oracle.build_variant (the loss variants Section 3.3 leaves to automatic
differentiation): none of them re-uses the oracle's formulas.  Central finite differences of the
variant's own loss with respect to every entry of Q and P and to tau; Euler's identity for the
joint scaling (Q, tau) -> (cQ, c tau); cosine gradients orthogonal to their rows and invariant
losses under row scaling; the role-swap symmetry of the two-direction loss; reduction to the base
oracle; a hand-worked two-positive example."""
import math

import numpy as np
import pytest

from test_oracle_pins import _fd_grad, _rand


def _lists(pos):
    return [[int(v)] for v in pos]


def _multi(rng, B, N, mask):
    out = []
    for i in range(B):
        k = int(rng.integers(1, 4))
        cand = [j for j in range(N) if not (mask and j == i)]
        out.append(sorted(rng.choice(cand, size=min(k, len(cand)), replace=False).tolist()))
    return out


@pytest.mark.parametrize("cosine", [False, True])
@pytest.mark.parametrize("two", [False, True])
@pytest.mark.parametrize("mask", [0, 1])
@pytest.mark.parametrize("tau", [1.0, 0.2])
def test_variant_gradients_match_finite_differences(oracle, cosine, two, mask, tau):
    B, N, d = 4, 7, 5
    Q, P, pos = _rand(31 + 2 * cosine + two, B, N, d, mask, dup=not two)
    Q *= 0.8
    P *= 0.8
    rng = np.random.default_rng(5)
    positives = _lists(pos) if two else _multi(rng, B, N, mask)
    out = oracle.build_variant(Q, P, positives, tau, mask, cosine, two)

    def loss(t=tau):
        return oracle.build_variant(Q, P, positives, t, mask, cosine, two)["loss"]

    gq = _fd_grad(loss, Q)
    gp = _fd_grad(loss, P)
    scale = max(np.abs(gq).max(), np.abs(gp).max(), 1.0)
    assert np.abs(out["dQ"] - gq).max() <= 2e-7 * scale
    assert np.abs(out["dP"] - gp).max() <= 2e-7 * scale
    h = 1e-6
    fd_tau = (loss(tau + h) - loss(tau - h)) / (2 * h)
    assert abs(out["dtau"] - fd_tau) <= 1e-6 * max(1.0, abs(fd_tau))


@pytest.mark.parametrize("two", [False, True])
def test_euler_identity_for_joint_scaling(oracle, two):
    """L(cQ, P, c tau) = L(Q, P, tau) for the dot product: d/dc at c = 1 gives
    sum_i <Q_i, dQ_i> + tau dL/dtau = 0, and likewise with P."""
    Q, P, pos = _rand(9, 5, 8, 4, 0, dup=not two)
    out = oracle.build_variant(Q, P, _lists(pos), 0.6, 0, False, two)
    assert abs((Q * out["dQ"]).sum() + 0.6 * out["dtau"]) <= 1e-12
    assert abs((P * out["dP"]).sum() + 0.6 * out["dtau"]) <= 1e-12


def test_cosine_is_scale_invariant_and_gradients_are_tangent(oracle):
    Q, P, pos = _rand(10, 5, 9, 6, 1)
    positives = _lists(pos)
    a = oracle.build_variant(Q, P, positives, 0.3, 1, True, False)
    rq = np.linspace(0.5, 3.0, 5)[:, None]
    rp = np.linspace(2.0, 0.25, 9)[:, None]
    b = oracle.build_variant(Q * rq, P * rp, positives, 0.3, 1, True, False)
    assert b["loss"] == pytest.approx(a["loss"], rel=1e-13)
    assert b["dtau"] == pytest.approx(a["dtau"], rel=1e-12)
    np.testing.assert_allclose(b["dQ"] * rq, a["dQ"], rtol=1e-11, atol=1e-14)   # 1/|x| Jacobian
    np.testing.assert_allclose(b["dP"] * rp, a["dP"], rtol=1e-11, atol=1e-14)
    assert np.abs((Q * a["dQ"]).sum(axis=1)).max() <= 1e-14      # no component along the row
    assert np.abs((P * a["dP"]).sum(axis=1)).max() <= 1e-14
    # unit rows: cosine and dot product agree on the loss (the gradients differ by the projection)
    Qu = Q / np.linalg.norm(Q, axis=1, keepdims=True)
    Pu = P / np.linalg.norm(P, axis=1, keepdims=True)
    c = oracle.build_variant(Qu, Pu, positives, 0.3, 1, False, False)
    assert c["loss"] == pytest.approx(a["loss"], rel=1e-13)


def test_two_direction_loss_is_symmetric_under_role_swap(oracle):
    """B = N pairs with a permutation as relevance map: swapping the roles of queries and passages
    (and inverting the map) leaves the loss unchanged and exchanges the gradients."""
    n, d = 6, 4
    rng = np.random.default_rng(12)
    Q, P = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    perm = rng.permutation(n)
    inv = np.argsort(perm)
    a = oracle.build_variant(Q, P, _lists(perm), 0.5, 0, False, True)
    b = oracle.build_variant(P, Q, _lists(inv), 0.5, 0, False, True)
    assert b["loss"] == pytest.approx(a["loss"], rel=1e-13)
    np.testing.assert_allclose(b["dQ"], a["dP"], rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(b["dP"], a["dQ"], rtol=1e-11, atol=1e-14)
    assert b["dtau"] == pytest.approx(a["dtau"], rel=1e-12)
    # and it is the mean of the two one-direction losses of the base oracle
    row = oracle.build_cache(Q, P, perm.astype(np.int32), 0.5, 0)
    col = oracle.build_cache(P, Q, inv.astype(np.int32), 0.5, 0)
    assert a["loss"] == pytest.approx(0.5 * (row["loss"] + col["loss"]), rel=1e-13)
    np.testing.assert_allclose(a["dQ"], 0.5 * (row["dQ"] + col["dP"]), rtol=1e-11, atol=1e-14)


def test_two_direction_with_extra_passages(oracle):
    """N > B: passages that are nobody's positive take part in the row softmax only.  With the B
    positive passages gathered, the column half is the base oracle with the roles swapped."""
    B, N, d, tau = 4, 9, 3, 0.7
    Q, P, _ = _rand(3, B, N, d, 0)
    pos = np.array([7, 2, 5, 0], np.int32)
    a = oracle.build_variant(Q, P, _lists(pos), tau, 0, False, True)
    row = oracle.build_cache(Q, P, pos, tau, 0)
    col = oracle.build_cache(P[pos], Q, np.arange(B, dtype=np.int32), tau, 0)
    assert a["loss"] == pytest.approx(0.5 * (row["loss"] + col["loss"]), rel=1e-13)
    np.testing.assert_allclose(a["dQ"], 0.5 * (row["dQ"] + col["dP"]), rtol=1e-11, atol=1e-14)
    want_dp = 0.5 * row["dP"]
    want_dp[pos] += 0.5 * col["dQ"]
    np.testing.assert_allclose(a["dP"], want_dp, rtol=1e-11, atol=1e-14)


def test_single_positive_reduces_to_the_base_oracle(oracle):
    Q, P, pos = _rand(14, 6, 11, 5, 1)
    a = oracle.build_variant(Q, P, _lists(pos), 0.4, 1, False, False)
    b = oracle.build_cache(Q, P, pos, 0.4, 1)
    assert a["loss"] == pytest.approx(b["loss"], rel=1e-14)
    np.testing.assert_allclose(a["dQ"], b["dQ"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(a["dP"], b["dP"], rtol=1e-12, atol=1e-15)


def test_two_positives_hand_worked(oracle):
    """P = I_3, Q = [[ln 1, ln 2, ln 3]], positives {0, 2}: p = (1/6, 2/6, 3/6);
    L = -(ln(1/6) + ln(3/6))/2; G = p - (1/2, 0, 1/2) = (-1/3, 1/3, 0); dQ = G (tau = 1, B = 1);
    dtau = -sum G S = (1/3) ln 1 - (1/3) ln 2 = -(ln 2)/3."""
    ln = math.log
    Q = np.array([[ln(1), ln(2), ln(3)]])
    out = oracle.build_variant(Q, np.eye(3), [[0, 2]], 1.0, 0, False, False)
    assert out["loss"] == pytest.approx(-(ln(1 / 6) + ln(3 / 6)) / 2, rel=1e-14)
    np.testing.assert_allclose(out["dQ"], [[-1 / 3, 1 / 3, 0.0]], rtol=0, atol=1e-15)
    assert out["dtau"] == pytest.approx(-ln(2) / 3, rel=1e-13)
    np.testing.assert_allclose(out["dP"], np.array([[-1 / 3], [1 / 3], [0.0]]) * Q, rtol=0,
                               atol=1e-15)


def test_variant_rejects_bad_positives(oracle):
    Q, P, _ = _rand(1, 3, 4, 2, 0)
    for bad in ([[0], [], [1]], [[0], [4], [1]], [[0], [1, 1], [2]]):
        with pytest.raises(ValueError):
            oracle.build_variant(Q, P, bad, 1.0, 0)
    with pytest.raises(ValueError):
        oracle.build_variant(Q, P, [[0], [1], [2]], 1.0, 1)          # positives on the mask
    with pytest.raises(ValueError):
        oracle.build_variant(Q, P, [[0, 1], [1], [2]], 1.0, 0, False, True)
