"""Pins for the oracle's Distance Gradient Cache (Section 5, Eq. 10-13): w_ij = dL/dd_ij by
central finite differences in every distance; for the dot product the two caches link up
(Eq. 12-13 reduce to Eq. 5-7); rows of w sum to zero; Eq. 11 on a bilinear distance
Phi(f, g) = f^T Omega g, sub-batch by sub-batch, against finite differences in Omega."""
import numpy as np
import pytest

from test_oracle_pins import _fd_grad, _rand


@pytest.mark.parametrize("tau", [1.0, 0.3])
@pytest.mark.parametrize("mask", [0, 1])
def test_w_is_the_derivative_of_the_loss_in_every_distance(oracle, tau, mask):
    B, N = 4, 7
    rng = np.random.default_rng(4)
    D = rng.standard_normal((B, N))
    _, _, pos = _rand(2, B, N, 2, mask)
    W = oracle.dist_w(D, pos, tau, mask)
    fd = _fd_grad(lambda: oracle.dist_loss(D, pos, tau, mask)["loss"], D)
    assert np.abs(W - fd).max() <= 1e-8
    assert np.abs(W.sum(axis=1)).max() <= 1e-15
    if mask:
        assert np.all(np.diag(W) == 0.0)


@pytest.mark.parametrize("mask", [0, 1])
def test_dot_product_links_the_two_caches(oracle, mask):
    """d_ij = <f_i, g_j>: dd_ij/df_i = g_j, so Eq. 12 is u_i = sum_j w_ij g_j = dQ_i of Eq. 5 and
    Eq. 13 is v_j = sum_i w_ij f_i = dP_j of Eq. 6-7; the loss and lse agree as well."""
    Q, P, pos = _rand(6, 5, 9, 4, mask)
    tau = 0.4
    base = oracle.build_cache(Q, P, pos, tau, mask)
    D = Q @ P.T
    out = oracle.dist_loss(D, pos, tau, mask)
    W = oracle.dist_w(D, pos, tau, mask)
    assert out["loss"] == pytest.approx(base["loss"], rel=1e-14)
    np.testing.assert_allclose(out["row_lse"], base["row_lse"], rtol=1e-14)
    np.testing.assert_allclose(W @ P, base["dQ"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(W.T @ Q, base["dP"], rtol=1e-12, atol=1e-15)


def test_eq_11_on_a_bilinear_distance_by_sub_batches(oracle):
    """Phi(f, g) = f^T Omega g.  dL/dOmega = sum over sub-batch pairs of F_S^T W_ST G_T (Eq. 11)
    equals the finite-difference gradient of the full-batch loss in Omega, and the representation
    gradients of Eq. 12-13, u = W (G Omega^T), v = W^T (F Omega), equal finite differences too."""
    rng = np.random.default_rng(68)
    B, N, df, dg, tau = 5, 8, 3, 4, 0.6
    F, G = rng.standard_normal((B, df)), rng.standard_normal((N, dg))
    Om = rng.standard_normal((df, dg)) * 0.5
    pos = np.array([1, 0, 7, 3, 3], np.int32)

    def loss():
        return oracle.dist_loss(F @ Om @ G.T, pos, tau, 0)["loss"]

    W = oracle.dist_w(F @ Om @ G.T, pos, tau, 0)
    acc = np.zeros_like(Om)
    for i0 in range(0, B, 2):                      # ragged sub-batches of queries and passages
        for j0 in range(0, N, 3):
            acc += F[i0:i0 + 2].T @ W[i0:i0 + 2, j0:j0 + 3] @ G[j0:j0 + 3]
    assert np.abs(acc - _fd_grad(loss, Om)).max() <= 1e-8
    assert np.abs(W @ (G @ Om.T) - _fd_grad(loss, F)).max() <= 1e-8
    assert np.abs(W.T @ (F @ Om) - _fd_grad(loss, G)).max() <= 1e-8
