"""GPU parity of the tiled Distance Gradient Cache (Section 5, Eq. 10-13) against the oracle:
first with the dot product as the distance, where the two caches must link up (Eq. 12-13 give the
cache of Eq. 5-7), then with a bilinear distance Phi(f, g) = f^T Omega g whose blocks the test
computes itself, as a caller's network would, checking Eq. 11 sub-batch by sub-batch."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


def _blocks(total, step):
    return [(a, min(step, total - a)) for a in range(0, total, step)]


@pytest.mark.parametrize("B,N,d,dtype,tau,mask,sq,st", [
    (200, 330, 64, "f32", 0.5, 0, 48, 40), (130, 130, 72, "f32", 0.2, 1, 16, 8),
    (128, 256, 768, "bf16", 1.0, 0, 64, 96), (257, 300, 128, "bf16", 0.3, 0, 100, 77),
])
def test_dot_product_distance_links_the_two_caches(binding, oracle, B, N, d, dtype, tau, mask, sq, st):
    prob = inputs.random_problem(B, N, d, dtype, seed=B + N, tau=tau, scale=d ** -0.5,
                                 mask_mode=mask, shared=bool(mask))
    Q, P, pos = to_device(prob)
    D64 = prob.Q.astype(np.float64) @ prob.P.astype(np.float64).T
    ref = oracle.dist_loss(D64, prob.pos_idx, tau, mask)
    Wref = oracle.dist_w(D64, prob.pos_idx, tau, mask)
    base = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, tau, mask)

    dc = binding.DistanceCache(pos, B, N, tau, mask)
    Dblk = torch.empty(sq, st + 5, device="cuda")                 # padded leading dimension
    for i0, bq in _blocks(B, sq):
        for j0, bn in _blocks(N, st):
            binding.gc_dist_dot_block(Q, P, i0, bq, j0, bn, Dblk[:bq, :bn])
            dc.accumulate(Dblk[:bq, :bn], i0, j0)
    dc.finish()
    torch.cuda.synchronize()
    assert int(dc.dev_status.item()) == 0
    assert abs(dc.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    lse = dc.row_lse.cpu().numpy().astype(np.float64)
    assert np.abs(lse - ref["row_lse"]).max() <= 1e-5 * max(1.0, np.abs(ref["row_lse"]).max())

    Wblk = torch.empty(sq, st, device="cuda")
    U = torch.zeros(B, d, device="cuda")
    V = torch.zeros(N, d, device="cuda")
    werr = 0.0
    for i0, bq in _blocks(B, sq):
        for j0, bn in _blocks(N, st):
            binding.gc_dist_dot_block(Q, P, i0, bq, j0, bn, Dblk[:bq, :bn])
            dc.w_block(Dblk[:bq, :bn], i0, j0, Wblk[:bq, :bn])
            w = Wblk[:bq, :bn]
            werr = max(werr, float(np.abs(w.cpu().numpy() - Wref[i0:i0 + bq, j0:j0 + bn]).max()))
            # Eq. 12-13 for the dot product: dd_ij/df_i = g_j, dd_ij/dg_j = f_i
            U[i0:i0 + bq] += w @ P[j0:j0 + bn].float()
            V[j0:j0 + bn] += w.T @ Q[i0:i0 + bq].float()
    torch.cuda.synchronize()
    assert werr <= 1e-4 * np.abs(Wref).max()
    assert np.abs(U.cpu().numpy() - base["dQ"]).max() <= 1e-4 * np.abs(base["dQ"]).max()
    assert np.abs(V.cpu().numpy() - base["dP"]).max() <= 1e-4 * np.abs(base["dP"]).max()
    if mask:
        assert bool((torch.diagonal(torch.from_numpy(Wref)) == 0).all())


def test_bilinear_distance_parameter_gradient_by_sub_batches(binding, oracle):
    """Eq. 11 with Phi(f, g) = f^T Omega g: the test plays the caller's network (it computes the
    distance blocks and dPhi/dOmega), the library supplies lse, loss and the w blocks."""
    rng = np.random.default_rng(11)
    B, N, df, dg, tau = 150, 260, 24, 40, 0.7
    F = rng.standard_normal((B, df)).astype(np.float32)
    G = rng.standard_normal((N, dg)).astype(np.float32)
    Om = (rng.standard_normal((df, dg)) * 0.2).astype(np.float32)
    pos = (rng.permutation(N)[:B]).astype(np.int32)
    D64 = F.astype(np.float64) @ Om.astype(np.float64) @ G.astype(np.float64).T
    Wref = oracle.dist_w(D64, pos, tau, 0)
    want = F.astype(np.float64).T @ Wref @ G.astype(np.float64)
    ref = oracle.dist_loss(D64, pos, tau, 0)

    Fd, Gd, Od = (torch.from_numpy(a).cuda() for a in (F, G, Om))
    posd = torch.from_numpy(pos).cuda()
    dc = binding.DistanceCache(posd, B, N, tau)
    for i0, bq in _blocks(B, 16):
        for j0, bn in _blocks(N, 8 * 7):
            dc.accumulate((Fd[i0:i0 + bq] @ Od @ Gd[j0:j0 + bn].T).contiguous(), i0, j0)
    dc.finish()
    acc = torch.zeros(df, dg, dtype=torch.float64, device="cuda")
    for i0, bq in _blocks(B, 16):
        for j0, bn in _blocks(N, 8 * 7):
            Dblk = (Fd[i0:i0 + bq] @ Od @ Gd[j0:j0 + bn].T).contiguous()
            Wblk = torch.empty_like(Dblk)
            dc.w_block(Dblk, i0, j0, Wblk)
            acc += Fd[i0:i0 + bq].double().T @ Wblk.double() @ Gd[j0:j0 + bn].double()
    torch.cuda.synchronize()
    assert abs(dc.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    assert np.abs(acc.cpu().numpy() - want).max() <= 1e-4 * np.abs(want).max()


def test_distance_calls_refuse_bad_blocks(binding):
    pos = torch.zeros(8, dtype=torch.int32, device="cuda")
    dc = binding.DistanceCache(pos, 8, 16, 1.0)
    with pytest.raises(binding.GradCacheError) as e:
        dc.accumulate(torch.zeros(4, 4, device="cuda"), 6, 0)         # rows past the last query
    assert e.value.status == 2
    with pytest.raises(binding.GradCacheError) as e:
        binding.gc_dist_dot_block(torch.zeros(8, 12, device="cuda"), torch.zeros(16, 12, device="cuda"),
                                  0, 4, 0, 4, torch.zeros(4, 4, device="cuda"))
    assert e.value.status == 9
