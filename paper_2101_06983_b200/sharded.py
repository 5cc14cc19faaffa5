"""Step 2 across several GPUs (Section 3.4 of the paper), one process per GPU.

Each rank holds the representations of its own examples.  One all-gather makes all of them
available everywhere (the paper's single extra communication); the loss is defined over the
gathered batch and every rank computes the gradients of its LOCAL representations only, so that
Step 3 needs no communication.  Where the paper recomputes the whole loss on every GPU, a rank
here does 1/world of it: the forward and dQ of its own queries against all passages, then, after
an all-gather of the B row logsumexps, dP of its own passages against all queries; the scalar
loss is an all-reduce of the ranks' shares.

This module is host-side plumbing (ranges, torch.distributed collectives, buffer layout); the two
compute steps are calls into the library (`binding.gc_shard_fwd_dq`, `binding.gc_shard_dp`), passed
in as `kernels` so that the plumbing can be exercised on CPU ranks with a stand-in.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_ranges(total: int, world: int) -> list[tuple[int, int]]:
    """Contiguous, balanced (first, count) ranges of `total` rows over `world` ranks: the first
    total % world ranks hold one row more."""
    base, rem = divmod(total, world)
    out, first = [], 0
    for r in range(world):
        n = base + (1 if r < rem else 0)
        out.append((first, n))
        first += n
    return out


def _world(group):
    if dist.is_available() and dist.is_initialized():
        return dist.get_world_size(group), dist.get_rank(group)
    return 1, 0


def gather_rows(local: torch.Tensor, counts: list[int], group=None) -> torch.Tensor:
    """All-gather of row blocks of unequal height: every rank contributes `local` (counts[rank]
    rows) and receives the concatenation in rank order.  Blocks are padded to the tallest one for
    the collective and compacted afterwards."""
    world, rank = _world(group)
    if world == 1:
        return local
    assert local.shape[0] == counts[rank]
    tall = max(counts)
    padded = local
    if local.shape[0] != tall:
        padded = local.new_zeros((tall,) + tuple(local.shape[1:]))
        padded[: local.shape[0]] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded.contiguous(), group=group)
    return torch.cat([parts[r][: counts[r]] for r in range(world)], dim=0)


class LibraryKernels:
    """The two rank-local compute steps as calls into libgradcache (CUDA tensors)."""

    def fwd_dq(self, Q_all, P_all, pos_all, tau, q0, q_count, loss_part, row_lse, dQ):
        from . import binding
        binding.gc_shard_fwd_dq(Q_all, P_all, pos_all, tau, q0, q_count, loss_part, row_lse, dQ)

    def dp(self, Q_all, P_all, pos_all, tau, row_lse, p0, p_count, dP):
        from . import binding
        binding.gc_shard_dp(Q_all, P_all, pos_all, tau, row_lse, p0, p_count, dP)


def sharded_build_cache(Q_local, P_local, pos_local, tau, B, N, kernels=None, group=None):
    """One sharded Step 2.

    Q_local [b x d], P_local [n x d]: this rank's rows of the batch, where rank r owns the r-th
    range of row_ranges(B, world) / row_ranges(N, world); pos_local [b] int32: positives of the
    local queries as row indices into the GATHERED passage matrix.  Returns
    (loss, row_lse_all [B], dQ_local [b x d], dP_local [n x d]); `loss` is the full-batch loss on
    every rank."""
    kernels = kernels or LibraryKernels()
    world, rank = _world(group)
    q_ranges, p_ranges = row_ranges(B, world), row_ranges(N, world)
    (q0, b), (p0, n) = q_ranges[rank], p_ranges[rank]
    if Q_local.shape[0] != b or P_local.shape[0] != n or pos_local.shape[0] != b:
        raise ValueError("local shapes do not match this rank's ranges")
    d = Q_local.shape[1]
    f32 = dict(dtype=torch.float32, device=Q_local.device)
    # the paper's one all-gather: all representations (and the relevance map) on every rank
    Q_all = gather_rows(Q_local, [c for _, c in q_ranges], group)
    P_all = gather_rows(P_local, [c for _, c in p_ranges], group)
    pos_all = gather_rows(pos_local, [c for _, c in q_ranges], group).contiguous()
    loss_part = torch.zeros(1, **f32)
    row_lse = torch.zeros(B, **f32)
    dQ = torch.empty(b, d, **f32)
    dP = torch.empty(n, d, **f32)
    kernels.fwd_dq(Q_all, P_all, pos_all, tau, q0, b, loss_part, row_lse, dQ)
    # every rank needs lse_i of every query for its passages' gradients: B floats in total
    lse_all = gather_rows(row_lse[q0:q0 + b], [c for _, c in q_ranges], group).contiguous()
    kernels.dp(Q_all, P_all, pos_all, tau, lse_all, p0, n, dP)
    if world > 1:
        dist.all_reduce(loss_part, op=dist.ReduceOp.SUM, group=group)
    return loss_part, lse_all, dQ, dP
