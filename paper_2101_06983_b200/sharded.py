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

`ShardedStep` owns every buffer of a step (gathered representations, exchanged logsumexps,
outputs), allocated once for a problem size and reused by every call: a step allocates nothing.
The three gathers of the first exchange (Q, P, pos_idx) are issued together without waiting in
between and land directly in the gathered matrices when every rank owns the same number of rows;
ragged splits go through padded blocks that are compacted afterwards.
"""
from __future__ import annotations

import time

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


class _Gather:
    """All-gather of row blocks into one preallocated matrix [total x ...], rank order.  With
    equal blocks the collective writes the matrix itself; otherwise it writes padded blocks and
    `finish` compacts them (one copy per rank, no allocation)."""

    def __init__(self, counts, tail_shape, dtype, device, group):
        self.counts, self.group = list(counts), group
        self.world = len(self.counts)
        self.total, self.tall = sum(self.counts), max(self.counts)
        self.even = all(c == self.tall for c in self.counts)
        self.out = torch.empty((self.total,) + tuple(tail_shape), dtype=dtype, device=device)
        if not self.even:
            self.padded_in = torch.zeros((self.tall,) + tuple(tail_shape), dtype=dtype, device=device)
            self.padded_out = torch.empty((self.world * self.tall,) + tuple(tail_shape), dtype=dtype,
                                          device=device)

    def start(self, local, rank):
        """Issues the collective; returns a work handle (None for a single rank)."""
        if local.shape[0] != self.counts[rank]:
            raise ValueError("local block does not match this rank's range")
        if self.world == 1:
            self.out.copy_(local)
            return None
        if self.even:
            return dist.all_gather_into_tensor(self.out, local.contiguous(), group=self.group,
                                               async_op=True)
        self.padded_in[: local.shape[0]].copy_(local)
        return dist.all_gather_into_tensor(self.padded_out, self.padded_in, group=self.group,
                                           async_op=True)

    def finish(self, work):
        if work is not None:
            work.wait()
        if self.world > 1 and not self.even:
            first = 0
            for r, c in enumerate(self.counts):
                self.out[first:first + c].copy_(self.padded_out[r * self.tall: r * self.tall + c])
                first += c
        return self.out


def gather_rows(local: torch.Tensor, counts: list[int], group=None) -> torch.Tensor:
    """One-off all-gather of row blocks of unequal height (allocates; `ShardedStep` does not)."""
    world, rank = _world(group)
    if world == 1:
        return local
    g = _Gather(counts, local.shape[1:], local.dtype, local.device, group)
    return g.finish(g.start(local, rank))


class LibraryKernels:
    """The two rank-local compute steps as calls into libgradcache (CUDA tensors)."""

    def __init__(self):
        self.ws = None
        self.status = None

    def _scratch(self, Q_all, P_all, b, n):
        from . import binding
        if self.ws is None:
            B, d = Q_all.shape
            N = P_all.shape[0]
            code = binding._dtype_code(Q_all)
            need = max(binding.gc_shard_workspace_bytes(B, N, d, code, b, N),
                       binding.gc_shard_workspace_bytes(B, N, d, code, B, n), 256)
            self.ws = torch.empty(need, dtype=torch.uint8, device=Q_all.device)
            self.status = torch.zeros(1, dtype=torch.int32, device=Q_all.device)
        return self.ws, self.status

    def fwd_dq(self, Q_all, P_all, pos_all, tau, mask_mode, q0, q_count, p_count, loss_part, row_lse,
               dQ):
        from . import binding
        ws, status = self._scratch(Q_all, P_all, q_count, p_count)
        binding.gc_shard_fwd_dq(Q_all, P_all, pos_all, tau, q0, q_count, loss_part, row_lse, dQ,
                                ws=ws, dev_status=status, mask_mode=mask_mode)

    def dp(self, Q_all, P_all, pos_all, tau, mask_mode, row_lse, p0, p_count, q_count, dP):
        from . import binding
        ws, status = self._scratch(Q_all, P_all, q_count, p_count)
        binding.gc_shard_dp(Q_all, P_all, pos_all, tau, row_lse, p0, p_count, dP, ws=ws,
                            dev_status=status, mask_mode=mask_mode)


class ShardedStep:
    """One sharded Step 2 for a fixed problem size, reusable across calls.

    Rank r owns the r-th range of row_ranges(B, world) of the queries and of row_ranges(N, world)
    of the passages.  `run(Q_local [b x d], P_local [n x d], pos_local [b] int32)` (positives as
    row indices into the GATHERED passage matrix) returns (loss [1], row_lse_all [B], dQ_local
    [b x d], dP_local [n x d]); `loss` is the full-batch loss on every rank.  The returned tensors
    are this object's buffers and are overwritten by the next call.  `timings` holds the seconds
    the last call spent in collectives and in the two compute steps when `measure=True` (host
    clock around synchronised sections: a diagnostic, it serialises the step)."""

    def __init__(self, B, N, d, dtype, device, kernels=None, group=None, mask_mode=0):
        self.B, self.N, self.d, self.group = B, N, d, group
        self.mask_mode = mask_mode
        self.kernels = kernels or LibraryKernels()
        self.world, self.rank = _world(group)
        self.q_ranges, self.p_ranges = row_ranges(B, self.world), row_ranges(N, self.world)
        (self.q0, self.b), (self.p0, self.n) = self.q_ranges[self.rank], self.p_ranges[self.rank]
        qc, pc = [c for _, c in self.q_ranges], [c for _, c in self.p_ranges]
        self.gQ = _Gather(qc, (d,), dtype, device, group)
        self.gP = _Gather(pc, (d,), dtype, device, group)
        self.gpos = _Gather(qc, (), torch.int32, device, group)
        self.glse = _Gather(qc, (), torch.float32, device, group)
        f32 = dict(dtype=torch.float32, device=device)
        self.loss_part = torch.zeros(1, **f32)
        self.row_lse = torch.zeros(B, **f32)
        self.dQ = torch.empty(self.b, d, **f32)
        self.dP = torch.empty(self.n, d, **f32)
        self.timings = {}

    def _sync(self, device):
        if device.type == "cuda":
            torch.cuda.synchronize(device)

    def run(self, Q_local, P_local, pos_local, tau, measure=False):
        if Q_local.shape[0] != self.b or P_local.shape[0] != self.n or pos_local.shape[0] != self.b:
            raise ValueError("local shapes do not match this rank's ranges")
        dev = Q_local.device
        t = [0.0, 0.0, 0.0, 0.0]

        def section(i, fn):
            if not measure:
                return fn()
            self._sync(dev)
            t0 = time.perf_counter()
            out = fn()
            self._sync(dev)
            t[i] += time.perf_counter() - t0
            return out

        # the paper's one all-gather: all representations (and the relevance map) on every
        # rank; the three collectives are in flight together
        def exchange():
            w = [self.gQ.start(Q_local, self.rank), self.gP.start(P_local, self.rank),
                 self.gpos.start(pos_local, self.rank)]
            return self.gQ.finish(w[0]), self.gP.finish(w[1]), self.gpos.finish(w[2])
        Q_all, P_all, pos_all = section(0, exchange)
        self.loss_part.zero_()
        section(1, lambda: self.kernels.fwd_dq(Q_all, P_all, pos_all, tau, self.mask_mode, self.q0,
                                               self.b, self.n, self.loss_part, self.row_lse, self.dQ))
        # every rank needs lse_i of every query for its passages' gradients: B floats in total
        lse_all = section(2, lambda: self.glse.finish(
            self.glse.start(self.row_lse[self.q0:self.q0 + self.b], self.rank)))
        section(3, lambda: self.kernels.dp(Q_all, P_all, pos_all, tau, self.mask_mode, lse_all,
                                           self.p0, self.n, self.b, self.dP))

        def reduce_loss():
            if self.world > 1:
                dist.all_reduce(self.loss_part, op=dist.ReduceOp.SUM, group=self.group)
        section(2, reduce_loss)
        if measure:
            self.timings = {"gather_reps_s": t[0], "fwd_dq_s": t[1], "lse_and_loss_s": t[2],
                            "dp_s": t[3]}
        return self.loss_part, lse_all, self.dQ, self.dP


def sharded_build_cache(Q_local, P_local, pos_local, tau, B, N, kernels=None, group=None,
                        mask_mode=0):
    """One sharded Step 2 with freshly allocated buffers (convenience; loops use ShardedStep)."""
    step = ShardedStep(B, N, Q_local.shape[1], Q_local.dtype, Q_local.device, kernels, group,
                       mask_mode)
    return step.run(Q_local, P_local, pos_local, tau)
