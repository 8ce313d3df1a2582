"""Row-sharded template recovery: plumbing around tsid_grad / tsid_apply (argument marshalling and the
one exchange step only; every arithmetic step of the path runs in the library's kernels).

The full-batch step splits exactly over a partition of the rows of Omega: rank r owns the rows
[r0, r1) of R and of P and a replica of Q.  Its G_P rows are complete; the G_Q of the ranks add up, and so
do the column counts |Omega^j| that TSID_NORM_COUNT divides by.  Per step: tsid_grad, one all-reduce (sum)
of G_Q (n x k fp32), tsid_apply.  Every rank applies the same update to its Q replica, so the replicas
stay bitwise equal.  The paper keeps template recovery on one GPU (Sec. 7 lists multi-GPU recovery as
future work); this module is that extension, not something the paper specifies.
"""
from __future__ import annotations

import torch

from . import binding as B


def row_block(m: int, rank: int, world: int) -> tuple[int, int]:
    """Rows [r0, r1) of rank `rank`: contiguous blocks whose sizes differ by at most one."""
    if not (world >= 1 and 0 <= rank < world):
        raise ValueError("need 0 <= rank < world")
    return m * rank // world, m * (rank + 1) // world


def shard_coo(rows: torch.Tensor, cols: torch.Tensor, vals: torch.Tensor, r0: int, r1: int):
    """The entries with r0 <= row < r1, rows renumbered from 0 (order kept)."""
    keep = (rows >= r0) & (rows < r1)
    return (rows[keep] - r0).to(torch.int32).contiguous(), cols[keep].contiguous(), vals[keep].contiguous()


def all_reduce_sum(t: torch.Tensor, dist=None, group=None) -> torch.Tensor:
    """Sum of `t` over the ranks, in place (identity without a process group)."""
    if dist is not None and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def symmetric_buffers(numel: int, device, dist, group=None):
    """A float32 buffer of `numel` elements on every rank of `group`, each mapped into all the others
    (torch's symmetric memory).  Returns (tensor, [device address on rank 0, rank 1, ...], barrier()).
    Needs one process per GPU with peer access; this build had one GPU per call, so this helper has not run
    on more than one GPU: the single-GPU tests pass the addresses of ordinary tensors instead."""
    import torch.distributed._symmetric_memory as symm_mem
    t = symm_mem.empty(numel, dtype=torch.float32, device=device)
    hdl = symm_mem.rendezvous(t, group if group is not None else dist.group.WORLD)
    return t, [int(p) for p in hdl.buffer_ptrs], hdl.barrier


class RowShard:
    """One rank's part of a row-sharded template: a library template over its rows, the gradient buffers
    and the exchange.  `rows`, `cols`, `vals` are this rank's entries with LOCAL row numbers."""

    def __init__(self, m_local: int, n: int, k: int, rows, cols, vals, *, precision=B.TSID_F32,
                 path=B.TSID_PATH_SPARSE, eta=0.01, lam=0.0, xi=0.1, clip=B.TSID_CLIP_NONE,
                 norm_p=B.TSID_NORM_NONE, norm_q=B.TSID_NORM_NONE, flags=0, dist=None, group=None):
        cfg = B.make_config(m_local, n, k, int(rows.numel()), precision, path, eta, lam, xi, clip, norm_p, norm_q, flags)
        self.T = B.Template(cfg, rows, cols, vals)
        self.dist, self.group = dist, group
        dev = rows.device
        self.GP = torch.empty(m_local * k, dtype=torch.float32, device=dev)
        self.GQ = torch.empty(n * k, dtype=torch.float32, device=dev)
        # the counts a column's normalisation divides by are those of the whole matrix
        _, cq = self.T.tsid_get_counts()
        self.col_counts = cq
        self.set_global_col_counts(all_reduce_sum(cq.clone(), dist, group))

    def set_global_col_counts(self, cq_global: torch.Tensor):
        self.T.tsid_set_norm_counts(None, cq_global)

    def grad(self, P_local, Q):
        self.T.tsid_grad(P_local, Q, self.GP, self.GQ)
        return self.GP, self.GQ

    def apply(self, P_local, Q):
        self.T.tsid_apply(P_local, Q, self.GP, self.GQ)

    def step(self, P_local, Q):
        """One full-batch step of the sharded template: local sums, sum-exchange of G_Q, local update."""
        self.grad(P_local, Q)
        all_reduce_sum(self.GQ, self.dist, self.group)
        self.apply(P_local, Q)

    def apply_sliced(self, P_local, q_ptrs, gq_ptrs, rank):
        """The exchange folded into the update kernel: this rank adds the partial G_Q of all ranks for its
        slice of Q's rows (plain loads through the given device addresses), updates the slice once and
        stores it into every replica; P is updated from the local sums.  The caller synchronises the ranks
        before (all tsid_grad done) and after (all slices stored)."""
        self.T.tsid_apply_sliced(P_local, self.GP, q_ptrs, gq_ptrs, rank)

    def sse(self, P_local, Q) -> float:
        """Sum of squared residuals over ALL ranks' entries."""
        s, _ = self.T.tsid_loss(P_local, Q)
        t = torch.tensor([s], dtype=torch.float64, device=P_local.device)
        return float(all_reduce_sum(t, self.dist, self.group)[0])

    def destroy(self):
        self.T.tsid_destroy()
