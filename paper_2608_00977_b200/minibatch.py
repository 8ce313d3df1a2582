"""Mini-batch form of template recovery: plumbing around tsid_grad_step (argument marshalling only).

The paper runs its updates over mini-batches of observed entries (Sec. 5.1: entries are grouped, their
per-entry updates aggregated per factor row and divided by the number of contributors, Eq. 9).  With this
library that is the full-batch step restricted to a batch: Omega is split into `batches` disjoint parts and one
epoch is one step per part, in order, on the same P and Q.  The count a row's sum is divided by
(TSID_NORM_COUNT) is then the number of ITS entries in the batch, which is Eq. 9's n.  Two forms:
`BatchedTemplate` (ONE library template over all batches: one layout pass, one workspace,
tsid_grad_step_batch) and the older `MiniBatches` (one template per batch), kept as its cross-check.  The
benchmarked path is the full-batch step (batches = 1).
"""
from __future__ import annotations

import torch

from . import binding as B


def split_batches(nnz: int, batches: int, seed: int, device) -> list[torch.Tensor]:
    """Index sets of `batches` disjoint parts of range(nnz): a seeded permutation cut into equal runs."""
    if batches < 1:
        raise ValueError("batches must be >= 1")
    g = torch.Generator(device="cpu").manual_seed(seed)
    perm = torch.randperm(nnz, generator=g).to(device)
    return [perm[nnz * b // batches: nnz * (b + 1) // batches] for b in range(batches)]


class MiniBatches:
    """One library template per batch of the observed entries; epoch() steps through them in order."""

    def __init__(self, m, n, k, rows, cols, vals, batches, seed=0, **cfg_kw):
        self.parts = split_batches(int(rows.numel()), batches, seed, rows.device)
        self.templates = []
        for idx in self.parts:
            cfg = B.make_config(m, n, k, int(idx.numel()), **cfg_kw)
            self.templates.append(B.Template(cfg, rows[idx].contiguous(), cols[idx].contiguous(), vals[idx].contiguous()))

    def epoch(self, P, Q):
        for T in self.templates:
            T.tsid_grad_step(P, Q)

    def sse(self, P, Q) -> float:
        return sum(T.tsid_loss(P, Q)[0] for T in self.templates)

    def destroy(self):
        for T in self.templates:
            T.tsid_destroy()


def batch_ids(nnz: int, batches: int, seed: int, device) -> torch.Tensor:
    """int32[nnz]: the batch of every entry, the same partition as split_batches gives."""
    ids = torch.empty(nnz, dtype=torch.int32, device=device)
    for b, idx in enumerate(split_batches(nnz, batches, seed, device)):
        ids[idx] = b
    return ids


class BatchedTemplate:
    """All batches in one library template (tsid_template_create_batched); epoch() steps through them in order."""

    def __init__(self, m, n, k, rows, cols, vals, batches, seed=0, **cfg_kw):
        self.batches = batches
        ids = batch_ids(int(rows.numel()), batches, seed, rows.device)
        cfg = B.make_config(m, n, k, int(rows.numel()), **cfg_kw)
        self.T = B.Template(cfg, rows, cols, vals, batch=ids, n_batches=batches)

    def epoch(self, P, Q):
        for b in range(self.batches):
            self.T.tsid_grad_step_batch(b, P, Q)

    def destroy(self):
        self.T.tsid_destroy()
