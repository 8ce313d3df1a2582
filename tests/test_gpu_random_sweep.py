"""Seeded random sweep of the sparse step against the oracle: shapes from 1 x 1 to thousands (tile edges +- 1),
every k the kernels are instantiated for and ragged ones, empty to fully observed, one heavy row and column,
both input orders, every clip / normalisation mode and every create flag."""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr
from paper_2608_00977_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(rng):
    prec = int(rng.integers(0, 2))
    k = int(rng.choice([4, 8, 12, 16, 20, 24, 32, 40, 48, 64, 72, 96, 128, 136, 200, 256]))
    if prec == 1 and k % 8:
        k = (k // 8 + 1) * 8
    m = int(rng.choice([1, 2, 3, 7, 33, 100, 257, 1000, 3000]))
    n = int(rng.choice([1, 2, 5, 31, 64, 129, 500, 2500]))
    dens = float(rng.choice([0.0, 0.001, 0.01, 0.05, 0.3, 0.9, 1.0]))
    cells = m * n
    nnz = cells if dens >= 1.0 else min(cells, int(round(dens * cells)) + int(rng.integers(0, 5)))
    ids = rng.choice(cells, nnz, replace=False) if nnz else np.zeros(0, dtype=np.int64)
    if nnz and rng.random() < 0.3 and m > 3 and n > 3:          # one full row and one full column
        hr, hc = int(rng.integers(0, m)), int(rng.integers(0, n))
        ids = rng.permutation(np.unique(np.concatenate([hr * n + np.arange(n), np.arange(m) * n + hc, ids])))
    order_sorted = rng.random() < 0.5
    if order_sorted:
        ids = np.sort(ids)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    ratings = rng.random() < 0.5
    vals = rng.integers(1, 6, len(ids)).astype(np.float32) if ratings else rng.standard_normal(len(ids)).astype(np.float32)
    clip, norm_p, norm_q = int(rng.integers(0, 4)), int(rng.integers(0, 2)), int(rng.integers(0, 2))
    if clip == B.TSID_CLIP_ASYM_ENTRY and prec == 0 and k > 128:
        clip = B.TSID_CLIP_ASYM_STEP                            # outside the entry-wise mode's limits
    flags = (B.TSID_VALIDATE if rng.random() < 0.5 else 0) | \
            (B.TSID_INPUT_ROW_SORTED if order_sorted and rng.random() < 0.5 else 0) | \
            (B.TSID_VALUES_U8 if ratings and rng.random() < 0.5 else 0)
    hyper = (float(rng.choice([0.01, 0.05])), float(rng.choice([0.0, 0.03])), float(rng.choice([0.05, 0.1, 2.0])))
    return m, n, k, rows, cols, vals, prec, clip, norm_p, norm_q, flags, hyper


def test_random_sweep_of_the_sparse_step():
    rng = np.random.default_rng(777)
    worst = 0.0
    for it in range(250):
        m, n, k, rows, cols, vals, prec, clip, norm_p, norm_q, flags, (eta, lam, xi) = _case(rng)
        P0 = (rng.standard_normal((m, k)) * k ** -0.25).astype(np.float32)
        Q0 = (rng.standard_normal((n, k)) * k ** -0.25).astype(np.float32)
        cfg = B.make_config(m, n, k, len(rows), prec, B.TSID_PATH_SPARSE, eta, lam, xi, clip, norm_p, norm_q, flags)
        T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
        P, Q = torch.tensor(P0, device=DEV), torch.tensor(Q0, device=DEV)
        GP, GQ = torch.full_like(P, 9.0), torch.full_like(Q, 9.0)
        sse, _ = T.tsid_loss(P, Q)
        T.tsid_grad_step(P, Q, GP, GQ)
        T.tsid_check()
        T.tsid_destroy()
        ref = oracle.grad_step(m, n, k, rows, cols, vals, P0, Q0, eta, lam, xi, clip, norm_p, norm_q, bf16_emulate=bool(prec))
        ref_sse, _ = oracle.loss(m, n, k, rows, cols, vals, P0, Q0, lam, bf16_emulate=bool(prec))
        errs = [relerr(GP.cpu().numpy(), ref.GP), relerr(GQ.cpu().numpy(), ref.GQ), relerr(P.cpu().numpy(), ref.P),
                relerr(Q.cpu().numpy(), ref.Q), abs(sse - ref_sse) / ref_sse if ref_sse > 0 else abs(sse)]
        worst = max(worst, max(errs))
        assert max(errs) <= 1e-4, (it, m, n, k, len(rows), prec, clip, norm_p, norm_q, flags, errs)
    assert worst <= 1e-4
