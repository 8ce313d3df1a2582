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


def _hybrid_case(rng):
    k = int(rng.choice([64, 128]))
    m = int(rng.choice([1, 5, 127, 128, 129, 300, 640, 1000, 2500]))
    n = int(rng.choice([1, 7, 100, 128, 200, 257, 900, 2048]))
    hot_r = int(min(m, rng.choice([1, 40, 128, 200, 400])))
    hot_c = int(min(n, rng.choice([1, 30, 128, 260, 500])))
    dens_hot = float(rng.choice([0.05, 0.3, 0.9, 1.0]))
    dens_bg = float(rng.choice([0.0, 0.002, 0.02, 0.2]))
    hr = rng.choice(m, hot_r, replace=False); hc = rng.choice(n, hot_c, replace=False)
    mask = rng.random((m, n)) < dens_bg
    mask[np.ix_(hr, hc)] |= rng.random((hot_r, hot_c)) < dens_hot
    rows, cols = np.nonzero(mask)
    if rng.random() < 0.5:
        p = rng.permutation(len(rows)); rows, cols = rows[p], cols[p]
    vals = rng.integers(-8, 9, len(rows)).astype(np.float32)
    clip, norm_p, norm_q = int(rng.integers(0, 3)), int(rng.integers(0, 2)), int(rng.integers(0, 2))
    return m, n, k, rows.astype(np.int32), cols.astype(np.int32), vals, clip, norm_p, norm_q


def test_random_sweep_of_the_hybrid_step():
    """The hybrid path on random shapes (below, at and above the tile edge; one ragged block to many), random hot
    blocks over thin or thick backgrounds, both input orders, integer data: the sums must equal the oracle's bit for
    bit whether a template ends up with tiles and a tail, tiles only, or on the sparse path after all."""
    rng = np.random.default_rng(4242)
    ran = with_tiles = tiles_only = 0
    for it in range(120):
        m, n, k, rows, cols, vals, clip, norm_p, norm_q = _hybrid_case(rng)
        nnz = len(rows)
        if nnz < max(m, n, ((m + 127) // 128) * ((n + 127) // 128), 1):
            with pytest.raises(B.TsidError) as e:      # outside the hybrid path's limits: refused up front
                B.tsid_workspace_bytes(B.make_config(m, n, k, nnz, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID))
            assert e.value.status == B.TSID_ERR_UNSUPPORTED
            continue
        P0 = rng.integers(-2, 3, (m, k)).astype(np.float32); Q0 = rng.integers(-2, 3, (n, k)).astype(np.float32)
        eta, lam, xi = 2.0 ** -10, float(rng.choice([0.0, 0.25])), float(rng.choice([0.5, 64.0]))
        cfg = B.make_config(m, n, k, nnz, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID, eta, lam, xi, clip, norm_p, norm_q, 0)
        T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
        path = T.tsid_get_info()[0]
        tiles, _, tail = T.tsid_get_hybrid_info()
        assert (path == B.TSID_PATH_HYBRID) == (tiles > 0) and 0 <= tail <= nnz
        with_tiles += tiles > 0; tiles_only += tiles > 0 and tail == 0; ran += 1
        P, Q = torch.tensor(P0, device=DEV), torch.tensor(Q0, device=DEV)
        GP, GQ = torch.full_like(P, 9.0), torch.full_like(Q, 9.0)
        T.tsid_grad_step(P, Q, GP, GQ)
        T.tsid_check()
        T.tsid_destroy()
        ref = oracle.grad_step(m, n, k, rows, cols, vals, P0, Q0, eta, lam, xi, clip, norm_p, norm_q)
        assert np.abs(ref.GP).max(initial=0) < 2 ** 22 and np.abs(ref.GQ).max(initial=0) < 2 ** 22
        assert np.array_equal(GP.cpu().numpy().astype(np.float64), ref.GP), (it, m, n, k, nnz, tiles, tail)
        assert np.array_equal(GQ.cpu().numpy().astype(np.float64), ref.GQ), (it, m, n, k, nnz, tiles, tail)
        assert relerr(P.cpu().numpy(), ref.P) <= 1e-6 and relerr(Q.cpu().numpy(), ref.Q) <= 1e-6, (it, m, n, k, clip, norm_p, norm_q)
    assert ran >= 50 and with_tiles >= 40 and tiles_only >= 3, (ran, with_tiles, tiles_only)
