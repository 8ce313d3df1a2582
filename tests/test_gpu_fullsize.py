"""Parity at the benchmark's full sizes, in the launch configuration bench.py times, on sampled outputs.

A gradient row depends only on the entries of its own row (column), so the oracle can recompute sampled
rows and columns one by one from the COO triples that fall in them: the sub-template keeps the sampled
rows (re-indexed) and ALL columns, and vice versa.  Samples: random rows / columns plus the most populated
ones (the rows that are split over many segments).
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _sampled_check(w, path, tol_g, n_random=48, n_hot=8, emulate=True):
    tpl = W.make_template(w, DEV, order="sorted")
    T = B.template_from_workload(tpl, path=path)
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    GP, GQ = torch.empty_like(P), torch.empty_like(Q)
    T.tsid_grad_step(P, Q, GP, GQ)
    T.tsid_check()
    got_path = T.tsid_get_info()[0]
    T.tsid_destroy()
    rng = np.random.default_rng(w.seed)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    worst = {}
    for side, idx_all, other, nrow, Xg, G, Xnew, norm in (
            ("rows", tpl.rows, tpl.cols, w.m, (P0, Q0), GP, P, w.norm_p),
            ("cols", tpl.cols, tpl.rows, w.n, (Q0, P0), GQ, Q, w.norm_q)):
        counts = torch.bincount(idx_all, minlength=nrow)
        hot = torch.topk(counts, n_hot).indices.cpu().numpy()
        sample = np.unique(np.concatenate([hot, rng.choice(nrow, n_random, replace=False)]))
        lut = torch.full((nrow,), -1, dtype=torch.int32, device=DEV)
        lut[torch.as_tensor(sample, device=DEV)] = torch.arange(len(sample), dtype=torch.int32, device=DEV)
        loc = lut[idx_all.long()]
        keep = loc >= 0
        sub_r = loc[keep].cpu().numpy(); sub_c = other[keep].cpu().numpy(); sub_v = tpl.vals[keep].cpu().numpy()
        Xs, Y = Xg[0][sample], Xg[1]
        # the sampled side plays the role of P (rows); only its half of the result is compared
        st = oracle.grad_step(len(sample), Y.shape[0], w.k, sub_r, sub_c, sub_v, Xs, Y, w.eta, w.lam, w.xi, w.clip,
                              norm, oracle.NORM_NONE, bf16_emulate=emulate)
        g = G[torch.as_tensor(sample, device=DEV).long()].cpu().numpy()
        x = Xnew[torch.as_tensor(sample, device=DEV).long()].cpu().numpy()
        worst[side] = (relerr(g, st.GP), relerr(x, st.P), int(counts.max()))
        assert worst[side][0] <= tol_g, (side, worst)
        assert worst[side][1] <= max(1e-4, tol_g / 10), (side, worst)
    return got_path, worst


def test_c5_full_size_sampled_rows_and_columns():
    path, worst = _sampled_check(W.C5, B.TSID_PATH_SPARSE, 1e-4)
    assert path == B.TSID_PATH_SPARSE
    assert worst["rows"][2] > 1024 and worst["cols"][2] > 1024     # split rows were among the samples


def test_c3_full_size_sampled_rows_and_columns():
    _sampled_check(W.C3, B.TSID_PATH_SPARSE, 1e-4)


def test_c4_full_size_dense_sampled_rows_and_columns():
    path, _ = _sampled_check(W.C4, B.TSID_PATH_AUTO, 1e-2)
    assert path == B.TSID_PATH_DENSE_TC


def test_c4_full_size_sparse_fp32_and_bf16():
    import dataclasses
    _sampled_check(dataclasses.replace(W.C4, precision="f32"), B.TSID_PATH_SPARSE, 1e-4, emulate=False)
    _sampled_check(W.C4, B.TSID_PATH_SPARSE, 1e-4)
