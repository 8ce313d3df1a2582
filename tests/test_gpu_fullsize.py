"""Parity at the benchmark's full sizes, in the launch configuration bench.py times, on sampled outputs.

A gradient row depends only on the entries of its own row (column), so the oracle can recompute sampled
rows and columns one by one from the COO triples that fall in them: the sub-template keeps the sampled
rows (re-indexed) and ALL columns, and vice versa.  Samples: 4096 random rows / columns plus the 16 most
populated ones (the rows that are split over many segments and, on the hybrid path, over many tile chunks).
Two global checks ride along: the trace identity sum <G_P, P> = sum <G_Q, Q> (both equal sum_Omega e_ij p_i.q_j)
over the whole outputs, and the sum of squared residuals of the sampled rows (tsid_residuals at their CSR
positions, added in fp64) against the oracle's loss on the same sub-template.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr, rowwise_relerr
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _sampled_check(w, path, tol_g, n_random=4096, n_hot=16, emulate=True, tol_trace=1e-5, tol_row=None):
    tpl = W.make_template(w, DEV, order="sorted")
    T = B.template_from_workload(tpl, path=path)
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    GP, GQ = torch.empty_like(P), torch.empty_like(Q)
    T.tsid_grad_step(P, Q, GP, GQ)
    T.tsid_check()
    got_path = T.tsid_get_info()[0]
    # run to run: the sums of a second evaluation at the same factors have the same bits
    GP2, GQ2 = torch.empty_like(P), torch.empty_like(Q)
    T.tsid_grad(tpl.P0, tpl.Q0, GP2, GQ2)
    assert torch.equal(GP2, GP) and torch.equal(GQ2, GQ)
    del GP2, GQ2
    # global: the trace identity, with the factor values the passes read
    bf = w.precision == "bf16"
    Pr = tpl.P0.bfloat16().double() if bf else tpl.P0.double()
    Qr = tpl.Q0.bfloat16().double() if bf else tpl.Q0.double()
    tr_p = float((GP.double() * Pr).sum()); tr_q = float((GQ.double() * Qr).sum())
    del Pr, Qr
    assert abs(tr_p - tr_q) <= tol_trace * max(abs(tr_p), abs(tr_q)), (tr_p, tr_q)
    e_csr = T.tsid_residuals(tpl.P0, tpl.Q0)
    row_ptr, _, _, col_ptr, _, _, perm = T.tsid_get_layout(copy=False)
    rng = np.random.default_rng(w.seed)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    worst = {}
    for side, idx_all, other, nrow, Xg, G, Xnew, norm, ptr in (
            ("rows", tpl.rows, tpl.cols, w.m, (P0, Q0), GP, P, w.norm_p, row_ptr),
            ("cols", tpl.cols, tpl.rows, w.n, (Q0, P0), GQ, Q, w.norm_q, col_ptr)):
        counts = torch.bincount(idx_all, minlength=nrow)
        hot = torch.topk(counts, min(n_hot, nrow)).indices.cpu().numpy()
        sample = np.unique(np.concatenate([hot, rng.choice(nrow, min(n_random, nrow), replace=False)]))
        sample_t = torch.as_tensor(sample, device=DEV).long()
        lut = torch.full((nrow,), -1, dtype=torch.int32, device=DEV)
        lut[sample_t] = torch.arange(len(sample), dtype=torch.int32, device=DEV)
        loc = lut[idx_all.long()]
        keep = loc >= 0
        sub_r = loc[keep].cpu().numpy(); sub_c = other[keep].cpu().numpy(); sub_v = tpl.vals[keep].cpu().numpy()
        del loc, keep, lut
        Xs, Y = Xg[0][sample], Xg[1]
        # the sampled side plays the role of P (rows); only its half of the result is compared
        st = oracle.grad_step(len(sample), Y.shape[0], w.k, sub_r, sub_c, sub_v, Xs, Y, w.eta, w.lam, w.xi, w.clip,
                              norm, oracle.NORM_NONE, bf16_emulate=emulate)
        g = G[sample_t].cpu().numpy()
        x = Xnew[sample_t].cpu().numpy()
        cnt = counts[sample_t].cpu().numpy()
        worst[side] = (relerr(g, st.GP), relerr(x, st.P), int(counts.max()), rowwise_relerr(g, st.GP, cnt))
        assert worst[side][0] <= tol_g, (side, worst)
        assert worst[side][1] <= max(1e-4, tol_g / 10), (side, worst)
        assert worst[side][3] <= (tol_row if tol_row is not None else tol_g), (side, worst)
        # global: squared residuals of the sampled rows (columns) at their positions in the CSR order
        lo, hi = ptr[sample_t], ptr[sample_t + 1]
        seg = torch.repeat_interleave(torch.arange(len(sample), device=DEV), (hi - lo))
        pos = torch.arange(int((hi - lo).sum()), device=DEV) - torch.repeat_interleave(torch.cumsum(hi - lo, 0) - (hi - lo), (hi - lo)) + lo[seg]
        if side == "cols":
            pos = perm[pos].long() & 0xFFFFFFFF
        sse_gpu = float((e_csr[pos].double() ** 2).sum())
        sse_ref, _ = oracle.loss(len(sample), Y.shape[0], w.k, sub_r, sub_c, sub_v, Xs, Y, 0.0, bf16_emulate=emulate)
        assert len(sub_r) == pos.numel() and abs(sse_gpu - sse_ref) <= 1e-5 * sse_ref, (side, sse_gpu, sse_ref)
        del seg, pos
    # one epoch of tsid_fit from the same factors ends on the same bits as the tsid_grad_step above (on the hybrid
    # path the fit leaves the tile passes' sums to the update kernel)
    del GP, GQ, e_csr
    P2, Q2 = tpl.P0.clone(), tpl.Q0.clone()
    T.tsid_fit(P2, Q2, 1)
    T.tsid_check()
    assert torch.equal(P2, P) and torch.equal(Q2, Q)
    T.tsid_destroy()
    return got_path, worst


def test_c5_full_size_sampled_rows_and_columns():
    path, worst = _sampled_check(W.C5, B.TSID_PATH_SPARSE, 1e-4)
    assert path == B.TSID_PATH_SPARSE
    assert worst["rows"][2] > 1024 and worst["cols"][2] > 1024     # split rows were among the samples


def test_c5_full_size_hybrid_path_as_benchmarked():
    # what TSID_PATH_AUTO runs on the 1e9-entry template: dense tiles on the tensor cores (E rounded to bf16
    # there: the tensor-core bar), the remaining entries on the gather-reduce passes
    # (measured: G 8e-5, per-row 2e-3, factors 4e-5; the bars below leave a factor of five)
    path, worst = _sampled_check(W.C5, B.TSID_PATH_AUTO, 1e-3, n_hot=8, tol_trace=1e-4, tol_row=1e-2)
    assert path == B.TSID_PATH_HYBRID


def test_c3_full_size_sampled_rows_and_columns():
    _sampled_check(W.C3, B.TSID_PATH_SPARSE, 1e-4)
    path, _ = _sampled_check(W.C3, B.TSID_PATH_AUTO, 1e-3, tol_trace=1e-4, tol_row=1e-2)
    assert path == B.TSID_PATH_HYBRID


def test_c4_full_size_dense_sampled_rows_and_columns():
    path, _ = _sampled_check(W.C4, B.TSID_PATH_AUTO, 1e-2, n_random=512, tol_trace=1e-4, tol_row=1e-1)
    assert path == B.TSID_PATH_DENSE_TC


def test_c4_full_size_sparse_fp32_and_bf16():
    import dataclasses
    _sampled_check(dataclasses.replace(W.C4, precision="f32"), B.TSID_PATH_SPARSE, 1e-4, n_random=512, emulate=False)
    _sampled_check(W.C4, B.TSID_PATH_SPARSE, 1e-4, n_random=512)
