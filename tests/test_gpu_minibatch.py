"""Mini-batch epochs (one full-batch step per batch of Omega, in order) against the oracle stepping through
the same batches: the paper-literal setting (entry-wise clip, Eq. 9's 1/n on the q side) and the default one."""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W
from paper_2608_00977_b200.minibatch import MiniBatches, split_batches

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("clip,norm_p,norm_q,eta", [(W.CLIP_ASYM_ENTRY, W.NORM_NONE, W.NORM_COUNT, 0.001),
                                                    (W.CLIP_ASYM_STEP, W.NORM_COUNT, W.NORM_COUNT, 0.02)])
def test_minibatch_epochs_against_the_oracle(clip, norm_p, norm_q, eta):
    # the p side of the literal setting is a plain sum over a row's entries: its step size has to be small
    w = small_workload("mb", 700, 500, 32, 40_000, positions="zipf", seed=41, values="ratings", noise_var=0.25,
                       eta=eta, lam=0.03, xi=0.1, clip=clip, norm_p=norm_p, norm_q=norm_q)
    tpl = W.make_template(w, DEV, order="shuffled")
    nb, epochs = 5, 3
    mb = MiniBatches(w.m, w.n, w.k, tpl.rows, tpl.cols, tpl.vals, nb, seed=9, precision=B.TSID_F32,
                     path=B.TSID_PATH_SPARSE, eta=w.eta, lam=w.lam, xi=w.xi, clip=clip, norm_p=norm_p, norm_q=norm_q)
    parts = split_batches(tpl.nnz, nb, 9, DEV)
    assert sorted(torch.cat(parts).tolist()) == list(range(tpl.nnz))           # a partition of Omega
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    sse = [mb.sse(P, Q)]
    for _ in range(epochs):
        mb.epoch(P, Q)
        sse.append(mb.sse(P, Q))
    r, c, v = tpl.rows.cpu().numpy(), tpl.cols.cpu().numpy(), tpl.vals.cpu().numpy()
    Pr, Qr = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    for _ in range(epochs):
        for idx in parts:
            i = idx.cpu().numpy()
            st = oracle.grad_step(w.m, w.n, w.k, r[i], c[i], v[i], Pr, Qr, w.eta, w.lam, w.xi, clip, norm_p, norm_q)
            Pr, Qr = st.P, st.Q
    assert relerr(P.cpu().numpy(), Pr) <= 5e-4 and relerr(Q.cpu().numpy(), Qr) <= 5e-4      # 15 steps of drift
    ref_sse, _ = oracle.loss(w.m, w.n, w.k, r, c, v, Pr, Qr, 0.0)
    assert abs(sse[-1] - ref_sse) / ref_sse <= 1e-3
    assert sse[-1] < sse[0]
    mb.destroy()
