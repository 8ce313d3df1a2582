"""Mini-batch epochs (one full-batch step per batch of Omega, in order) against the oracle stepping through
the same batches: the paper-literal setting (entry-wise clip, Eq. 9's 1/n on the q side) and the default one."""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W
from paper_2608_00977_b200.minibatch import BatchedTemplate, MiniBatches, batch_ids, split_batches

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


@pytest.mark.parametrize("precision", ["f32", "bf16"])
@pytest.mark.parametrize("clip,norm_p,norm_q,eta", [(W.CLIP_ASYM_ENTRY, W.NORM_NONE, W.NORM_COUNT, 0.001),
                                                    (W.CLIP_ASYM_STEP, W.NORM_COUNT, W.NORM_COUNT, 0.02)])
def test_one_template_for_all_batches(clip, norm_p, norm_q, eta, precision):
    """tsid_template_create_batched / tsid_grad_step_batch: one layout over (batch, row, col), a contiguous range of work
    segments per batch.  Every step against the oracle's step on the batch's entries (teacher-forced), the epochs against
    the oracle stepping through the same batches, and bit for bit against one template per batch."""
    w = small_workload("mb1", 700, 500, 32, 40_000, positions="zipf", seed=43, values="ratings", noise_var=0.25,
                       precision=precision, eta=eta, lam=0.03, xi=0.1, clip=clip, norm_p=norm_p, norm_q=norm_q)
    tpl = W.make_template(w, DEV, order="shuffled")
    nb, epochs = 5, 2
    prec = B.TSID_BF16_SHADOW if precision == "bf16" else B.TSID_F32
    kw = dict(precision=prec, path=B.TSID_PATH_SPARSE, eta=w.eta, lam=w.lam, xi=w.xi, clip=clip, norm_p=norm_p, norm_q=norm_q)
    bt = BatchedTemplate(w.m, w.n, w.k, tpl.rows, tpl.cols, tpl.vals, nb, seed=9, **kw)
    mb = MiniBatches(w.m, w.n, w.k, tpl.rows, tpl.cols, tpl.vals, nb, seed=9, **kw)
    parts = split_batches(tpl.nnz, nb, 9, DEV)
    ids = batch_ids(tpl.nnz, nb, 9, DEV)
    assert all(bool((ids[idx] == b).all()) for b, idx in enumerate(parts))
    r, c, v = tpl.rows.cpu().numpy(), tpl.cols.cpu().numpy(), tpl.vals.cpu().numpy()
    emu = precision == "bf16"
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    P2, Q2 = tpl.P0.clone(), tpl.Q0.clone()
    Pr, Qr = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    GP, GQ = torch.empty_like(P), torch.empty_like(Q)
    for ep in range(epochs):
        for b, idx in enumerate(parts):
            i = idx.cpu().numpy()
            Pin, Qin = P.cpu().numpy(), Q.cpu().numpy()
            bt.T.tsid_grad_step_batch(b, P, Q, GP, GQ)
            bt.T.tsid_check()
            st = oracle.grad_step(w.m, w.n, w.k, r[i], c[i], v[i], Pin, Qin, w.eta, w.lam, w.xi, clip, norm_p, norm_q, bf16_emulate=emu)
            errs = [relerr(GP.cpu().numpy(), st.GP), relerr(GQ.cpu().numpy(), st.GQ), relerr(P.cpu().numpy(), st.P), relerr(Q.cpu().numpy(), st.Q)]
            assert max(errs) <= 1e-4, (ep, b, errs)
            mb.templates[b].tsid_grad_step(P2, Q2)
            assert torch.equal(P2, P) and torch.equal(Q2, Q)          # the same bits as a template of the batch alone
            st = oracle.grad_step(w.m, w.n, w.k, r[i], c[i], v[i], Pr, Qr, w.eta, w.lam, w.xi, clip, norm_p, norm_q, bf16_emulate=emu)
            Pr, Qr = st.P, st.Q
    assert relerr(P.cpu().numpy(), Pr) <= 5e-4 and relerr(Q.cpu().numpy(), Qr) <= 5e-4
    # the handle is for batch steps only; bad batch numbers are refused
    with pytest.raises(B.TsidError) as e:
        bt.T.tsid_grad_step(P, Q)
    assert e.value.status == B.TSID_ERR_UNSUPPORTED
    with pytest.raises(B.TsidError) as e:
        bt.T.tsid_grad_step_batch(nb, P, Q)
    assert e.value.status == B.TSID_ERR_INVALID_ARG
    bad = ids.clone(); bad[7] = nb
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(w.m, w.n, w.k, tpl.nnz, **kw), tpl.rows, tpl.cols, tpl.vals, batch=bad, n_batches=nb)
    assert e.value.status == B.TSID_ERR_INDEX_RANGE
    bt.destroy(); mb.destroy()
