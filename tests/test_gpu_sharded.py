"""Row-sharded template recovery (tsid_grad, one sum of G_Q, tsid_apply) against the oracle's full-batch
steps.  One GPU is enough: the shards of a template run one after the other and their G_Q buffers are
summed here, which is all an all-reduce does."""
import numpy as np
import pytest
import torch

import oracle
from helpers import F32_TOL, np_coo, relerr, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import sharded as S
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = {
    "plain": dict(precision="f32", eta=0.01, lam=0.0, clip=W.CLIP_NONE, norm_p=W.NORM_NONE, norm_q=W.NORM_NONE),
    "clip-count": dict(precision="f32", eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT,
                       norm_q=W.NORM_COUNT),
    "paper-literal": dict(precision="f32", eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_ENTRY, norm_p=W.NORM_NONE,
                          norm_q=W.NORM_COUNT),
    "bf16": dict(precision="bf16", eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT,
                 norm_q=W.NORM_COUNT),
}


@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("world", [2, 3])
def test_sharded_steps_match_the_full_batch_oracle(case, world):
    kw = CASES[case]
    m, n, k, nnz, steps = 1501, 700, 32, 120_000, 3
    w = small_workload("shard-" + case, m, n, k, nnz, positions="zipf", seed=11 + world, **kw)
    tpl = W.make_template(w, DEV, order="shuffled")
    prec = B.TSID_BF16_SHADOW if w.precision == "bf16" else B.TSID_F32
    shards, Ps, Qs = [], [], []
    for r in range(world):
        r0, r1 = S.row_block(m, r, world)
        rows, cols, vals = S.shard_coo(tpl.rows, tpl.cols, tpl.vals, r0, r1)
        shards.append(S.RowShard(r1 - r0, n, k, rows, cols, vals, precision=prec, eta=w.eta, lam=w.lam, xi=w.xi,
                                 clip=w.clip, norm_p=w.norm_p, norm_q=w.norm_q))
        Ps.append(tpl.P0[r0:r1].clone().contiguous())
        Qs.append(tpl.Q0.clone())
    # the exchange of the column counts, then of G_Q in every step
    cq = sum(s.col_counts.clone() for s in shards)
    assert int(cq.sum()) == tpl.nnz
    for s in shards:
        s.set_global_col_counts(cq)
    for _ in range(steps):
        for s, P, Q in zip(shards, Ps, Qs):
            s.grad(P.view(-1), Q.view(-1))
        total = shards[0].GQ.clone()
        for s in shards[1:]:
            total += s.GQ
        for s, P, Q in zip(shards, Ps, Qs):
            s.GQ.copy_(total)
            s.apply(P.view(-1), Q.view(-1))
            s.T.tsid_check()
    for Q in Qs[1:]:
        assert torch.equal(Q, Qs[0])                      # the replicas never drift apart
    rows, cols, vals = np_coo(tpl)
    bf = w.precision == "bf16"
    Pr, Qr, _ = oracle.fit(m, n, k, rows, cols, vals, tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(), steps, w.eta, w.lam,
                           w.xi, w.clip, w.norm_p, w.norm_q, bf16_emulate=bf, history=False)
    tol = 2e-3 if bf else F32_TOL      # bf16: the shadows of later steps round slightly different fp32 values
    assert relerr(torch.cat(Ps).cpu().numpy(), Pr) <= tol
    assert relerr(Qs[0].cpu().numpy(), Qr) <= tol
    # the global SSE is the sum of the shards' SSEs
    sse = sum(s.T.tsid_loss(P.view(-1), Q.view(-1))[0] for s, P, Q in zip(shards, Ps, Qs))
    ref_sse, _ = oracle.loss(m, n, k, rows, cols, vals, Pr, Qr, w.lam, bf16_emulate=bf)
    assert abs(sse - ref_sse) <= (2e-2 if bf else 1e-4) * ref_sse
    for s in shards:
        s.destroy()


def test_one_shard_equals_grad_step_bitwise():
    w = small_workload("shard-one", 900, 400, 16, 40_000, seed=5, eta=0.05, lam=0.03, clip=W.CLIP_ASYM_STEP,
                       norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV)
    s = S.RowShard(w.m, w.n, w.k, tpl.rows, tpl.cols, tpl.vals, eta=w.eta, lam=w.lam, xi=w.xi, clip=w.clip,
                   norm_p=w.norm_p, norm_q=w.norm_q)
    T = B.template_from_workload(tpl, path=B.TSID_PATH_SPARSE)
    Pa, Qa, Pb, Qb = tpl.P0.clone(), tpl.Q0.clone(), tpl.P0.clone(), tpl.Q0.clone()
    for _ in range(3):
        s.step(Pa.view(-1), Qa.view(-1))
        T.tsid_grad_step(Pb.view(-1), Qb.view(-1))
    assert torch.equal(Pa, Pb) and torch.equal(Qa, Qb)
    s.destroy(); T.tsid_destroy()


def test_split_step_argument_errors_and_counts():
    w = small_workload("shard-args", 300, 200, 8, 5_000, seed=9, norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV)
    T = B.template_from_workload(tpl, path=B.TSID_PATH_SPARSE)
    L = B.lib()
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    GP, GQ = torch.empty_like(P), torch.empty_like(Q)
    # null or misaligned gradient buffers are refused before any launch
    assert L.tsid_grad(T.h, P.data_ptr(), Q.data_ptr(), None, GQ.data_ptr()) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_apply(T.h, P.data_ptr(), Q.data_ptr(), GP.data_ptr() + 4, GQ.data_ptr()) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_grad(None, P.data_ptr(), Q.data_ptr(), GP.data_ptr(), GQ.data_ptr()) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_get_counts(None, None, None) == B.TSID_ERR_INVALID_ARG
    # counts are the row and column degrees of the template
    cp, cq = T.tsid_get_counts()
    rows, cols, _ = np_coo(tpl)
    assert np.array_equal(cp.cpu().numpy(), np.bincount(rows, minlength=w.m))
    assert np.array_equal(cq.cpu().numpy(), np.bincount(cols, minlength=w.n))
    # grad + apply with the template's own counts is tsid_grad_step
    T.tsid_set_norm_counts(cp, cq)
    Pa, Qa = tpl.P0.clone(), tpl.Q0.clone()
    T.tsid_grad(Pa, Qa, GP, GQ)
    T.tsid_apply(Pa, Qa, GP, GQ)
    T.tsid_grad_step(P, Q)
    assert torch.equal(Pa, P) and torch.equal(Qa, Q)
    # doubled column counts halve the normalised part of the column direction
    T.tsid_set_norm_counts(None, cq * 2)
    Pb, Qb = tpl.P0.clone(), tpl.Q0.clone()
    T.tsid_grad(Pb, Qb, GP, GQ)
    T.tsid_apply(Pb, Qb, GP, GQ)
    ref = oracle.grad_step(w.m, w.n, w.k, rows, cols, np_coo(tpl)[2], tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(),
                           w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
    s2 = np.where(2 * np.bincount(cols, minlength=w.n) > 1, 2 * np.bincount(cols, minlength=w.n), 1)[:, None]
    Qexp = tpl.Q0.cpu().numpy().astype(np.float64) + w.eta * (2.0 * ref.GQ / s2 - 2.0 * w.lam * tpl.Q0.cpu().numpy())
    assert relerr(Qb.cpu().numpy(), Qexp) <= F32_TOL
    assert torch.equal(Pb, P)
    T.tsid_destroy()


def test_sharded_dense_path():
    """Row shards that run the tcgen05 variant: the split step and the sum of G_Q work the same way."""
    m, n, k, world = 512, 384, 64, 2
    w = W.Workload("shard-dense", m, n, k, int(0.3 * m * n), "bernoulli", density=0.30, seed=21, values="lowrank",
                   noise_var=1e-4, precision="bf16", eta=0.2, lam=0.0, clip=W.CLIP_NONE, norm_p=W.NORM_COUNT,
                   norm_q=W.NORM_COUNT, epochs=3)
    tpl = W.make_template(w, DEV, order="shuffled")
    shards, Ps, Qs = [], [], []
    for r in range(world):
        r0, r1 = S.row_block(m, r, world)
        rows, cols, vals = S.shard_coo(tpl.rows, tpl.cols, tpl.vals, r0, r1)
        shards.append(S.RowShard(r1 - r0, n, k, rows, cols, vals, precision=B.TSID_BF16_SHADOW, path=B.TSID_PATH_DENSE_TC,
                                 eta=w.eta, lam=w.lam, xi=w.xi, clip=w.clip, norm_p=w.norm_p, norm_q=w.norm_q))
        assert shards[-1].T.tsid_get_info()[0] == B.TSID_PATH_DENSE_TC
        Ps.append(tpl.P0[r0:r1].clone().contiguous())
        Qs.append(tpl.Q0.clone())
    cq = sum(s.col_counts.clone() for s in shards)
    for s in shards:
        s.set_global_col_counts(cq)
    for s, P, Q in zip(shards, Ps, Qs):
        s.grad(P, Q)
    total = shards[0].GQ + shards[1].GQ
    for s, P, Q in zip(shards, Ps, Qs):
        s.GQ.copy_(total)
        s.apply(P, Q)
        s.T.tsid_check()
    assert torch.equal(Qs[0], Qs[1])
    rows, cols, vals = np_coo(tpl)
    ref = oracle.grad_step(m, n, k, rows, cols, vals, tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(), w.eta, w.lam, w.xi,
                           w.clip, w.norm_p, w.norm_q, bf16_emulate=True)
    assert relerr(total.view(n, k).cpu().numpy(), ref.GQ) <= 1e-2      # the dense path rounds E to bf16
    assert relerr(torch.cat(Ps).cpu().numpy(), ref.P) <= 1e-3 and relerr(Qs[0].cpu().numpy(), ref.Q) <= 1e-3
    for s in shards:
        s.destroy()


@pytest.mark.parametrize("case", ["clip-count", "paper-literal", "bf16"])
@pytest.mark.parametrize("world", [2, 3])
def test_update_with_the_exchange_folded_in(case, world):
    """tsid_apply_sliced: every emulated rank reduces and updates its slice of Q and stores it into all
    replicas.  With all replicas and parts on one GPU the 'peer' addresses are ordinary device addresses."""
    kw = CASES[case]
    m, n, k, nnz, steps = 1203, 650, 32, 90_000, 3
    w = small_workload("fused-" + case, m, n, k, nnz, positions="zipf", seed=31 + world, **kw)
    tpl = W.make_template(w, DEV, order="shuffled")
    prec = B.TSID_BF16_SHADOW if w.precision == "bf16" else B.TSID_F32
    shards, Ps, Qs = [], [], []
    for r in range(world):
        r0, r1 = S.row_block(m, r, world)
        rows, cols, vals = S.shard_coo(tpl.rows, tpl.cols, tpl.vals, r0, r1)
        shards.append(S.RowShard(r1 - r0, n, k, rows, cols, vals, precision=prec, eta=w.eta, lam=w.lam, xi=w.xi,
                                 clip=w.clip, norm_p=w.norm_p, norm_q=w.norm_q))
        Ps.append(tpl.P0[r0:r1].clone().contiguous())
        Qs.append(tpl.Q0.clone())
    cq = sum(s.col_counts.clone() for s in shards)
    for s in shards:
        s.set_global_col_counts(cq)
    q_ptrs = [Q.data_ptr() for Q in Qs]
    gq_ptrs = [s.GQ.data_ptr() for s in shards]
    for _ in range(steps):
        for s, P, Q in zip(shards, Ps, Qs):
            s.grad(P, Q)
        torch.cuda.synchronize()                       # "all parts complete"
        for r, (s, P) in enumerate(zip(shards, Ps)):
            s.apply_sliced(P, q_ptrs, gq_ptrs, r)
        torch.cuda.synchronize()                       # "all slices stored"
        for s in shards:
            s.T.tsid_check()
    for Q in Qs[1:]:
        assert torch.equal(Q, Qs[0])
    rows, cols, vals = np_coo(tpl)
    bf = w.precision == "bf16"
    Pr, Qr, _ = oracle.fit(m, n, k, rows, cols, vals, tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(), steps, w.eta, w.lam,
                           w.xi, w.clip, w.norm_p, w.norm_q, bf16_emulate=bf, history=False)
    tol = 2e-3 if bf else F32_TOL
    assert relerr(torch.cat(Ps).cpu().numpy(), Pr) <= tol and relerr(Qs[0].cpu().numpy(), Qr) <= tol
    # argument checks
    L = B.lib()
    T = shards[0].T
    import ctypes as C
    qa = (C.c_void_p * world)(*q_ptrs); ga = (C.c_void_p * world)(*gq_ptrs)
    assert L.tsid_apply_sliced(T.h, Ps[0].data_ptr(), shards[0].GP.data_ptr(), qa, ga, world, world) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_apply_sliced(T.h, Ps[0].data_ptr(), shards[0].GP.data_ptr(), qa, ga, 0, 17) == B.TSID_ERR_INVALID_ARG
    ga[1] = None
    assert L.tsid_apply_sliced(T.h, Ps[0].data_ptr(), shards[0].GP.data_ptr(), qa, ga, 0, world) == B.TSID_ERR_INVALID_ARG
    for s in shards:
        s.destroy()


@pytest.mark.parametrize("precision", ["f32", "bf16"])
def test_two_processes_step_a_row_sharded_template_over_a_process_group(precision):
    """RowShard.step with a real process group: two processes (both on this GPU), gloo underneath, three steps,
    rank 0 checks the assembled factors against the oracle's full-batch steps.  The exchange happens on the host
    with a bounded timeout; no kernel of one rank waits for the other, and no NVLink multicast is involved."""
    import os
    import socket
    import subprocess
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   NCCL_NVLS_ENABLE="0")
        procs.append(subprocess.Popen([sys.executable, os.path.join(here, "sharded_worker.py"), precision], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        outs.append(out)
    assert all(p.returncode == 0 for p in procs), outs
    assert "replicas_equal True" in outs[0]
