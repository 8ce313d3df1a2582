"""Hybrid path (dense 128 x 128 tiles of the degree-ordered template on the tensor cores, the rest on the
gather-reduce passes) against the oracle, through the C ABI.

Bars: bit-exact on small-integer instances (every product, residual and sum is exact in bf16 / fp16 / fp32,
so a wrong tile, rank table, transposed tile, chunk sum or tail entry shows as a wrong bit); on real values G
within 1e-2 and the updated factors within 1e-3 of the bf16-emulation oracle (the tiles round E to bf16
before the second product), training RMSE within 1 % of the plain oracle; run-to-run bitwise determinism.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import np_coo, relerr, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _blocky(m, n, hot_r, hot_c, dens_hot, dens_bg, seed):
    """COO positions with a populated block on scattered hot rows x hot columns over a thin background."""
    rng = np.random.default_rng(seed)
    hr = rng.choice(m, hot_r, replace=False); hc = rng.choice(n, hot_c, replace=False)
    mask = rng.random((m, n)) < dens_bg
    sub = rng.random((hot_r, hot_c)) < dens_hot
    mask[np.ix_(hr, hc)] |= sub
    rows, cols = np.nonzero(mask)
    return rows.astype(np.int32), cols.astype(np.int32), rng


def _make(rows, cols, vals, m, n, k, path, eta=2.0 ** -10, lam=0.0, xi=0.1, clip=0, norm=(0, 0), flags=0):
    cfg = B.make_config(m, n, k, len(rows), B.TSID_BF16_SHADOW, path, eta, lam, xi, clip, norm[0], norm[1], flags)
    return B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))


@pytest.mark.parametrize("m,n,k,shuffle", [(1000, 700, 64, True), (700, 1000, 128, False), (384, 256, 128, True),
                                           (5000, 300, 64, True)])
def test_hybrid_exact_on_small_integers(m, n, k, shuffle):
    rows, cols, rng = _blocky(m, n, min(300, m), min(260, n), 0.5, 0.01, seed=m + n + k)
    if shuffle:
        p = rng.permutation(len(rows)); rows, cols = rows[p], cols[p]
    vals = rng.integers(-8, 9, len(rows)).astype(np.float32)
    P = rng.integers(-2, 3, (m, k)).astype(np.float32); Q = rng.integers(-2, 3, (n, k)).astype(np.float32)
    T = _make(rows, cols, vals, m, n, k, B.TSID_PATH_HYBRID)
    assert T.tsid_get_info()[0] == B.TSID_PATH_HYBRID
    tiles, mine, tail = T.tsid_get_hybrid_info()
    assert tiles >= 4 and mine >= 480 and tail < len(rows)
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    GP, GQ = torch.full_like(Pd, 3.0), torch.full_like(Qd, 3.0)
    T.tsid_grad_step(Pd, Qd, GP, GQ)
    T.tsid_check()
    ref = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    assert np.abs(ref.GP).max() < 2 ** 20 and np.abs(ref.GQ).max() < 2 ** 20
    assert np.array_equal(GP.cpu().numpy().astype(np.float64), ref.GP)
    assert np.array_equal(GQ.cpu().numpy().astype(np.float64), ref.GQ)
    assert np.array_equal(Pd.cpu().numpy(), ref.P) and np.array_equal(Qd.cpu().numpy(), ref.Q)
    # the split step gives the same sums, and the loss / residual calls still cover every entry
    GP2, GQ2 = torch.empty_like(GP), torch.empty_like(GQ)
    P0, Q0 = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    T.tsid_grad(P0, Q0, GP2, GQ2)
    assert torch.equal(GP2, GP) and torch.equal(GQ2, GQ)
    sse, _ = T.tsid_loss(P0, Q0)
    assert sse == oracle.loss(m, n, k, rows, cols, vals, P, Q, 0.0)[0]
    T.tsid_destroy()


def _zipf(k, seed, m=3000, n=2000, nnz=600_000):
    return small_workload("hyb-zipf-k%d" % k, m, n, k, nnz, positions="zipf", precision="bf16", seed=seed,
                          values="ratings", noise_var=0.25, eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_STEP,
                          norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT, epochs=8)


@pytest.mark.parametrize("k", [64, 128])
def test_hybrid_step_against_oracle_and_sparse_path(k):
    w = _zipf(k, seed=40 + k)
    tpl = W.make_template(w, DEV, order="shuffled")
    r, c, v = np_coo(tpl)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    out = {}
    for path in (B.TSID_PATH_HYBRID, B.TSID_PATH_SPARSE):
        T = B.template_from_workload(tpl, path=path)
        assert T.tsid_get_info()[0] == path
        if path == B.TSID_PATH_HYBRID:
            tiles, mine, tail = T.tsid_get_hybrid_info()
            assert tiles > 10 and tail < 0.8 * tpl.nnz, (tiles, mine, tail)
        P, Q = tpl.P0.clone(), tpl.Q0.clone()
        GP, GQ = torch.empty_like(P), torch.empty_like(Q)
        T.tsid_grad_step(P, Q, GP, GQ)
        T.tsid_check()
        out[path] = [x.cpu().numpy() for x in (GP, GQ, P, Q)]
        T.tsid_destroy()
    ref = oracle.grad_step(w.m, w.n, w.k, r, c, v, P0, Q0, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q, bf16_emulate=True)
    d = out[B.TSID_PATH_HYBRID]
    errs = dict(GP=relerr(d[0], ref.GP), GQ=relerr(d[1], ref.GQ), P=relerr(d[2], ref.P), Q=relerr(d[3], ref.Q))
    assert errs["GP"] <= 1e-2 and errs["GQ"] <= 1e-2 and errs["P"] <= 1e-3 and errs["Q"] <= 1e-3, errs
    s = out[B.TSID_PATH_SPARSE]
    assert relerr(d[0], s[0]) <= 1e-2 and relerr(d[1], s[1]) <= 1e-2


@pytest.mark.parametrize("k", [128, 64])
def test_hybrid_trajectory_rmse_determinism_and_graph_replay(k):
    w = _zipf(k, seed=91)
    tpl = W.make_template(w, DEV)
    r, c, v = np_coo(tpl)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    T = B.template_from_workload(tpl, path=B.TSID_PATH_HYBRID)
    assert T.tsid_get_info()[0] == B.TSID_PATH_HYBRID
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    hist = np.array(T.tsid_fit(P, Q, w.epochs, loss_every=1))
    _, _, ref_hist = oracle.fit(w.m, w.n, w.k, r, c, v, P0, Q0, w.epochs, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
    rm, rm_ref = np.sqrt(hist / len(r)), np.sqrt(ref_hist / len(r))
    assert np.all(np.abs(rm - rm_ref) / rm_ref <= 0.01), (rm, rm_ref)
    P2, Q2 = tpl.P0.clone(), tpl.Q0.clone()
    T.tsid_fit(P2, Q2, w.epochs)                    # replayed from a graph
    assert torch.equal(P2, P) and torch.equal(Q2, Q)
    P3, Q3 = tpl.P0.clone(), tpl.Q0.clone()
    for _ in range(w.epochs):
        T.tsid_grad_step(P3, Q3)
    assert torch.equal(P3, P) and torch.equal(Q3, Q)
    # tsid_fit's epochs leave the tile sums to the update kernel and keep the rank-ordered shadow copies current
    # there (one launch per side): per epoch three kernels fewer than tsid_grad_step, the same bits (above)
    per_step = T.tsid_get_info()[1]
    assert T.tsid_get_fit_launches(w.epochs) == 2 + w.epochs * (per_step - 3)
    T.tsid_destroy()
    Ts = B.template_from_workload(tpl, path=B.TSID_PATH_SPARSE)
    assert Ts.tsid_get_fit_launches(5) == 1 + 5 * (Ts.tsid_get_info()[1] - 1)
    Ts.tsid_destroy()
    T2 = B.template_from_workload(tpl, path=B.TSID_PATH_HYBRID)       # a second handle: same bits
    P4, Q4 = tpl.P0.clone(), tpl.Q0.clone()
    T2.tsid_fit(P4, Q4, w.epochs)
    assert torch.equal(P4, P) and torch.equal(Q4, Q)


def test_hybrid_falls_back_to_sparse():
    # no tile reaches the threshold: the handle runs the sparse path and gives its bits
    w = small_workload("hyb-thin", 2000, 1500, 64, 15_000, precision="bf16", seed=3)
    tpl = W.make_template(w, DEV)
    Th = B.template_from_workload(tpl, path=B.TSID_PATH_HYBRID)
    Ts = B.template_from_workload(tpl, path=B.TSID_PATH_SPARSE)
    assert Th.tsid_get_info()[0] == B.TSID_PATH_SPARSE and Th.tsid_get_hybrid_info() == (0, 0, tpl.nnz)
    res = []
    for T in (Th, Ts):
        P, Q = tpl.P0.clone(), tpl.Q0.clone()
        T.tsid_fit(P, Q, 3)
        res.append((P, Q))
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
    # a duplicated cell cannot live in a dense tile: sparse path, every occurrence counted
    rows, cols, rng = _blocky(600, 500, 300, 260, 0.5, 0.01, seed=8)
    rows = np.concatenate([rows, rows[:5]]); cols = np.concatenate([cols, cols[:5]])
    vals = rng.integers(-8, 9, len(rows)).astype(np.float32)
    T = _make(rows, cols, vals, 600, 500, 64, B.TSID_PATH_HYBRID)
    assert T.tsid_get_info()[0] == B.TSID_PATH_SPARSE
    P = rng.integers(-2, 3, (600, 64)).astype(np.float32); Q = rng.integers(-2, 3, (500, 64)).astype(np.float32)
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    GP, GQ = torch.empty_like(Pd), torch.empty_like(Qd)
    T.tsid_grad_step(Pd, Qd, GP, GQ)
    ref = oracle.grad_step(600, 500, 64, rows, cols, vals, P, Q, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    assert np.array_equal(GP.cpu().numpy().astype(np.float64), ref.GP)
    with pytest.raises(B.TsidError) as e:
        _make(rows, cols, vals, 600, 500, 64, B.TSID_PATH_HYBRID, flags=B.TSID_VALIDATE)
    assert e.value.status == B.TSID_ERR_DUPLICATE


def test_hybrid_dispatch_rules():
    for bad in (B.make_config(3000, 2000, 64, 600_000, B.TSID_F32, B.TSID_PATH_HYBRID),
                B.make_config(3000, 2000, 32, 600_000, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID),
                B.make_config(3000, 2000, 64, 600_000, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID, clip=B.TSID_CLIP_ASYM_ENTRY),
                B.make_config(3000, 2000, 64, 600_000, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID, flags=B.TSID_VALUES_U8),
                B.make_config(300_000, 2000, 64, 10_000, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID)):
        with pytest.raises(B.TsidError) as e:
            B.tsid_workspace_bytes(bad)
        assert e.value.status == B.TSID_ERR_UNSUPPORTED
    # AUTO: small templates stay on the sparse path; the workspace of AUTO equals that of the path it resolves to
    small = B.make_config(3000, 2000, 64, 600_000, B.TSID_BF16_SHADOW, B.TSID_PATH_AUTO)
    assert B.tsid_workspace_bytes(small) == B.tsid_workspace_bytes(
        B.make_config(3000, 2000, 64, 600_000, B.TSID_BF16_SHADOW, B.TSID_PATH_SPARSE))
    big = B.make_config(200_000, 100_000, 64, 100_000_000, B.TSID_BF16_SHADOW, B.TSID_PATH_AUTO)
    assert B.tsid_workspace_bytes(big) == B.tsid_workspace_bytes(
        B.make_config(200_000, 100_000, 64, 100_000_000, B.TSID_BF16_SHADOW, B.TSID_PATH_HYBRID))
