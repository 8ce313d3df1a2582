"""Parity of the CUDA path with the CPU oracle, element by element, through the C ABI.

Bars: fp32 path: max|a - ref| / max|ref| <= 1e-4 for G_P, G_Q, P', Q'.  bf16 path: the same bar
against the oracle's bf16-emulation mode (inputs rounded to bf16, double sums); against the plain
oracle, per-entry residual error <= 2e-2 and training RMSE within 1 %.  Integers bit-exact (layout tests).
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import F32_TOL, gpu_step, np_coo, oracle_step, relerr, rowwise_relerr, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _assert_step(tpl, precision, tol=F32_TOL):
    emu = precision == B.TSID_BF16_SHADOW
    T, P1, Q1, GP, GQ = gpu_step(tpl, precision=precision)
    ref = oracle_step(tpl, tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(), bf16_emulate=emu)
    errs = dict(GP=relerr(GP, ref.GP), GQ=relerr(GQ, ref.GQ), P=relerr(P1, ref.P), Q=relerr(Q1, ref.Q))
    assert all(v <= tol for v in errs.values()), errs
    # and row by row, so that a thinly populated row cannot hide behind the largest one (entry-wise clip: the sums
    # are of clipped terms, whose scale the floor of the per-row metric does not describe; left to the metric above)
    if tpl.w.clip != W.CLIP_ASYM_ENTRY:
        cr = np.bincount(tpl.rows.cpu().numpy(), minlength=tpl.w.m); cc = np.bincount(tpl.cols.cpu().numpy(), minlength=tpl.w.n)
        rw = dict(GP=rowwise_relerr(GP, ref.GP, cr), GQ=rowwise_relerr(GQ, ref.GQ, cc))
        assert all(v <= tol for v in rw.values()), rw
    T.tsid_destroy()
    return errs


def test_c1_step_fp32():
    _assert_step(W.make_template(W.C1, DEV), B.TSID_F32)


@pytest.mark.parametrize("precision", [B.TSID_F32, B.TSID_BF16_SHADOW])
@pytest.mark.parametrize("k", [8, 16, 24, 32, 48, 64, 96, 128, 200, 256])
def test_rank_sweep(k, precision):
    """Every kernel instantiation, ragged k (not a power of two), several tiles and a ragged tail."""
    w = small_workload("k%d" % k, 1500, 1100, k, 90_000 + 13, positions="zipf", seed=100 + k,
                       values="ratings", noise_var=0.25, eta=0.05, lam=0.03, clip=W.CLIP_ASYM_STEP,
                       norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT)
    _assert_step(W.make_template(w, DEV, order="shuffled"), precision)


def test_k_multiple_of_4_fp32():
    for k in (4, 12, 20):
        w = small_workload("k%d" % k, 700, 500, k, 20_000, seed=k)
        _assert_step(W.make_template(w, DEV, order="shuffled"), B.TSID_F32)


@pytest.mark.parametrize("clip", [W.CLIP_NONE, W.CLIP_ASYM_STEP, W.CLIP_ASYM_GRAD, W.CLIP_ASYM_ENTRY])
@pytest.mark.parametrize("norm_p,norm_q", [(0, 0), (0, 1), (1, 1)])
def test_modes(clip, norm_p, norm_q):
    w = small_workload("modes", 900, 1300, 32, 60_000, positions="zipf", seed=5, values="ratings", noise_var=0.25,
                       eta=0.05, lam=0.03, xi=0.1, clip=clip, norm_p=norm_p, norm_q=norm_q)
    tpl = W.make_template(w, DEV, order="shuffled")
    _assert_step(tpl, B.TSID_F32)
    if clip == W.CLIP_ASYM_STEP:   # the clip must bite, and cap increases at eta * xi
        T, P1, Q1, _, _ = gpu_step(tpl)
        inc = P1 - tpl.P0.cpu().numpy()
        assert inc.max() <= w.eta * w.xi * (1 + 1e-5) and np.isclose(inc.max(), w.eta * w.xi, rtol=1e-5)
        assert inc.min() < -w.eta * w.xi


@pytest.mark.parametrize("precision", [B.TSID_F32, B.TSID_BF16_SHADOW])
@pytest.mark.parametrize("k", [16, 40, 64, 128])
def test_entrywise_clip_rank_sweep(k, precision):
    """Sec. 5.3 applied entry by entry (literal Eq. 9 normalisation: q side only), every staged instantiation."""
    w = small_workload("entry-k%d" % k, 1200, 900, k, 70_000 + 7, positions="zipf", seed=300 + k, values="ratings",
                       noise_var=0.25, eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_ENTRY, norm_p=W.NORM_NONE,
                       norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV, order="shuffled")
    _assert_step(tpl, precision)
    T, P1, _, GP, _ = gpu_step(tpl, precision=precision)
    assert GP.max() <= 0.1 * np.bincount(tpl.rows.cpu().numpy(), minlength=w.m).max() + 1e-3   # each term <= xi


def test_split_rows_and_empty_rows():
    """Rows far longer than one segment (fixed-order grid-level reduction) next to empty rows and columns."""
    m, n, k = 40, 9000, 64
    rng = np.random.default_rng(3)
    rows, cols = [], []
    for i, cnt in enumerate([8990, 5000, 1025, 1024, 1023, 513, 512, 511, 1, 0, 33]):
        c = rng.choice(n - 7, cnt, replace=False)      # the last 7 columns stay empty
        rows.append(np.full(cnt, i * 3)); cols.append(c)
    rows = np.concatenate(rows).astype(np.int32); cols = np.concatenate(cols).astype(np.int32)
    p = rng.permutation(len(rows)); rows, cols = rows[p], cols[p]
    vals = rng.standard_normal(len(rows)).astype(np.float32)
    P0 = (rng.standard_normal((m, k)) * 0.4).astype(np.float32); Q0 = (rng.standard_normal((n, k)) * 0.4).astype(np.float32)
    for prec, emu in ((B.TSID_F32, False), (B.TSID_BF16_SHADOW, True)):
        cfg = B.make_config(m, n, k, len(rows), prec, B.TSID_PATH_SPARSE, 0.05, 0.03, 0.1, B.TSID_CLIP_ASYM_STEP, 1, 1)
        T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
        P = torch.tensor(P0, device=DEV); Q = torch.tensor(Q0, device=DEV)
        GP = torch.full_like(P, 7.0); GQ = torch.full_like(Q, 7.0)      # stale contents must be overwritten
        T.tsid_grad_step(P, Q, GP, GQ)
        ref = oracle.grad_step(m, n, k, rows, cols, vals, P0, Q0, 0.05, 0.03, 0.1, 1, 1, 1, bf16_emulate=emu)
        assert relerr(GP.cpu().numpy(), ref.GP) <= F32_TOL and relerr(GQ.cpu().numpy(), ref.GQ) <= F32_TOL
        assert relerr(P.cpu().numpy(), ref.P) <= F32_TOL and relerr(Q.cpu().numpy(), ref.Q) <= F32_TOL
        assert not GP[27].any() and not GQ[-7:].any()                   # empty row / columns: exact zeros
        T.tsid_destroy()


@pytest.mark.parametrize("precision,emu", [(B.TSID_F32, False), (B.TSID_BF16_SHADOW, True)])
def test_degenerate_shapes(precision, emu):
    """One cell, one row, one column, and a fully observed matrix (Omega = every cell)."""
    rng = np.random.default_rng(17)
    k = 16
    for m, n in ((1, 1), (1, 3000), (3000, 1), (37, 53)):
        ids = np.arange(m * n)
        rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
        p = rng.permutation(m * n); rows, cols = rows[p], cols[p]
        vals = rng.standard_normal(m * n).astype(np.float32)
        P0 = (rng.standard_normal((m, k)) * 0.5).astype(np.float32); Q0 = (rng.standard_normal((n, k)) * 0.5).astype(np.float32)
        cfg = B.make_config(m, n, k, m * n, precision, B.TSID_PATH_SPARSE, 0.05, 0.03, 0.1, B.TSID_CLIP_ASYM_STEP, 1, 1,
                            B.TSID_VALIDATE)
        T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
        P = torch.tensor(P0, device=DEV); Q = torch.tensor(Q0, device=DEV)
        GP, GQ = torch.empty_like(P), torch.empty_like(Q)
        T.tsid_grad_step(P, Q, GP, GQ)
        T.tsid_check()
        ref = oracle.grad_step(m, n, k, rows, cols, vals, P0, Q0, 0.05, 0.03, 0.1, 1, 1, 1, bf16_emulate=emu)
        for got, want in ((GP, ref.GP), (GQ, ref.GQ), (P, ref.P), (Q, ref.Q)):
            assert relerr(got.cpu().numpy(), want) <= F32_TOL, (m, n)
        if not emu:   # the fully observed case is the textbook dense formula
            E = np.zeros((m, n)); E[rows, cols] = vals
            E = E - P0.astype(np.float64) @ Q0.astype(np.float64).T
            assert relerr(GP.cpu().numpy(), E @ Q0) <= F32_TOL and relerr(GQ.cpu().numpy(), E.T @ P0) <= F32_TOL
        T.tsid_destroy()


def test_zero_gradient_at_truth_and_empty_template():
    m, n, k = 300, 200, 16
    rng = np.random.default_rng(4)
    P = rng.integers(-3, 4, (m, k)).astype(np.float32); Q = rng.integers(-3, 4, (n, k)).astype(np.float32)
    ids = rng.choice(m * n, 5000, replace=False)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    vals = np.sum(P[rows] * Q[cols], axis=1).astype(np.float32)
    for prec in (B.TSID_F32, B.TSID_BF16_SHADOW):   # small integers are exact in bf16 too
        cfg = B.make_config(m, n, k, 5000, prec, B.TSID_PATH_SPARSE, 0.3, 0.0, 0.1, B.TSID_CLIP_ASYM_STEP, 1, 1)
        T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
        Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
        GP, GQ = torch.ones_like(Pd), torch.ones_like(Qd)
        T.tsid_grad_step(Pd, Qd, GP, GQ)
        assert not GP.any() and not GQ.any()
        assert torch.equal(Pd.cpu(), torch.tensor(P)) and torch.equal(Qd.cpu(), torch.tensor(Q))
        assert T.tsid_loss(Pd, Qd)[0] == 0.0
        T.tsid_destroy()
    # empty Omega: pure decay
    cfg = B.make_config(m, n, k, 0, B.TSID_F32, B.TSID_PATH_SPARSE, 0.1, 0.5, 0.1, 0, 1, 1)
    z = torch.zeros(0, dtype=torch.int32, device=DEV)
    T = B.Template(cfg, z, z, torch.zeros(0, device=DEV))
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    T.tsid_grad_step(Pd, Qd)
    assert relerr(Pd.cpu().numpy(), P * 0.9) < 1e-6 and relerr(Qd.cpu().numpy(), Q * 0.9) < 1e-6


def test_bf16_against_plain_oracle_residual_and_rmse():
    """bf16 path vs the fp32-input oracle: residual error <= 2e-2, training RMSE within 1 %."""
    w = W.scaled(W.C3, "C3-small", 6000, 4000, 400_000, epochs=10)
    tpl = W.make_template(w, DEV, order="shuffled")
    r, c, v = np_coo(tpl)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    T = B.template_from_workload(tpl)
    e = T.tsid_residuals(tpl.P0, tpl.Q0).cpu().numpy()
    lay = oracle.layout(w.m, w.n, r, c, v)
    csr_rows = np.repeat(np.arange(w.m, dtype=np.int32), np.diff(lay.row_ptr))
    e_ref = oracle.residuals(w.m, w.n, w.k, csr_rows, lay.col_idx, lay.val_csr, P0, Q0)
    assert np.max(np.abs(e - e_ref)) <= 2e-2
    e_emu = oracle.residuals(w.m, w.n, w.k, csr_rows, lay.col_idx, lay.val_csr, P0, Q0, bf16_emulate=True)
    assert np.max(np.abs(e - e_emu)) <= 1e-5 * max(1.0, np.max(np.abs(e_emu)))
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    hist = T.tsid_fit(P, Q, w.epochs, loss_every=1)
    _, _, ref_hist = oracle.fit(w.m, w.n, w.k, r, c, v, P0, Q0, w.epochs, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
    rm, rm_ref = np.sqrt(np.array(hist) / len(r)), np.sqrt(ref_hist / len(r))
    assert np.all(np.abs(rm - rm_ref) / rm_ref <= 0.01), (rm, rm_ref)
    assert rm[-1] < rm[0]


def test_c1_fit_trajectory_and_loss():
    w = W.C1
    tpl = W.make_template(w, DEV)
    r, c, v = np_coo(tpl)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    T = B.template_from_workload(tpl)
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    hist = np.array(T.tsid_fit(P, Q, w.epochs, loss_every=1))
    Pr, Qr, ref_hist = oracle.fit(w.m, w.n, w.k, r, c, v, P0, Q0, w.epochs, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
    assert len(hist) == w.epochs + 1
    assert np.max(np.abs(hist - ref_hist) / ref_hist) <= 1e-4
    assert np.all(np.diff(hist) < 0)
    assert relerr(P.cpu().numpy(), Pr) <= 5e-4 and relerr(Q.cpu().numpy(), Qr) <= 5e-4   # 20 steps of drift
    sse, obj = T.tsid_loss(P, Q)
    sse_r, obj_r = oracle.loss(w.m, w.n, w.k, r, c, v, P.cpu().numpy(), Q.cpu().numpy(), 0.0)
    assert abs(sse - sse_r) / sse_r <= 1e-5 and abs(obj - obj_r) / obj_r <= 1e-5
    # fit without loss evaluation gives bitwise the same factors; so does a second run (determinism)
    for _ in range(2):
        P2, Q2 = tpl.P0.clone(), tpl.Q0.clone()
        T.tsid_fit(P2, Q2, w.epochs)
        assert torch.equal(P2, P) and torch.equal(Q2, Q)
    P3, Q3 = tpl.P0.clone(), tpl.Q0.clone()
    for _ in range(w.epochs):
        T.tsid_grad_step(P3, Q3)
    assert torch.equal(P3, P) and torch.equal(Q3, Q)


@pytest.mark.parametrize("path,precision", [(B.TSID_PATH_SPARSE, B.TSID_F32), (B.TSID_PATH_SPARSE, B.TSID_BF16_SHADOW),
                                            (B.TSID_PATH_DENSE_TC, B.TSID_BF16_SHADOW)])
def test_fit_graph_replay_equals_step_by_step(path, precision):
    """tsid_fit replays its epochs from a captured graph (8 steps per launch, the rest one by one): bitwise the
    factors of the same number of tsid_grad_step calls; again on the same arrays (the cached graph), on other
    arrays (a new capture) and below the replay threshold."""
    w = small_workload("graph", 512, 384, 64, 30_000, positions="zipf", seed=21, values="ratings", noise_var=0.25,
                       eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV, order="shuffled")
    T = B.template_from_workload(tpl, path=path, precision=precision)
    assert T.tsid_get_info()[0] == path
    Pa, Qa = tpl.P0.clone(), tpl.Q0.clone()
    Pb, Qb = tpl.P0.clone(), tpl.Q0.clone()
    Pr, Qr = tpl.P0.clone(), tpl.Q0.clone()
    done = 0
    for epochs, (P, Q) in ((37, (Pa, Qa)), (16, (Pa, Qa)), (5, (Pa, Qa)), (58, (Pb, Qb))):
        if P is Pb:
            Pr.copy_(tpl.P0); Qr.copy_(tpl.Q0)
        T.tsid_fit(P, Q, epochs)
        for _ in range(epochs):
            T.tsid_grad_step(Pr, Qr)
        T.tsid_check()
        assert torch.equal(P, Pr) and torch.equal(Q, Qr), (epochs, done)
        done += epochs
    T.tsid_destroy()


def test_fit_inside_a_callers_graph_capture():
    """tsid_fit with loss_every = 0 enqueues work only: a caller can capture it into a CUDA graph of its own
    (the library then launches step by step instead of replaying its own graph) and replay it."""
    w = small_workload("cap", 384, 256, 32, 20_000, positions="zipf", seed=23, values="ratings", noise_var=0.25,
                       eta=0.05, lam=0.03, xi=0.1, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV, order="shuffled")
    s = torch.cuda.Stream(device=DEV)
    cfg = B.make_config(w.m, w.n, w.k, tpl.nnz, B.TSID_BF16_SHADOW, B.TSID_PATH_SPARSE, w.eta, w.lam, w.xi, w.clip,
                        w.norm_p, w.norm_q)
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        T = B.Template(cfg, tpl.rows, tpl.cols, tpl.vals, stream=s)
        P, Q = tpl.P0.clone(), tpl.Q0.clone()
        Pr, Qr = tpl.P0.clone(), tpl.Q0.clone()
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            T.tsid_fit(P, Q, 12)
        g.replay()
        g.replay()
        for _ in range(24):
            T.tsid_grad_step(Pr, Qr)
        T.tsid_check()
    torch.cuda.synchronize()
    assert torch.equal(P, Pr) and torch.equal(Q, Qr)
    T.tsid_destroy()


def test_objective_with_regulariser():
    w = small_workload("obj", 800, 600, 32, 40_000, seed=11, lam=0.05)
    tpl = W.make_template(w, DEV, order="shuffled")
    r, c, v = np_coo(tpl)
    T = B.template_from_workload(tpl)
    sse, obj = T.tsid_loss(tpl.P0, tpl.Q0)
    sse_r, obj_r = oracle.loss(w.m, w.n, w.k, r, c, v, tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(), w.lam)
    assert abs(sse - sse_r) / sse_r <= 1e-5 and abs(obj - obj_r) / obj_r <= 1e-5 and obj > sse


def test_c2_full_size_step_and_determinism():
    """Full C2 (10M entries, Zipf): one oracle step takes seconds, so compare every element."""
    tpl = W.make_template(W.C2, DEV, order="shuffled")
    errs = _assert_step(tpl, B.TSID_F32)
    T, P1, Q1, GP, GQ = gpu_step(tpl)
    T2, P1b, Q1b, GPb, GQb = gpu_step(tpl)
    for a, b in ((P1, P1b), (Q1, Q1b), (GP, GPb), (GQ, GQb)):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_nonfinite_is_reported():
    w = small_workload("nf", 200, 150, 16, 3000, seed=2, eta=1e30)
    tpl = W.make_template(w, DEV)
    T = B.template_from_workload(tpl)
    P, Q = tpl.P0.clone() * 1e20, tpl.Q0.clone() * 1e20
    T.tsid_grad_step(P, Q)
    with pytest.raises(B.TsidError) as e:
        T.tsid_check()
    assert e.value.status == B.TSID_ERR_NONFINITE


def test_argument_errors():
    w = small_workload("arg", 64, 48, 16, 500, seed=1)
    tpl = W.make_template(w, DEV)
    T = B.template_from_workload(tpl)
    import ctypes as C
    L = B.lib()
    assert L.tsid_grad_step(T.h, None, tpl.Q0.data_ptr(), None, None) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_grad_step(T.h, tpl.P0.data_ptr() + 4, tpl.Q0.data_ptr(), None, None) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_fit(T.h, tpl.P0.data_ptr(), tpl.Q0.data_ptr(), -1, 0, None) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_grad_step(None, None, None, None, None) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_destroy(None) == B.TSID_OK
    assert b"epochs" in L.tsid_last_error(T.h)


@pytest.mark.parametrize("precision,k", [("f32", 32), ("bf16", 64), ("bf16", 128)])
def test_byte_value_streams_give_the_same_bits(precision, k):
    """TSID_VALUES_U8: ratings streamed as one byte each.  Same arithmetic, so the same bits; a value that
    is not an integer in [0, 255] is refused at create."""
    w = small_workload("u8", 3000, 1700, k, 200_000, positions="zipf", precision=precision, seed=3 + k,
                       values="ratings", eta=0.05, lam=0.03, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT,
                       norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV, order="shuffled")
    assert float(tpl.vals.min()) >= 1 and float(tpl.vals.max()) <= 5
    outs = []
    for flags in (0, B.TSID_VALUES_U8):
        T = B.template_from_workload(tpl, path=B.TSID_PATH_SPARSE, flags=flags)
        P, Q = tpl.P0.clone(), tpl.Q0.clone()
        GP, GQ = torch.empty_like(P), torch.empty_like(Q)
        T.tsid_grad_step(P, Q, GP, GQ)
        T.tsid_grad_step(P, Q)
        T.tsid_check()
        outs.append((P, Q, GP, GQ))
        T.tsid_destroy()
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    bad = tpl.vals.clone()
    bad[7] = 2.5
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(w.m, w.n, w.k, tpl.nnz, flags=B.TSID_VALUES_U8), tpl.rows, tpl.cols, bad)
    assert e.value.status == B.TSID_ERR_UNSUPPORTED


@pytest.mark.parametrize("precision", ["f32", "bf16"])
def test_host_buffer_call_equals_the_device_path(precision):
    """tsid_fit_host (pinned host triples and factors in, fitted factors out; the factors are uploaded on a
    second stream while the layout is built) gives bitwise what create + fit give on device buffers."""
    w = small_workload("host", 2100, 1300, 32, 150_000, positions="zipf", precision=precision, seed=77,
                       values="ratings", eta=0.05, lam=0.03, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT,
                       norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, DEV, order="shuffled")
    T = B.template_from_workload(tpl, path=B.TSID_PATH_SPARSE)
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    T.tsid_fit(P, Q, 4)
    sse_dev, _ = T.tsid_loss(P, Q)
    T.tsid_destroy()
    prec = B.TSID_BF16_SHADOW if precision == "bf16" else B.TSID_F32
    cfg = B.make_config(w.m, w.n, w.k, tpl.nnz, prec, B.TSID_PATH_SPARSE, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
    ws = torch.empty(B.tsid_workspace_bytes_host(cfg) + 256, dtype=torch.uint8, device=DEV)
    hP, hQ = tpl.P0.cpu().pin_memory(), tpl.Q0.cpu().pin_memory()
    sse = B.tsid_fit_host(cfg, tpl.rows.cpu().pin_memory(), tpl.cols.cpu().pin_memory(), tpl.vals.cpu().pin_memory(),
                          hP, hQ, 4, ws, want_sse=True)
    assert torch.equal(hP, P.cpu()) and torch.equal(hQ, Q.cpu())
    assert sse == sse_dev
