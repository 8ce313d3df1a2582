"""Dense tcgen05 masked-GEMM variant against the oracle (same Omega given as COO), through the C ABI.

Bars for this path (bf16 operands, fp32 accumulation, R held as fp16, E rounded to bf16 before the
second contraction): exact on small-integer instances; G within 1e-2 (infinity-norm relative) of the
bf16-emulation oracle; per-entry residual within 2e-2 and training RMSE within 1 % of the plain oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import np_coo, relerr
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bernoulli(m, n, k, density, seed, **kw):
    base = dict(values="lowrank", noise_var=1e-4, precision="bf16", eta=0.2, lam=0.0, clip=W.CLIP_NONE,
                norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT, epochs=10)
    base.update(kw)
    return W.Workload("dense-%dx%d-k%d" % (m, n, k), m, n, k, int(density * m * n), "bernoulli", density=density,
                      seed=seed, **base)


@pytest.mark.parametrize("m,n,k", [(256, 128, 64), (128, 384, 128), (512, 256, 128), (256, 2048, 64),
                                   (19200, 512, 64)])
def test_dense_exact_on_small_integers(m, n, k):
    """Integer factors and ratings: every product, residual and sum is exact in bf16/fp16/fp32, so the
    tensor-core path must reproduce the oracle bit for bit (any wrong tile, swizzle or descriptor shows).
    256 x 2048 makes several CTAs share a row block (column range split, partial gradient blocks added
    in a fixed order); 19200 x 512 has more row blocks than SMs in one pass and a split in the other."""
    rng = np.random.default_rng(m + n + k)
    P = rng.integers(-2, 3, (m, k)).astype(np.float32); Q = rng.integers(-2, 3, (n, k)).astype(np.float32)
    mask = rng.random((m, n)) < 0.3
    rows, cols = np.nonzero(mask)
    p = rng.permutation(len(rows)); rows, cols = rows[p].astype(np.int32), cols[p].astype(np.int32)
    vals = rng.integers(-8, 9, len(rows)).astype(np.float32)
    cfg = B.make_config(m, n, k, len(rows), B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
    assert T.tsid_get_info()[0] == B.TSID_PATH_DENSE_TC
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    GP, GQ = torch.full_like(Pd, 3.0), torch.full_like(Qd, 3.0)
    T.tsid_grad_step(Pd, Qd, GP, GQ)
    T.tsid_check()
    ref = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    assert np.abs(ref.GP).max() < 2 ** 20          # sums stay exactly representable in fp32
    assert np.array_equal(GP.cpu().numpy().astype(np.float64), ref.GP)
    assert np.array_equal(GQ.cpu().numpy().astype(np.float64), ref.GQ)
    assert np.array_equal(Pd.cpu().numpy(), ref.P) and np.array_equal(Qd.cpu().numpy(), ref.Q)
    T.tsid_destroy()


@pytest.mark.parametrize("k", [64, 128])
def test_dense_step_against_oracle_and_sparse_path(k):
    w = _bernoulli(640, 384, k, 0.30, seed=31 + k)
    tpl = W.make_template(w, DEV, order="shuffled")
    r, c, v = np_coo(tpl)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    out = {}
    for path in (B.TSID_PATH_DENSE_TC, B.TSID_PATH_SPARSE):
        T = B.template_from_workload(tpl, path=path)
        assert T.tsid_get_info()[0] == path
        P, Q = tpl.P0.clone(), tpl.Q0.clone()
        GP, GQ = torch.empty_like(P), torch.empty_like(Q)
        T.tsid_grad_step(P, Q, GP, GQ)
        T.tsid_check()
        out[path] = [x.cpu().numpy() for x in (GP, GQ, P, Q)]
        T.tsid_destroy()
    ref = oracle.grad_step(w.m, w.n, w.k, r, c, v, P0, Q0, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q, bf16_emulate=True)
    d = out[B.TSID_PATH_DENSE_TC]
    errs = dict(GP=relerr(d[0], ref.GP), GQ=relerr(d[1], ref.GQ), P=relerr(d[2], ref.P), Q=relerr(d[3], ref.Q))
    assert errs["GP"] <= 1e-2 and errs["GQ"] <= 1e-2 and errs["P"] <= 1e-3 and errs["Q"] <= 1e-3, errs
    s = out[B.TSID_PATH_SPARSE]
    assert relerr(d[0], s[0]) <= 1e-2 and relerr(d[1], s[1]) <= 1e-2
    # Against the oracle that rounds what this path rounds (R to fp16, E to bf16 before the second product) only two
    # things are left: fp32 summation order (1e-5 of the largest sum), and the rare residual that sits so close to
    # the midpoint of two bf16 values that the last bit of the fp32 dot product decides its rounding (measured: 2 in
    # 10^4 entries).  Such a flip moves ONE term of one gradient row by one bf16 step of e times a factor value, so
    # almost every element meets the first bound, and no element is off by more than two flipped terms.
    ref2 = oracle.grad_step(w.m, w.n, w.k, r, c, v, P0, Q0, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q,
                            bf16_emulate=oracle.EMU_TENSOR)
    e2 = oracle.residuals(w.m, w.n, w.k, r, c, v, P0, Q0, bf16_emulate=oracle.EMU_TENSOR)
    flip = 2.0 ** -8 * np.max(np.abs(e2)) * max(np.max(np.abs(P0)), np.max(np.abs(Q0)))
    for got, want in ((d[0], ref2.GP), (d[1], ref2.GQ)):
        err = np.abs(got - want)
        loose = err > 1e-5 * np.max(np.abs(want))
        assert loose.mean() <= 0.01 and err.max() <= 2 * flip, (loose.mean(), err.max(), flip)
    assert relerr(d[2], ref2.P) <= 1e-4 and relerr(d[3], ref2.Q) <= 1e-4


@pytest.mark.parametrize("side", ["rows", "cols"])
def test_dense_per_entry_residual_through_an_identity_factor(side):
    """The residual the tensor-core path itself forms (R held in fp16, S from TMEM, E rounded to bf16), entry by
    entry: with Q = I (n = k = 128) the first gradient is G_P = E Q = E, with P = I (m = k) it is G_Q = E^T.  Bar of
    this path: 2e-2 against the plain oracle on a 1-5 rating scale; against the oracle's tensor-core emulation
    level the values are equal (one term per sum)."""
    rng = np.random.default_rng(17 if side == "rows" else 18)
    k = 128
    m, n = (384, k) if side == "rows" else (k, 384)
    mask = rng.random((m, n)) < 0.3
    rows, cols = np.nonzero(mask)
    rows, cols = rows.astype(np.int32), cols.astype(np.int32)
    vals = rng.integers(1, 6, len(rows)).astype(np.float32)
    X = (3.0 + rng.standard_normal((max(m, n), k))).astype(np.float32)      # predictions around the rating scale
    eye = np.eye(k, dtype=np.float32)
    P, Q = (X, eye) if side == "rows" else (eye, X)
    cfg = B.make_config(m, n, k, len(rows), B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    T = B.Template(cfg, torch.tensor(rows, device=DEV), torch.tensor(cols, device=DEV), torch.tensor(vals, device=DEV))
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    GP, GQ = torch.empty_like(Pd), torch.empty_like(Qd)
    T.tsid_grad(Pd, Qd, GP, GQ)
    T.tsid_check()
    E = GP.cpu().numpy() if side == "rows" else GQ.cpu().numpy().T          # [m, n]: e_ij on Omega, 0 elsewhere
    assert np.all(E[~mask] == 0.0)
    e_plain = oracle.residuals(m, n, k, rows, cols, vals, P, Q)
    assert np.max(np.abs(E[rows, cols] - e_plain)) <= 2e-2
    assert np.max(np.abs(e_plain)) > 2.0                                    # residuals of the size of the scale
    e_tc = oracle.residuals(m, n, k, rows, cols, vals, P, Q, bf16_emulate=oracle.EMU_TENSOR)
    assert np.array_equal(E[rows, cols].astype(np.float64), e_tc)
    T.tsid_destroy()


def test_dense_trajectory_rmse_and_determinism():
    w = _bernoulli(512, 512, 128, 0.30, seed=77)
    tpl = W.make_template(w, DEV)
    r, c, v = np_coo(tpl)
    P0, Q0 = tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy()
    T = B.template_from_workload(tpl)             # AUTO: dense at 30 % density
    assert T.tsid_get_info() == (B.TSID_PATH_DENSE_TC, 4)
    P, Q = tpl.P0.clone(), tpl.Q0.clone()
    hist = np.array(T.tsid_fit(P, Q, w.epochs, loss_every=1))
    _, _, ref_hist = oracle.fit(w.m, w.n, w.k, r, c, v, P0, Q0, w.epochs, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
    rm, rm_ref = np.sqrt(hist / len(r)), np.sqrt(ref_hist / len(r))
    assert np.all(np.abs(rm - rm_ref) / rm_ref <= 0.01), (rm, rm_ref)
    assert rm[-1] < 0.8 * rm[0]
    P2, Q2 = tpl.P0.clone(), tpl.Q0.clone()
    T.tsid_fit(P2, Q2, w.epochs)
    assert torch.equal(P2, P) and torch.equal(Q2, Q)


def test_dense_dispatch_rules():
    w = _bernoulli(256, 256, 128, 0.30, seed=5)
    tpl = W.make_template(w, DEV)
    # AUTO stays sparse when the template does not qualify (fp32 factors) or is too sparse
    T = B.template_from_workload(tpl, precision=B.TSID_F32)
    assert T.tsid_get_info()[0] == B.TSID_PATH_SPARSE
    ws = _bernoulli(256, 256, 128, 0.02, seed=6)
    assert B.template_from_workload(W.make_template(ws, DEV)).tsid_get_info()[0] == B.TSID_PATH_SPARSE
    for bad in (B.make_config(200, 256, 128, 10, B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC),
                B.make_config(256, 256, 32, 10, B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC),
                B.make_config(256, 256, 128, 10, B.TSID_F32, B.TSID_PATH_DENSE_TC)):
        with pytest.raises(B.TsidError) as e:
            B.tsid_workspace_bytes(bad)
        assert e.value.status == B.TSID_ERR_UNSUPPORTED
    big = torch.tensor([1e6], device=DEV)
    z = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(B.TsidError) as e:     # beyond the fp16 range of the dense copy of R
        B.Template(B.make_config(128, 128, 64, 1, B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC), z, z, big)
    assert e.value.status == B.TSID_ERR_UNSUPPORTED
    # a cell listed twice cannot live in a dense matrix: refused, with or without TSID_VALIDATE
    rr = torch.tensor([0, 5, 5, 9], dtype=torch.int32, device=DEV); cc = torch.tensor([1, 7, 7, 2], dtype=torch.int32, device=DEV)
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(128, 128, 64, 4, B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC), rr, cc, torch.ones(4, device=DEV))
    assert e.value.status == B.TSID_ERR_DUPLICATE


def test_bounded_wait_expiry_is_reported_and_the_context_stays_usable():
    """Failure detection without a fault: the load-issuing thread of the tensor-core kernel is told to stop before
    work item 1 and the waits get a budget of 2e5 cycles.  The waits run out, every CTA flags it, frees its tensor
    memory and returns; the next synchronising call reports it; a fresh handle then computes the exact result."""
    rng = np.random.default_rng(99)
    m, n, k = 256, 512, 64
    P = rng.integers(-2, 3, (m, k)).astype(np.float32); Q = rng.integers(-2, 3, (n, k)).astype(np.float32)
    mask = rng.random((m, n)) < 0.3
    rows, cols = np.nonzero(mask)
    rows, cols = rows.astype(np.int32), cols.astype(np.int32)
    vals = rng.integers(-8, 9, len(rows)).astype(np.float32)
    cfg = B.make_config(m, n, k, len(rows), B.TSID_BF16_SHADOW, B.TSID_PATH_DENSE_TC, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    dev = [torch.tensor(x, device=DEV) for x in (rows, cols, vals)]
    T = B.Template(cfg, *dev)
    T.tsid_debug_stall_tile_pass(200_000, 1)
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    GP, GQ = torch.empty_like(Pd), torch.empty_like(Qd)
    T.tsid_grad_step(Pd, Qd, GP, GQ)                 # enqueues; the stall shows at the next synchronising call
    with pytest.raises(B.TsidError) as e:
        T.tsid_check()
    assert e.value.status == B.TSID_ERR_CUDA and "bounded device-side wait expired" in str(e.value)
    T.tsid_destroy()
    with pytest.raises(B.TsidError) as e:            # the hook belongs to the tensor-core path
        Ts = B.Template(B.make_config(m, n, k, len(rows), B.TSID_BF16_SHADOW, B.TSID_PATH_SPARSE), *dev)
        Ts.tsid_debug_stall_tile_pass(200_000, 1)
    assert e.value.status == B.TSID_ERR_UNSUPPORTED
    T2 = B.Template(cfg, *dev)
    Pd, Qd = torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV)
    T2.tsid_grad_step(Pd, Qd, GP, GQ)
    T2.tsid_check()
    ref = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 2.0 ** -10, 0.0, 0.1, 0, 0, 0)
    assert np.array_equal(GP.cpu().numpy().astype(np.float64), ref.GP)
    assert np.array_equal(GQ.cpu().numpy().astype(np.float64), ref.GQ)
    assert np.array_equal(Pd.cpu().numpy(), ref.P) and np.array_equal(Qd.cpu().numpy(), ref.Q)
