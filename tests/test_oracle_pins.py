"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's loops: they use hand-worked numbers
(tests/golden), exact rational brute force over a dense masked matrix, numpy
dense algebra, finite differences of the loss, and invariants.
"""
import itertools
import struct
from fractions import Fraction

import numpy as np
import pytest

import oracle
from conftest import read_golden

RNG = np.random.default_rng(12345)


def _arr(g, key, shape=None, dtype=np.float64):
    a = np.array(g[key], dtype=dtype)
    return a.reshape(shape) if shape else a


def _inst(g):
    m, n, k = int(g["m"][0]), int(g["n"][0]), int(g["k"][0])
    return (m, n, k, _arr(g, "rows", dtype=np.int32), _arr(g, "cols", dtype=np.int32),
            _arr(g, "vals", dtype=np.float32), _arr(g, "P", (m, k), np.float32),
            _arr(g, "Q", (n, k), np.float32))


# ---------------------------------------------------------------- hand-worked 3x2 example
def test_worked_example_residuals_sums_loss(golden_3x2):
    g = golden_3x2
    m, n, k, rows, cols, vals, P, Q = _inst(g)
    e = oracle.residuals(m, n, k, rows, cols, vals, P, Q)
    assert np.array_equal(e, _arr(g, "e"))
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.1, 0.25, 2.0)
    assert np.array_equal(st.GP, _arr(g, "GP", (m, k)))
    assert np.array_equal(st.GQ, _arr(g, "GQ", (n, k)))
    sse, obj = oracle.loss(m, n, k, rows, cols, vals, P, Q, 0.25)
    assert sse == g["sse"][0] and obj == g["obj"][0]
    tr = g["trace"][0]
    assert np.sum(st.GP * P) == tr and np.sum(st.GQ * Q) == tr
    assert np.sum(e * np.sum(P[rows] * Q[cols], axis=1)) == tr


@pytest.mark.parametrize("tag,clip,norm", [
    ("none_unclipped", oracle.CLIP_NONE, oracle.NORM_NONE),
    ("none_step", oracle.CLIP_ASYM_STEP, oracle.NORM_NONE),
    ("count_step", oracle.CLIP_ASYM_STEP, oracle.NORM_COUNT),
])
def test_worked_example_updates(golden_3x2, tag, clip, norm):
    g = golden_3x2
    m, n, k, rows, cols, vals, P, Q = _inst(g)
    eta, lam, xi = g["eta"][0], g["lambda"][0], g["xi"][0]
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, xi, clip, norm, norm)
    np.testing.assert_allclose(st.P, _arr(g, "P1_" + tag, (m, k)), rtol=0, atol=1e-7)
    np.testing.assert_allclose(st.Q, _arr(g, "Q1_" + tag, (n, k)), rtol=0, atol=1e-7)
    # the loss after the step, from the exact decimal factors of the golden file
    Pn = _arr(g, "P1_" + tag, (m, k)); Qn = _arr(g, "Q1_" + tag, (n, k))
    sse = sum((float(vals[t]) - Pn[rows[t]] @ Qn[cols[t]]) ** 2 for t in range(len(vals)))
    assert abs(sse - g["sse1_" + tag][0]) < 1e-12
    sse_o, obj_o = oracle.loss(m, n, k, rows, cols, vals, st.P, st.Q, lam)
    assert abs(sse_o - g["sse1_" + tag][0]) < 1e-5
    if "obj1_" + tag in g:
        assert abs(obj_o - g["obj1_" + tag][0]) < 1e-5


def test_worked_example_directions(golden_3x2):
    g = golden_3x2
    m, n, k, rows, cols, vals, P, Q = _inst(g)
    eta, lam = g["eta"][0], g["lambda"][0]
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, 2.0)
    assert np.array_equal(st.DP, _arr(g, "DP_none", (m, k)))
    assert np.array_equal(st.DQ, _arr(g, "DQ_none", (n, k)))
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, 1e30, oracle.CLIP_ASYM_STEP,
                          oracle.NORM_COUNT, oracle.NORM_COUNT)
    assert np.array_equal(st.DP, _arr(g, "DP_count", (m, k)))
    assert np.array_equal(st.DQ, _arr(g, "DQ_count", (n, k)))
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, 2.0, oracle.CLIP_ASYM_GRAD)
    assert np.array_equal(st.DP, _arr(g, "DP_none_gradclip", (m, k)))
    assert np.array_equal(st.DQ, _arr(g, "DQ_none_gradclip", (n, k)))
    # literal Eq. 9 setting: P side not normalised, Q side divided by the column count
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, 2.0, oracle.CLIP_NONE,
                          oracle.NORM_NONE, oracle.NORM_COUNT)
    assert np.array_equal(st.DP, _arr(g, "DP_none", (m, k)))
    assert np.array_equal(st.DQ, _arr(g, "DQ_count", (n, k)))


def test_worked_example_entrywise_clip(golden_3x2):
    """Sec. 5.3 taken entry by entry: clipped per-entry directions, summed, divided by the count on the q side."""
    g = golden_3x2
    m, n, k, rows, cols, vals, P, Q = _inst(g)
    eta, lam, xi = g["eta"][0], g["lambda"][0], g["xi"][0]
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, xi, oracle.CLIP_ASYM_ENTRY, 0, 0)
    assert np.array_equal(st.GP, _arr(g, "GP_entry", (m, k))) and np.array_equal(st.GQ, _arr(g, "GQ_entry", (n, k)))
    np.testing.assert_allclose(st.P, _arr(g, "P1_entry_none", (m, k)), rtol=0, atol=1e-7)
    np.testing.assert_allclose(st.Q, _arr(g, "Q1_entry_none", (n, k)), rtol=0, atol=1e-7)
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, xi, oracle.CLIP_ASYM_ENTRY, 0, 1)
    np.testing.assert_allclose(st.P, _arr(g, "P1_entry_none", (m, k)), rtol=0, atol=1e-7)
    np.testing.assert_allclose(st.Q, _arr(g, "Q1_entry_count", (n, k)), rtol=0, atol=1e-7)
    # with a threshold that never bites and lambda = 0 it is the plain summed direction 2 G / s
    big = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, 0.0, 1e30, oracle.CLIP_ASYM_ENTRY, 1, 1)
    ref = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, 0.0, 1e30, oracle.CLIP_NONE, 1, 1)
    np.testing.assert_allclose(big.DP, ref.DP, rtol=1e-15) and np.testing.assert_allclose(big.DQ, ref.DQ, rtol=1e-15)


def test_worked_example_entrywise_clip_with_bf16_emulation(golden_3x2):
    """The entry-wise clip on a bf16 template: rounded values wherever a factor is read (regulariser included),
    step added to the fp32 master.  Hand-worked numbers, plus the identity with the plain branch on pre-rounded
    factors, so that rounding only one operand, or reading the master in the regulariser, fails here."""
    g = golden_3x2
    m, n, k, rows, cols, vals, _, Q = _inst(g)
    P = _arr(g, "P_emu", (m, k), np.float32)
    eta, lam, xi = g["eta"][0], g["lambda"][0], g["xi"][0]
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, xi, oracle.CLIP_ASYM_ENTRY, 0, 0, bf16_emulate=True)
    assert np.array_equal(st.GP, _arr(g, "GP_entry_emu", (m, k)))
    assert np.array_equal(st.GQ, _arr(g, "GQ_entry_emu", (n, k)))
    np.testing.assert_allclose(st.P, _arr(g, "P1_entry_emu_none", (m, k)), rtol=0, atol=1e-7)
    np.testing.assert_allclose(st.Q, _arr(g, "Q1_entry_emu_none", (n, k)), rtol=0, atol=1e-7)
    assert st.GP[0, 0] != 0.8388671875          # what the master value in the regulariser would give
    # on random factors: the sums equal those of the plain branch fed pre-rounded factors, the step starts
    # from the unrounded master
    rng = np.random.default_rng(5)
    m2, n2, k2, nnz = 23, 17, 8, 140
    cells = rng.choice(m2 * n2, nnz, replace=False)
    r2, c2 = (cells // n2).astype(np.int32), (cells % n2).astype(np.int32)
    v2 = rng.normal(size=nnz).astype(np.float32)
    P2 = rng.normal(size=(m2, k2)).astype(np.float32); Q2 = rng.normal(size=(n2, k2)).astype(np.float32)
    rnd = np.vectorize(oracle.bf16_round, otypes=[np.float32])
    Pr, Qr = rnd(P2), rnd(Q2)
    assert np.any(Pr != P2) and np.any(Qr != Q2)
    for norms in ((0, 0), (0, 1), (1, 1)):
        emu = oracle.grad_step(m2, n2, k2, r2, c2, v2, P2, Q2, 0.05, 0.3, 0.4, oracle.CLIP_ASYM_ENTRY, *norms, bf16_emulate=True)
        pre = oracle.grad_step(m2, n2, k2, r2, c2, v2, Pr, Qr, 0.05, 0.3, 0.4, oracle.CLIP_ASYM_ENTRY, *norms)
        assert np.array_equal(emu.GP, pre.GP) and np.array_equal(emu.GQ, pre.GQ)
        assert np.array_equal(emu.DP, pre.DP) and np.array_equal(emu.DQ, pre.DQ)
        np.testing.assert_allclose(emu.P, (P2.astype(np.float64) + 0.05 * pre.DP).astype(np.float32), rtol=0, atol=0)
        np.testing.assert_allclose(emu.Q, (Q2.astype(np.float64) + 0.05 * pre.DQ).astype(np.float32), rtol=0, atol=0)
        assert np.any(emu.P != pre.P)


def test_worked_example_layout(golden_3x2):
    g = golden_3x2
    lay = oracle.layout(3, 2, _arr(g, "shuf_rows", dtype=np.int32), _arr(g, "shuf_cols", dtype=np.int32),
                        _arr(g, "shuf_vals", dtype=np.float32))
    for key in ("row_ptr", "col_idx", "val_csr", "col_ptr", "row_idx", "val_csc", "perm"):
        assert np.array_equal(getattr(lay, key).astype(np.float64), _arr(g, key)), key


# ---------------------------------------------------------------- 8x6 rank-2 brute force (exact rationals)
def _brute_force_dense(m, n, k, mask, R, P, Q, eta, lam, xi, clip, norm_p, norm_q):
    """Dense, masked, exact: loops over every cell of the m x n matrix with Fractions."""
    F = Fraction
    E = [[(R[i][j] - sum(P[i][l] * Q[j][l] for l in range(k))) if mask[i][j] else F(0)
          for j in range(n)] for i in range(m)]
    GP = [[sum(E[i][j] * Q[j][l] for j in range(n)) for l in range(k)] for i in range(m)]
    GQ = [[sum(E[i][j] * P[i][l] for i in range(m)) for l in range(k)] for j in range(n)]
    cr = [sum(mask[i]) for i in range(m)]
    cc = [sum(mask[i][j] for i in range(m)) for j in range(n)]
    if clip == oracle.CLIP_ASYM_ENTRY:   # every observed cell adds its own clipped direction
        GP = [[sum(min(2 * E[i][j] * Q[j][l] - 2 * lam * P[i][l], xi) for j in range(n) if mask[i][j])
               for l in range(k)] for i in range(m)]
        GQ = [[sum(min(2 * E[i][j] * P[i][l] - 2 * lam * Q[j][l], xi) for i in range(m) if mask[i][j])
               for l in range(k)] for j in range(n)]

    def upd(X, G, cnt, norm):
        out = []
        for r, row in enumerate(X):
            s = max(1, cnt[r]) if norm else 1
            new = []
            for l, x in enumerate(row):
                if clip == oracle.CLIP_ASYM_ENTRY:
                    new.append(x + eta * G[r][l] / s)
                    continue
                d = 2 * G[r][l] / s - 2 * lam * x
                if clip == oracle.CLIP_ASYM_STEP:
                    d = min(d, xi)          # the verbal rule: positive values above xi become xi
                elif clip == oracle.CLIP_ASYM_GRAD:
                    d = max(d, -xi)
                new.append(x + eta * d)
            out.append(new)
        return out

    sse = sum(E[i][j] ** 2 for i in range(m) for j in range(n))
    return GP, GQ, upd(P, GP, cr, norm_p), upd(Q, GQ, cc, norm_q), sse


@pytest.mark.parametrize("clip,norm_p,norm_q", list(itertools.product(
    [oracle.CLIP_NONE, oracle.CLIP_ASYM_STEP, oracle.CLIP_ASYM_GRAD, oracle.CLIP_ASYM_ENTRY], [0, 1], [0, 1])))
def test_8x6_rank2_brute_force(clip, norm_p, norm_q):
    g = read_golden("rank2_8x6.txt")
    m, n, k = 8, 6, 2
    F = Fraction
    Pt = np.array(g["P_true"]).reshape(m, k); Qt = np.array(g["Q_true"]).reshape(n, k)
    P0 = np.array(g["P0"]).reshape(m, k); Q0 = np.array(g["Q0"]).reshape(n, k)
    mask = np.array(g["mask"], dtype=int).reshape(m, n)
    noise = np.array(g["noise"]).reshape(m, n)
    R = Pt @ Qt.T + noise           # small dyadic rationals: exact in float32
    rows, cols = np.nonzero(mask)
    order = np.array(g["order"], dtype=int)        # a fixed shuffle of the entries
    rows, cols = rows[order].astype(np.int32), cols[order].astype(np.int32)
    vals = R[rows, cols].astype(np.float32)
    assert np.array_equal(vals.astype(np.float64), R[rows, cols])
    eta, lam, xi = F(1, 16), F(1, 32), F(1, 2)
    fr = lambda A: [[F(float(x)) for x in row] for row in A]
    GP, GQ, P1, Q1, sse = _brute_force_dense(m, n, k, mask.tolist(), fr(R), fr(P0), fr(Q0),
                                             eta, lam, xi, clip, norm_p, norm_q)
    st = oracle.grad_step(m, n, k, rows, cols, vals, P0, Q0, float(eta), float(lam), float(xi),
                          clip, norm_p, norm_q)
    tof = lambda A: np.array([[float(x) for x in row] for row in A])
    np.testing.assert_allclose(st.GP, tof(GP), rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(st.GQ, tof(GQ), rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(st.P, tof(P1).astype(np.float32), rtol=0, atol=1e-7)
    np.testing.assert_allclose(st.Q, tof(Q1).astype(np.float32), rtol=0, atol=1e-7)
    sse_o, _ = oracle.loss(m, n, k, rows, cols, vals, P0, Q0, float(lam))
    assert abs(sse_o - float(sse)) < 1e-12
    # the clip must actually bite in this example, on both sides
    if clip == oracle.CLIP_ASYM_STEP:
        assert (st.DP == float(xi)).any() and (st.DQ == float(xi)).any()


# ---------------------------------------------------------------- closed forms and invariants
def _random_instance(m, n, k, nnz, seed, integer=False):
    rng = np.random.default_rng(seed)
    ids = rng.choice(m * n, size=nnz, replace=False)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    if integer:
        P = rng.integers(-3, 4, (m, k)).astype(np.float32)
        Q = rng.integers(-3, 4, (n, k)).astype(np.float32)
    else:
        P = rng.standard_normal((m, k)).astype(np.float32) * 0.5
        Q = rng.standard_normal((n, k)).astype(np.float32) * 0.5
    vals = rng.standard_normal(nnz).astype(np.float32)
    return rows, cols, vals, P, Q


def test_zero_gradient_at_true_factors():
    """Exactly low-rank noiseless data (the paper's synthetic recipe, Sec. 6.1): e = 0, G = 0."""
    m, n, k, nnz = 40, 30, 4, 500
    rows, cols, _, P, Q = _random_instance(m, n, k, nnz, 1, integer=True)
    vals = np.sum(P[rows].astype(np.float64) * Q[cols], axis=1).astype(np.float32)
    assert not np.any(oracle.residuals(m, n, k, rows, cols, vals, P, Q))
    for norm in (0, 1):
        st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.3, 0.0, 0.1,
                              oracle.CLIP_ASYM_STEP, norm, norm)
        assert not np.any(st.GP) and not np.any(st.GQ)
        assert np.array_equal(st.P, P) and np.array_equal(st.Q, Q)
    assert oracle.loss(m, n, k, rows, cols, vals, P, Q, 0.0) == (0.0, 0.0)


def test_finite_differences_of_the_objective():
    """-D (norm NONE, no clip) is the gradient of Eq. (rmf-obj): central differences in double."""
    m, n, k, nnz = 25, 18, 5, 200
    rows, cols, vals, P, Q = _random_instance(m, n, k, nnz, 2)
    lam = 0.07
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.01, lam, 0.1)

    def obj(Pd, Qd):   # independent dense statement of the objective, in double
        M = np.zeros((m, n)); M[rows, cols] = 1
        Rd = np.zeros((m, n)); Rd[rows, cols] = vals
        return np.sum(M * (Rd - Pd @ Qd.T) ** 2) + lam * (np.sum(Pd ** 2) + np.sum(Qd ** 2))

    Pd, Qd = P.astype(np.float64), Q.astype(np.float64)
    assert abs(obj(Pd, Qd) - oracle.loss(m, n, k, rows, cols, vals, P, Q, lam)[1]) < 1e-9
    h = 1e-5
    rng = np.random.default_rng(3)
    for _ in range(40):
        i, l = rng.integers(m), rng.integers(k)
        Pp, Pm = Pd.copy(), Pd.copy(); Pp[i, l] += h; Pm[i, l] -= h
        fd = (obj(Pp, Qd) - obj(Pm, Qd)) / (2 * h)
        assert abs(fd + st.DP[i, l]) <= 1e-6 * max(1.0, abs(fd))
        j, l = rng.integers(n), rng.integers(k)
        Qp, Qm = Qd.copy(), Qd.copy(); Qp[j, l] += h; Qm[j, l] -= h
        fd = (obj(Pd, Qp) - obj(Pd, Qm)) / (2 * h)
        assert abs(fd + st.DQ[j, l]) <= 1e-6 * max(1.0, abs(fd))


def test_count_mode_is_gradient_of_weighted_objective():
    """With norm COUNT, -s_i D_i is the gradient of SSE + lam (sum_i s_i |p_i|^2 + sum_j s_j |q_j|^2)."""
    m, n, k, nnz = 12, 9, 3, 60
    rows, cols, vals, P, Q = _random_instance(m, n, k, nnz, 4)
    lam = 0.05
    sP = np.maximum(1, np.bincount(rows, minlength=m)); sQ = np.maximum(1, np.bincount(cols, minlength=n))
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.01, lam, 0.1, 0, 1, 1)

    def obj(Pd, Qd):
        e = vals - np.sum(Pd[rows] * Qd[cols], axis=1)
        return np.sum(e ** 2) + lam * (np.sum(sP[:, None] * Pd ** 2) + np.sum(sQ[:, None] * Qd ** 2))

    Pd, Qd = P.astype(np.float64), Q.astype(np.float64)
    h = 1e-5
    for i in range(m):
        Pp, Pm = Pd.copy(), Pd.copy(); Pp[i, 1] += h; Pm[i, 1] -= h
        fd = (obj(Pp, Qd) - obj(Pm, Qd)) / (2 * h)
        assert abs(fd + sP[i] * st.DP[i, 1]) <= 1e-6 * max(1.0, abs(fd))
    for j in range(n):
        Qp, Qm = Qd.copy(), Qd.copy(); Qp[j, 2] += h; Qm[j, 2] -= h
        fd = (obj(Pd, Qp) - obj(Pd, Qm)) / (2 * h)
        assert abs(fd + sQ[j] * st.DQ[j, 2]) <= 1e-6 * max(1.0, abs(fd))


def test_dense_special_case_matches_matrix_products():
    """Omega = every cell: G_P = (R - P Q^T) Q and G_Q = (R - P Q^T)^T P (numpy, double)."""
    m, n, k = 17, 13, 6
    rng = np.random.default_rng(5)
    P = rng.standard_normal((m, k)).astype(np.float32); Q = rng.standard_normal((n, k)).astype(np.float32)
    R = rng.standard_normal((m, n)).astype(np.float32)
    ids = rng.permutation(m * n)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    vals = R[rows, cols]
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.01, 0.0, 0.1)
    E = R.astype(np.float64) - P.astype(np.float64) @ Q.astype(np.float64).T
    np.testing.assert_allclose(st.GP, E @ Q, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(st.GQ, E.T @ P, rtol=1e-12, atol=1e-12)
    assert abs(oracle.loss(m, n, k, rows, cols, vals, P, Q, 0.0)[0] - np.sum(E ** 2)) < 1e-9
    # a transposed operand would fail here: m != n and P, Q are not symmetric in any way
    np.testing.assert_allclose(oracle.residuals(m, n, k, rows, cols, vals, P, Q), E[rows, cols],
                               rtol=1e-12, atol=1e-12)


def test_trace_identity_and_single_entry():
    m, n, k, nnz = 60, 45, 8, 900
    rows, cols, vals, P, Q = _random_instance(m, n, k, nnz, 6)
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.01, 0.0, 0.1)
    e = oracle.residuals(m, n, k, rows, cols, vals, P, Q)
    pq = np.sum(P[rows].astype(np.float64) * Q[cols], axis=1)
    t = np.sum(e * pq)
    assert abs(np.sum(st.GP * P) - t) < 1e-9 and abs(np.sum(st.GQ * Q) - t) < 1e-9
    # one observed entry: only one row of each gradient is non-zero
    i, j, r = 7, 11, np.float32(1.75)
    st = oracle.grad_step(m, n, k, [i], [j], [r], P, Q, 0.01, 0.0, 0.1)
    e1 = float(r) - float(P[i].astype(np.float64) @ Q[j].astype(np.float64))
    np.testing.assert_allclose(st.GP[i], e1 * Q[j].astype(np.float64), rtol=1e-14)
    np.testing.assert_allclose(st.GQ[j], e1 * P[i].astype(np.float64), rtol=1e-14)
    assert not np.any(np.delete(st.GP, i, axis=0)) and not np.any(np.delete(st.GQ, j, axis=0))
    # an empty template: pure decay of both factors
    st = oracle.grad_step(m, n, k, [], [], [], P, Q, 0.1, 0.5, 0.1, 0, 1, 1)
    np.testing.assert_allclose(st.P, P * (1 - 0.1), rtol=1e-6)


def test_scaling_invariance():
    """lambda = 0: residuals are invariant under (P, Q) -> (cP, Q/c); G_P -> G_P/c, G_Q -> c G_Q."""
    m, n, k, nnz = 30, 20, 4, 250
    rows, cols, vals, P, Q = _random_instance(m, n, k, nnz, 7)
    c = 4.0   # a power of two: the scaling is exact in floating point
    a = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.01, 0.0, 0.1)
    b = oracle.grad_step(m, n, k, rows, cols, vals, P * c, Q / c, 0.01, 0.0, 0.1)
    np.testing.assert_allclose(b.GP, a.GP / c, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(b.GQ, a.GQ * c, rtol=1e-13, atol=1e-13)


def test_clip_closed_form_and_bound():
    """Sec. 5.3: the nested min/max equals min(g, xi) for xi > 0; increases are capped at eta*xi."""
    for xi in (0.1, 2.0, 1e-3):
        for gval in np.concatenate([np.linspace(-10, 10, 401), [xi, -xi, 0.0, 1e30, -1e30]]):
            assert oracle.clip_nested(float(gval), xi) == min(float(gval), xi)
    m, n, k, nnz = 30, 20, 4, 250
    rows, cols, vals, P, Q = _random_instance(m, n, k, nnz, 8)
    eta, xi = 0.05, 0.1
    st = oracle.grad_step(m, n, k, rows, cols, vals, P * 3, Q * 3, eta, 0.03, xi, oracle.CLIP_ASYM_STEP, 1, 1)
    assert (st.P.astype(np.float64) - 3 * P).max() <= eta * xi + 1e-6
    assert (st.Q.astype(np.float64) - 3 * Q).max() <= eta * xi + 1e-6
    assert (st.DP <= xi).all() and (st.DP == xi).any() and (st.DP < -xi).any()
    un = oracle.grad_step(m, n, k, rows, cols, vals, P * 3, Q * 3, eta, 0.03, xi, oracle.CLIP_NONE, 1, 1)
    assert np.array_equal(st.DP, np.minimum(un.DP, xi)) and np.array_equal(st.DQ, np.minimum(un.DQ, xi))
    gr = oracle.grad_step(m, n, k, rows, cols, vals, P * 3, Q * 3, eta, 0.03, xi, oracle.CLIP_ASYM_GRAD, 1, 1)
    assert np.array_equal(gr.DP, np.maximum(un.DP, -xi))


def test_monotone_loss_at_small_step():
    m, n, k, nnz = 200, 150, 8, 6000
    rng = np.random.default_rng(9)
    ids = rng.choice(m * n, nnz, replace=False)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    s = k ** -0.25
    Pt, Qt = rng.standard_normal((m, k)) * s, rng.standard_normal((n, k)) * s
    vals = (np.sum(Pt[rows] * Qt[cols], axis=1) + 0.01 * rng.standard_normal(nnz)).astype(np.float32)
    P0 = (rng.standard_normal((m, k)) * s).astype(np.float32)
    Q0 = (rng.standard_normal((n, k)) * s).astype(np.float32)
    for clip in (oracle.CLIP_NONE, oracle.CLIP_ASYM_STEP):
        _, _, hist = oracle.fit(m, n, k, rows, cols, vals, P0, Q0, 30, 0.005, 0.0, 0.1, clip, 0, 0)
        assert np.all(np.diff(hist) < 0), hist
    _, _, hist = oracle.fit(m, n, k, rows, cols, vals, P0, Q0, 30, 0.2, 0.0, 0.1, oracle.CLIP_NONE, 1, 1)
    assert np.all(np.diff(hist) < 0), hist
    # fit is `epochs` applications of grad_step
    P2, Q2, _ = oracle.fit(m, n, k, rows, cols, vals, P0, Q0, 2, 0.01, 0.02, 0.1, 1, 1, 0)
    a = oracle.grad_step(m, n, k, rows, cols, vals, P0, Q0, 0.01, 0.02, 0.1, 1, 1, 0)
    b = oracle.grad_step(m, n, k, rows, cols, vals, a.P, a.Q, 0.01, 0.02, 0.1, 1, 1, 0)
    assert np.array_equal(P2, b.P) and np.array_equal(Q2, b.Q)


# ---------------------------------------------------------------- bf16 rounding and emulation switch
def test_bf16_round_table():
    with open(__import__("os").path.join(__import__("conftest").ROOT, "tests", "golden", "bf16_rne.txt")) as f:
        rowsf = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rowsf) >= 12
    for a, b in rowsf:
        x = struct.unpack("<f", struct.pack("<I", int(a, 16)))[0]
        y = oracle.bf16_round(x)
        got = struct.unpack("<I", struct.pack("<f", y))[0]
        assert got == int(b, 16) << 16, (a, b, hex(got))


def test_bf16_emulation_rounds_inputs_only():
    m, n, k, nnz = 30, 20, 8, 300
    rows, cols, vals, P, Q = _random_instance(m, n, k, nnz, 10)
    import torch
    Pb = torch.from_numpy(P).to(torch.bfloat16).to(torch.float32).numpy()   # library RNE rounding
    Qb = torch.from_numpy(Q).to(torch.bfloat16).to(torch.float32).numpy()
    a = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.05, 0.03, 0.1, 1, 1, 1, bf16_emulate=True)
    b = oracle.grad_step(m, n, k, rows, cols, vals, Pb, Qb, 0.05, 0.03, 0.1, 1, 1, 1)
    assert np.array_equal(a.GP, b.GP) and np.array_equal(a.GQ, b.GQ)
    # the regulariser and the update keep the fp32 master values
    s = np.maximum(1, np.bincount(rows, minlength=m))[:, None]
    D = np.minimum(2 * a.GP / s - 2 * 0.03 * P.astype(np.float64), 0.1)
    np.testing.assert_allclose(a.P, (P + 0.05 * D).astype(np.float32), rtol=0, atol=1e-7)
    e = oracle.residuals(m, n, k, rows, cols, vals, P, Q, bf16_emulate=True)
    np.testing.assert_allclose(e, vals - np.sum(Pb[rows].astype(np.float64) * Qb[cols], axis=1), atol=1e-12)


def test_fp16_round_table_and_library_cast():
    with open(__import__("os").path.join(__import__("conftest").ROOT, "tests", "golden", "fp16_rne.txt")) as f:
        rowsf = [l.split("#")[0].split() for l in f if l.split("#")[0].strip()]
    assert len(rowsf) >= 15
    for a, b in rowsf:
        x = struct.unpack("<f", struct.pack("<I", int(a, 16)))[0]
        got = struct.unpack("<I", struct.pack("<f", oracle.fp16_round(x)))[0]
        assert got == int(b, 16), (a, b, hex(got))
    # and a library's round-to-nearest-even cast on random values over the whole range of a rating matrix
    rng = np.random.default_rng(3)
    xs = np.concatenate([rng.normal(0, 3, 2000), rng.uniform(-70000, 70000, 200), rng.normal(0, 1e-6, 200)]).astype(np.float32)
    with np.errstate(over="ignore"):
        ref = xs.astype(np.float16).astype(np.float32)
    got = np.array([oracle.fp16_round(float(x)) for x in xs], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


def test_tensor_core_emulation_level(golden_3x2):
    """Level 2 of the emulation switch: r -> binary16, e -> bfloat16 before the gradient products, factors -> bfloat16.
    A hand-worked value where each rounding decides the result, then dense algebra with library casts."""
    g = golden_3x2
    m, n, k, rows, cols, _, P, Q = _inst(g)
    vals = _arr(g, "vals_tensor", dtype=np.float32)
    e = oracle.residuals(m, n, k, rows, cols, vals, P, Q, bf16_emulate=oracle.EMU_TENSOR)
    assert np.array_equal(e, _arr(g, "e_tensor"))
    st = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.1, 0.25, 2.0, bf16_emulate=oracle.EMU_TENSOR)
    assert np.array_equal(st.GP, _arr(g, "GP_tensor", (m, k))) and np.array_equal(st.GQ, _arr(g, "GQ_tensor", (n, k)))
    lvl1 = oracle.grad_step(m, n, k, rows, cols, vals, P, Q, 0.1, 0.25, 2.0, bf16_emulate=True)
    assert not np.array_equal(lvl1.GP, st.GP)
    # random instance: E = mask .* bf16(fp16(R) - Pb Qb^T) by numpy on the dense matrix, then two dense products
    import torch
    m2, n2, k2, nnz = 37, 29, 16, 500
    rows, cols, vals, P2, Q2 = _random_instance(m2, n2, k2, nnz, 21)
    vals = (vals * 3).astype(np.float32)
    Pb = torch.from_numpy(P2).to(torch.bfloat16).to(torch.float64).numpy()
    Qb = torch.from_numpy(Q2).to(torch.bfloat16).to(torch.float64).numpy()
    R16 = np.zeros((m2, n2)); M = np.zeros((m2, n2))
    R16[rows, cols] = torch.from_numpy(vals).to(torch.float16).to(torch.float64).numpy(); M[rows, cols] = 1
    E = torch.from_numpy(((R16 - Pb @ Qb.T) * M).astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    st = oracle.grad_step(m2, n2, k2, rows, cols, vals, P2, Q2, 0.05, 0.03, 0.1, 1, 1, 1, bf16_emulate=oracle.EMU_TENSOR)
    np.testing.assert_allclose(st.GP, E @ Qb, rtol=0, atol=1e-12)
    np.testing.assert_allclose(st.GQ, E.T @ Pb, rtol=0, atol=1e-12)
    assert np.max(np.abs(st.GP - oracle.grad_step(m2, n2, k2, rows, cols, vals, P2, Q2, 0.05, 0.03, 0.1, 1, 1, 1,
                                                  bf16_emulate=True).GP)) > 1e-4      # the level is not a no-op
    # the update still starts from the fp32 master and regularises with it
    s = np.maximum(1, np.bincount(rows, minlength=m2))[:, None]
    D = np.minimum(2 * st.GP / s - 2 * 0.03 * P2.astype(np.float64), 0.1)
    np.testing.assert_allclose(st.P, (P2 + 0.05 * D).astype(np.float32), rtol=0, atol=1e-7)


# ---------------------------------------------------------------- layout
@pytest.mark.parametrize("m,n,nnz,seed", [(50, 40, 600, 1), (1, 70, 33, 2), (64, 1, 20, 3), (9, 9, 81, 4), (5, 5, 0, 5)])
def test_layout_against_lexsort_and_invariants(m, n, nnz, seed):
    rng = np.random.default_rng(seed)
    ids = rng.choice(m * n, nnz, replace=False)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    vals = rng.standard_normal(nnz).astype(np.float32)
    lay = oracle.layout(m, n, rows, cols, vals)
    o = np.lexsort((cols, rows))      # library sort: primary rows, secondary cols
    assert np.array_equal(lay.col_idx, cols[o]) and np.array_equal(lay.val_csr, vals[o])
    assert np.array_equal(lay.row_ptr, np.concatenate([[0], np.cumsum(np.bincount(rows, minlength=m))]))
    oc = np.lexsort((rows, cols))
    assert np.array_equal(lay.row_idx, rows[oc]) and np.array_equal(lay.val_csc, vals[oc])
    assert np.array_equal(lay.col_ptr, np.concatenate([[0], np.cumsum(np.bincount(cols, minlength=n))]))
    assert np.array_equal(np.sort(lay.perm), np.arange(nnz))
    assert np.array_equal(lay.val_csc, lay.val_csr[lay.perm])
    csr_rows = np.repeat(np.arange(m), np.diff(lay.row_ptr))
    assert np.array_equal(csr_rows[lay.perm], lay.row_idx)
    assert np.array_equal(lay.col_idx[lay.perm], np.repeat(np.arange(n), np.diff(lay.col_ptr)))


def test_layout_duplicates_break_ties_by_input_position():
    rows = np.array([1, 0, 1, 1], np.int32); cols = np.array([2, 0, 2, 1], np.int32)
    vals = np.array([10, 20, 30, 40], np.float32)
    lay = oracle.layout(2, 3, rows, cols, vals)
    assert lay.val_csr.tolist() == [20, 40, 10, 30] and lay.val_csc.tolist() == [20, 40, 10, 30]
