"""Pins of the Stage II oracle (Sec. 5.2, Eq. 10 with Adam) against the mathematics and a library optimiser."""
import numpy as np
import torch

import oracle


def _problem(m=30, d=7, k=3, ncols=5, seed=0, density=0.6):
    rng = np.random.default_rng(seed)
    P = rng.standard_normal((m, k)).astype(np.float32) * 0.7
    Q = rng.standard_normal((d, k)).astype(np.float32) * 0.7
    cols = []
    for j in range(ncols):
        r = np.nonzero(rng.random(m) < density)[0]
        cols.append(r if j != 2 else r[:0])          # column 2 has no observation
    col_ptr = np.concatenate([[0], np.cumsum([len(c) for c in cols])]).astype(np.int64)
    row_idx = np.concatenate(cols).astype(np.int32)
    vals = rng.standard_normal(len(row_idx)).astype(np.float32)
    return m, d, k, col_ptr, row_idx, vals, P, Q


def _loss_col(Rhat, rows, r, c, lam):
    e = r - Rhat[rows] @ c
    return float(e @ e + lam * c @ c)


def test_first_adam_step_has_magnitude_eta_and_sign_of_minus_gradient():
    """Textbook property of Adam with bias correction: the first step is -eta g / (|g| + eps)."""
    m, d, k, cp, ri, v, P, Q = _problem()
    Rhat = P.astype(np.float64) @ Q.astype(np.float64).T
    C, _ = oracle.extend(m, d, k, cp, ri, v, P, Q, eta=0.05, lam=0.1, iters=1)
    for j in range(len(cp) - 1):
        rows, r = ri[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]].astype(np.float64)
        g = -2 * Rhat[rows].T @ r                      # gradient of Eq. 10 at C = 0
        np.testing.assert_allclose(C[j], -0.05 * g / (np.abs(g) + 1e-8), rtol=1e-12, atol=1e-15)
    assert not C[2].any()                               # no observation, C = 0, gradient 0: stays 0


def test_matches_torch_adam_on_the_same_objective():
    """Special case that reduces to a library routine: torch.optim.Adam on Eq. 10 built with autograd."""
    m, d, k, cp, ri, v, P, Q = _problem(seed=3)
    eta, lam, iters = 0.03, 0.05, 25
    C, sse = oracle.extend(m, d, k, cp, ri, v, P, Q, eta, lam, iters)
    Rhat = torch.tensor(P, dtype=torch.float64) @ torch.tensor(Q, dtype=torch.float64).T
    Ct = torch.zeros(len(cp) - 1, d, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([Ct], lr=eta, betas=(0.9, 0.999), eps=1e-8)
    colof = np.repeat(np.arange(len(cp) - 1), np.diff(cp))
    rows_t, cols_t = torch.tensor(ri, dtype=torch.long), torch.tensor(colof, dtype=torch.long)
    r_t = torch.tensor(v, dtype=torch.float64)
    for _ in range(iters):
        opt.zero_grad()
        pred = (Rhat[rows_t] * Ct[cols_t]).sum(dim=1)
        loss = ((r_t - pred) ** 2).sum() + lam * (Ct ** 2).sum()
        loss.backward()
        opt.step()
    np.testing.assert_allclose(C, Ct.detach().numpy(), rtol=1e-9, atol=1e-12)
    pred = (Rhat[rows_t] * Ct.detach()[cols_t]).sum(dim=1)
    assert abs(sse - float(((r_t - pred) ** 2).sum())) < 1e-9


def test_converges_to_the_ridge_solution_and_loss_decreases():
    m, d, k, cp, ri, v, P, Q = _problem(m=60, d=3, k=3, ncols=4, seed=5, density=0.9)
    Rhat = P.astype(np.float64) @ Q.astype(np.float64).T
    lam = 0.2
    C, _ = oracle.extend(m, d, k, cp, ri, v, P, Q, eta=0.02, lam=lam, iters=3000)
    prev = None
    for j in (0, 1, 3):
        rows, r = ri[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]].astype(np.float64)
        A = Rhat[rows]
        star = np.linalg.solve(A.T @ A + lam * np.eye(d), A.T @ r)      # closed form of the regularised LS
        np.testing.assert_allclose(C[j], star, atol=2e-3)
        l0 = _loss_col(Rhat, rows, r, np.zeros(d), lam)
        l1 = _loss_col(Rhat, rows, r, oracle.extend(m, d, k, cp, ri, v, P, Q, 0.02, lam, 50)[0][j], lam)
        assert l1 < l0


def test_columns_are_independent_and_warm_start_continues():
    """Chunking cannot change the result: a column alone gives the same coefficients as in the full call."""
    m, d, k, cp, ri, v, P, Q = _problem(seed=7)
    C, sse = oracle.extend(m, d, k, cp, ri, v, P, Q, 0.04, 0.1, 12)
    tot = 0.0
    for j in range(len(cp) - 1):
        cpj = np.array([0, cp[j + 1] - cp[j]], dtype=np.int64)
        Cj, sj = oracle.extend(m, d, k, cpj, ri[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]], P, Q, 0.04, 0.1, 12)
        assert np.array_equal(Cj[0], C[j])
        tot += sj
    assert abs(tot - sse) < 1e-9
    # gradient of Eq. 10 by finite differences through a single tiny-step probe: one Adam step from C0
    # moves against the sign of dL/dC evaluated at C0
    C0 = np.random.default_rng(1).standard_normal(C.shape) * 0.3
    C1, _ = oracle.extend(m, d, k, cp, ri, v, P, Q, 1e-3, 0.1, 1, C0=C0)
    Rhat = P.astype(np.float64) @ Q.astype(np.float64).T
    h = 1e-6
    for j in (0, 1, 4):
        rows, r = ri[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]].astype(np.float64)
        for a in range(d):
            cp_, cm_ = C0[j].copy(), C0[j].copy(); cp_[a] += h; cm_[a] -= h
            fd = (_loss_col(Rhat, rows, r, cp_, 0.1) - _loss_col(Rhat, rows, r, cm_, 0.1)) / (2 * h)
            step = C1[j, a] - C0[j, a]
            np.testing.assert_allclose(step, -1e-3 * fd / (abs(fd) + 1e-8), rtol=1e-5, atol=1e-12)


def test_mixed_precision_form_is_the_same_iteration_and_rounds_only_the_product_operands():
    """orc_extend_mixed: without rounding it is orc_extend re-associated (pinned above against torch's Adam); with
    rounding, the two places where a bfloat16 value enters are checked by dense algebra with a library's casts."""
    m, d, k, cp, ri, v, P, Q = _problem(m=40, d=9, k=4, ncols=6, seed=5)
    rng = np.random.default_rng(1)
    C0 = (rng.standard_normal((len(cp) - 1, d)) * 0.3).astype(np.float32)
    for c0 in (None, C0):
        a, sa = oracle.extend(m, d, k, cp, ri, v, P, Q, 0.03, 0.05, 12, C0=c0)
        b, sb = oracle.extend_mixed(m, d, k, cp, ri, v, P, Q, 0.03, 0.05, 12, C0=c0, round_operands=False)
        np.testing.assert_allclose(b, a, rtol=1e-9, atol=1e-12)
        assert abs(sa - sb) <= 1e-9 * sa

    def bf(x):
        return torch.tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    Qb, Pd = bf(Q), P.astype(np.float64)
    # one step with eps so large that the step is -eta g / eps: reads off the gradient, from a warm start
    eta, lam, eps = 1.0, 0.05, 1e6
    C1, _ = oracle.extend_mixed(m, d, k, cp, ri, v, P, Q, eta, lam, 1, C0=C0, eps=eps)
    for j in range(len(cp) - 1):
        rows, r = ri[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]].astype(np.float64)
        W = Qb.T @ bf(C0[j])                               # first product: both operands rounded
        e = r - Pd[rows] @ W                               # residuals in full precision
        U = Pd[rows].T @ e
        g = -2 * Qb @ bf(U) + 2 * lam * C0[j].astype(np.float64)    # second product: both operands rounded, C itself not
        np.testing.assert_allclose(C1[j] - C0[j], -eta * g / (np.abs(g) + eps), rtol=1e-9, atol=1e-15)
    # and the rounding is not a no-op on these inputs
    C1f, _ = oracle.extend_mixed(m, d, k, cp, ri, v, P, Q, eta, lam, 1, C0=C0, eps=eps, round_operands=False)
    assert np.max(np.abs(C1f - C1)) > 1e-3 * np.max(np.abs(C1 - C0))
    # the SSE it reports is that of the rounded first product at the returned coefficients
    C2, sse = oracle.extend_mixed(m, d, k, cp, ri, v, P, Q, 0.03, lam, 5)
    tot = 0.0
    for j in range(len(cp) - 1):
        rows, r = ri[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]].astype(np.float64)
        tot += float(np.sum((r - Pd[rows] @ (Qb.T @ bf(C2[j]))) ** 2))
    assert abs(tot - sse) <= 1e-9 * sse
