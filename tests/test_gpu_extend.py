"""Stage II extension (Sec. 5.2, Eq. 10 + Adam): CUDA path against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr
from paper_2608_00977_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _problem(m, d, k, ncols, per_col, seed, hot=None):
    rng = np.random.default_rng(seed)
    P = (rng.standard_normal((m, k)) * k ** -0.25).astype(np.float32)
    Q = (rng.standard_normal((d, k)) * k ** -0.25).astype(np.float32)
    cols = []
    for j in range(ncols):
        cnt = per_col if hot is None or j not in hot else hot[j]
        cnt = min(m, int(rng.integers(max(0, cnt - cnt // 2), cnt + cnt // 2 + 1)))
        cols.append(np.sort(rng.choice(m, cnt, replace=False)))
    cols[min(3, ncols - 1)] = cols[0][:0]                      # one column without observations
    col_ptr = np.concatenate([[0], np.cumsum([len(c) for c in cols])]).astype(np.int64)
    row_idx = np.concatenate(cols).astype(np.int32)
    vals = (rng.standard_normal(len(row_idx)) * 1.5).astype(np.float32)
    return P, Q, col_ptr, row_idx, vals


def _run_gpu(P, Q, cp, ri, v, chunk, iters, eta, lam, C0=None):
    ncols, d = len(cp) - 1, Q.shape[0]
    Ch = torch.zeros(ncols, d) if C0 is None else torch.tensor(C0, dtype=torch.float32)
    Ch = Ch.pin_memory()
    sse = B.tsid_extend(torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV), torch.tensor(cp).pin_memory(),
                        torch.tensor(ri).pin_memory(), torch.tensor(v).pin_memory(), Ch, chunk, iters, eta, lam,
                        want_sse=True)
    return Ch.numpy().copy(), sse


@pytest.mark.parametrize("m,d,k,ncols,per_col,chunk", [(500, 96, 32, 300, 60, 64), (300, 40, 16, 130, 30, 1000),
                                                       (800, 200, 64, 257, 80, 100), (64, 8, 4, 5, 10, 2)])
def test_extend_matches_oracle(m, d, k, ncols, per_col, chunk):
    P, Q, cp, ri, v = _problem(m, d, k, ncols, per_col, seed=m + d)
    eta, lam, iters = 0.02, 0.05, 15
    C, sse = _run_gpu(P, Q, cp, ri, v, chunk, iters, eta, lam)
    Cr, sse_r = oracle.extend(m, d, k, cp, ri, v, P, Q, eta, lam, iters)
    assert relerr(C, Cr) <= 2e-3, relerr(C, Cr)     # Adam divides by sqrt(v): fp32 noise on tiny gradients is amplified
    assert abs(sse - sse_r) / sse_r <= 1e-3
    assert not C[min(3, ncols - 1)].any()


def test_extend_random_shapes_by_conditioning_free_measures():
    """A seeded sweep over shapes, chunk widths, step counts and warm starts.  A coefficient whose gradient
    q_t . U_j nearly cancels has no stable digits in fp32 (each step's rounding of U changes it by ~1e-3 of
    itself, and Adam turns that ratio error into ~1e-3 of a step; an exactly cancelling one can step the other
    way), so the bound on max |C - C_ref| holds for all but a few coordinates in ten thousand; what the fit
    itself fixes is compared tightly: the SSE, and C in the root mean square."""
    rng = np.random.default_rng(2024)
    checked = bad = total = 0
    for _ in range(60):
        k = int(rng.choice([4, 8, 16, 32, 64, 128])); m = int(rng.choice([1, 5, 64, 300, 1000]))
        d = int(rng.choice([1, 3, 8, 40, 96, 128, 200, 520])); ncols = int(rng.choice([1, 2, 5, 130, 257]))
        per = int(rng.choice([0, 1, 3, 30, 200]))
        P = (rng.standard_normal((m, k)) * k ** -0.25).astype(np.float32)
        Q = (rng.standard_normal((d, k)) * k ** -0.25).astype(np.float32)
        cols = [np.sort(rng.choice(m, min(m, int(rng.integers(0, 2 * per + 1))), replace=False)) for _ in range(ncols)]
        cp = np.concatenate([[0], np.cumsum([len(c) for c in cols])]).astype(np.int64)
        ri = np.concatenate(cols).astype(np.int32)
        v = (rng.standard_normal(len(ri)) * 1.5).astype(np.float32)
        chunk = int(rng.choice([1, 2, 7, 64, 1000])); iters = int(rng.choice([1, 3, 10])); lam = float(rng.choice([0.0, 0.05]))
        C0 = (rng.standard_normal((ncols, d)) * 0.1).astype(np.float32) if rng.random() < 0.3 else None
        C, sse = _run_gpu(P, Q, cp, ri, v, chunk, iters, 0.02, lam, C0=C0)
        Cr, sse_r = oracle.extend(m, d, k, cp, ri, v, P, Q, 0.02, lam, iters, C0=C0)
        assert abs(sse - sse_r) <= 1e-4 * max(sse_r, 1e-12), (m, d, k, ncols, per, chunk, iters)
        scale = max(float(np.abs(Cr).max()), 1e-12)
        err = np.abs(C - Cr)
        assert float(np.sqrt(np.mean(err ** 2))) <= 1e-3 * scale, (m, d, k, ncols, per, chunk, iters)
        bad += int((err > 2e-3 * scale).sum()); total += err.size; checked += 1
    assert checked == 60 and bad <= max(3, total // 2000), (bad, total)


def test_extend_chunking_is_invisible_and_loss_decreases():
    P, Q, cp, ri, v = _problem(1200, 64, 32, 400, 2500 // 8, seed=9, hot={7: 1200, 100: 1100})   # split columns
    outs = [_run_gpu(P, Q, cp, ri, v, chunk, 10, 0.02, 0.05) for chunk in (400, 64, 7)]
    for C, sse in outs[1:]:
        assert np.array_equal(C, outs[0][0])             # bitwise: columns are independent
        assert abs(sse - outs[0][1]) <= 1e-12 * sse      # chunk totals are added in a different order
    sse0 = float(np.sum(v.astype(np.float64) ** 2))                            # C = 0 predicts 0
    assert outs[0][1] < 0.95 * sse0
    # warm start: 6 + 4 steps is not the same as 10 (Adam's moments restart), but it keeps descending
    C6, s6 = _run_gpu(P, Q, cp, ri, v, 64, 6, 0.02, 0.05)
    C10, s10 = _run_gpu(P, Q, cp, ri, v, 64, 4, 0.02, 0.05, C0=C6)
    assert s10 < s6


def test_extend_cold_start_ignores_host_contents():
    P, Q, cp, ri, v = _problem(300, 40, 16, 130, 30, seed=4)
    ref, _ = _run_gpu(P, Q, cp, ri, v, 50, 8, 0.02, 0.05)
    Ch = torch.full((130, 40), 7.0).pin_memory()
    B.tsid_extend(torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV), torch.tensor(cp).pin_memory(),
                  torch.tensor(ri).pin_memory(), torch.tensor(v).pin_memory(), Ch, 50, 8, 0.02, 0.05, cold_start=True)
    assert np.array_equal(Ch.numpy(), ref)


def test_extend_errors():
    P, Q, cp, ri, v = _problem(64, 8, 4, 5, 10, seed=1)
    bad = ri.copy(); bad[3] = 64
    with pytest.raises(B.TsidError) as e:
        _run_gpu(P, Q, cp, bad, v, 2, 3, 0.02, 0.05)
    assert e.value.status == B.TSID_ERR_INDEX_RANGE
    cfg = B.TsidExtendConfig(64, 8, 6, 5, 2, 3, 0.02, 0.05, 0.9, 0.999, 1e-8, 0, None, None, 0)
    import ctypes as C
    need = C.c_size_t(0)
    assert B.lib().tsid_extend_workspace_bytes(C.byref(cfg), torch.tensor(cp).data_ptr(), C.byref(need)) == B.TSID_ERR_UNSUPPORTED


@pytest.mark.parametrize("m,d,k,ncols,per_col,chunk", [(800, 200, 64, 257, 80, 100), (600, 264, 128, 300, 70, 150),
                                                       (900, 1032, 64, 700, 90, 333)])
def test_extend_tensor_core_form(m, d, k, ncols, per_col, chunk):
    """TSID_EXTEND_TC: the gradient product on the tensor cores with bf16 operands (the paper's mixed
    precision).  Adam turns a gradient coordinate into a step of about +-eta whatever its size, so where the
    gradient is smaller than bf16's rounding the two precisions may step in opposite directions: the
    coefficients are compared in the mean, the fit exactly, and the product itself through a run whose eps
    is so large that the step is proportional to the gradient."""
    P, Q, cp, ri, v = _problem(m, d, k, ncols, per_col, seed=m + d + k)
    args = (torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV), torch.tensor(cp).pin_memory(),
            torch.tensor(ri).pin_memory(), torch.tensor(v).pin_memory())
    Ch = torch.zeros(ncols, d).pin_memory()
    # (1) eps = 1e4 >> |g|: one step from C = 0 gives C = -eta g / eps up to 1e-4 relative: the product itself
    B.tsid_extend(*args, Ch, chunk, 1, 1.0, 0.05, eps=1e4, tensor_cores=True)
    Cr, _ = oracle.extend(m, d, k, cp, ri, v, P, Q, 1.0, 0.05, 1, eps=1e4)
    assert relerr(Ch.numpy(), Cr) <= 1e-2, relerr(Ch.numpy(), Cr)       # bf16 operands, fp32 accumulation
    # (1b) the same from random coefficients (warm start): the step now also depends on the first product W = C Q
    rng = np.random.default_rng(5)
    C0 = (rng.standard_normal((ncols, d)) * 0.05).astype(np.float32)
    Ch.copy_(torch.tensor(C0))
    B.tsid_extend(*args, Ch, chunk, 1, 1.0, 0.05, eps=1e4, tensor_cores=True)
    Cr, _ = oracle.extend(m, d, k, cp, ri, v, P, Q, 1.0, 0.05, 1, C0=C0, eps=1e4)
    step_err = float(np.max(np.abs((Ch.numpy() - C0) - (Cr - C0))) / np.max(np.abs(Cr - C0)))
    assert step_err <= 1e-2, step_err
    # (2) the fit
    eta, lam, iters = 0.02, 0.05, 12
    Ch.zero_()
    sse_tc = B.tsid_extend(*args, Ch, chunk, iters, eta, lam, want_sse=True, tensor_cores=True)
    C_tc = Ch.numpy().copy()
    Cr, sse_r = oracle.extend(m, d, k, cp, ri, v, P, Q, eta, lam, iters)
    rms = float(np.sqrt(np.mean((C_tc - Cr) ** 2)) / np.sqrt(np.mean(Cr ** 2)))
    assert rms <= 0.1, rms
    assert abs(sse_tc - sse_r) / sse_r <= 1e-3
    assert not C_tc[min(3, ncols - 1)].any()
    # (3) element by element against the oracle that rounds the operands of the two products as this form does
    # (the loose bounds above compare a bf16 computation with an fp64 one; here only fp32 summation is left, plus
    # Adam's sensitivity on coordinates whose gradient nearly cancels, which the fp32 form has as well)
    # One thing besides summation order is left: a coordinate of U that sits within fp32 rounding of the midpoint of
    # two bf16 values rounds the other way in the kernel (about 1 in 10^4); that moves the whole gradient of its column
    # by one bf16 step of that coordinate times a row of Q.  So: all but a few columns within 1e-5, none further off
    # than two such flips.
    colof = np.repeat(np.arange(ncols), np.diff(cp))
    U0 = np.zeros((ncols, k)); np.add.at(U0, colof, v[:, None].astype(np.float64) * P[ri].astype(np.float64))
    flip = 2.0 * 2.0 ** -8 * np.abs(U0).max() * np.abs(Q).max() * (1.0 / 1e4)      # in units of the step: eta / eps = 1e-4
    for c0 in (None, C0):
        Ch.zero_() if c0 is None else Ch.copy_(torch.tensor(c0))
        B.tsid_extend(*args, Ch, chunk, 1, 1.0, 0.05, eps=1e4, tensor_cores=True)
        Cm, _ = oracle.extend_mixed(m, d, k, cp, ri, v, P, Q, 1.0, 0.05, 1, C0=c0, eps=1e4)
        base = 0.0 if c0 is None else c0
        err = np.abs((Ch.numpy() - base) - (Cm - base))
        loose = err > 1e-5 * np.max(np.abs(Cm - base))
        assert loose.any(axis=1).mean() <= 0.03 and err.max() <= 2 * 2 * flip, (loose.any(axis=1).mean(), err.max(), flip)
    Cm, sse_m = oracle.extend_mixed(m, d, k, cp, ri, v, P, Q, eta, lam, iters)
    scale = float(np.abs(Cm).max())
    err = np.abs(C_tc - Cm)
    assert abs(sse_tc - sse_m) <= 1e-4 * sse_m, (sse_tc, sse_m)
    assert float(np.sqrt(np.mean(err ** 2))) <= 1e-3 * scale and int((err > 2e-3 * scale).sum()) <= max(3, err.size // 2000), (
        float(np.sqrt(np.mean(err ** 2))) / scale, int((err > 2e-3 * scale).sum()), err.size)
    # a shape the tensor-core form does not take is refused, not silently run another way
    with pytest.raises(B.TsidError) as e:
        B.tsid_extend(torch.tensor(P[:, :32].copy(), device=DEV), torch.tensor(Q[:, :32].copy(), device=DEV), *args[2:], Ch,
                      chunk, 1, eta, lam, tensor_cores=True)
    assert e.value.status == B.TSID_ERR_UNSUPPORTED


def test_extend_tensor_core_form_refuses_a_width_it_cannot_tile():
    """d must be a multiple of 8 (16-byte rows of the bf16 copy, a TMA requirement): 260 is refused, not padded."""
    P, Q, cp, ri, v = _problem(300, 260, 64, 40, 30, seed=2)
    Ch = torch.zeros(40, 260).pin_memory()
    with pytest.raises(B.TsidError) as e:
        B.tsid_extend(torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV), torch.tensor(cp).pin_memory(),
                      torch.tensor(ri).pin_memory(), torch.tensor(v).pin_memory(), Ch, 20, 2, 0.02, 0.05, tensor_cores=True)
    assert e.value.status == B.TSID_ERR_UNSUPPORTED
    # the fp32 form takes the same shape
    B.tsid_extend(torch.tensor(P, device=DEV), torch.tensor(Q, device=DEV), torch.tensor(cp).pin_memory(),
                  torch.tensor(ri).pin_memory(), torch.tensor(v).pin_memory(), Ch, 20, 2, 0.02, 0.05)
    Cr, _ = oracle.extend(300, 260, 64, cp, ri, v, P, Q, 0.02, 0.05, 2)
    assert relerr(Ch.numpy(), Cr) <= 2e-3
