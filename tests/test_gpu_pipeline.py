"""The whole method end to end on a synthetic low-rank matrix with held-out entries: column sampling
(Sec. 5.1), template recovery (Stage I, Secs. 3.2 / 5.1 / 5.3), extension (Stage II, Sec. 5.2, Eq. 10),
prediction R^ = (P Q^T) C and the paper's error measure NMAE (Sec. 6.1).  No dataset is involved: the
matrix is the paper's own synthetic recipe (product of two random factors, random mask)."""
import numpy as np
import pytest
import torch

from paper_2608_00977_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def nmae(pred, truth, lo, hi):
    """Normalised mean absolute error over the test entries: sum |pred - truth| / (count (max - min))."""
    return float(np.mean(np.abs(pred - truth)) / (hi - lo))


@pytest.mark.parametrize("tensor_cores", [False, True])
def test_sample_recover_extend_predict(tensor_cores):
    rng = np.random.default_rng(12)
    m, n, rank, k = 1500, 1200, 6, 64
    A, Bm = rng.standard_normal((m, rank)), rng.standard_normal((n, rank))
    R = (A @ Bm.T / np.sqrt(rank)).astype(np.float32)
    mask = rng.random((m, n)) < 0.35
    test = mask & (rng.random((m, n)) < 0.1)          # held out
    train = mask & ~test
    rows, cols = np.nonzero(train)
    vals = R[rows, cols]
    rows_t, cols_t = torch.tensor(rows.astype(np.int32), device=DEV), torch.tensor(cols.astype(np.int32), device=DEV)
    vals_t = torch.tensor(vals, device=DEV)

    # template: 40 % of the columns
    colmap, tr, tc, tv, d = B.tsid_sample_template(m, n, rows_t, cols_t, vals_t, 0.4, 2024)
    assert d == 480 and d % 8 == 0
    cfg = B.make_config(m, d, k, tr.numel(), B.TSID_F32, B.TSID_PATH_SPARSE, 0.05, 0.02, 0.1, B.TSID_CLIP_ASYM_STEP,
                        B.TSID_NORM_COUNT, B.TSID_NORM_COUNT)
    T = B.Template(cfg, tr.contiguous(), tc.contiguous(), tv.contiguous())
    g = torch.Generator(device=DEV).manual_seed(3)
    P = (torch.randn(m, k, device=DEV, generator=g) * k ** -0.25).contiguous()
    Q = (torch.randn(d, k, device=DEV, generator=g) * k ** -0.25).contiguous()
    hist = T.tsid_fit(P, Q, 300, loss_every=300)
    assert hist[-1] < 0.1 * hist[0]
    T.tsid_destroy()

    # extension: every column of the full matrix against the recovered template
    order = np.lexsort((rows, cols))
    col_ptr = np.zeros(n + 1, np.int64)
    col_ptr[1:] = np.cumsum(np.bincount(cols, minlength=n))
    Ch = torch.zeros(n, d).pin_memory()
    B.tsid_extend(P, Q, torch.tensor(col_ptr).pin_memory(), torch.tensor(rows[order].astype(np.int32)).pin_memory(),
                  torch.tensor(vals[order]).pin_memory(), Ch, 300, 60, 0.02, 0.01, cold_start=True,
                  tensor_cores=tensor_cores)

    # prediction on the held-out entries: R^_ij = p_i . (Q^T C_j)
    W = Ch.numpy().astype(np.float64) @ Q.cpu().numpy().astype(np.float64)          # n x k
    ti, tj = np.nonzero(test)
    pred = np.einsum("ek,ek->e", P.cpu().numpy().astype(np.float64)[ti], W[tj])
    truth = R[ti, tj]
    lo, hi = float(R[mask].min()), float(R[mask].max())
    err = nmae(pred, truth, lo, hi)
    base = nmae(np.full_like(truth, vals.mean()), truth, lo, hi)       # predicting the mean rating
    print("NMAE %.4f (mean predictor %.4f), tensor cores %s" % (err, base, tensor_cores))
    assert err < 0.35 * base
