"""The largest template the interface admits: nnz = 2^31 - 1 entries (2,000,000 x 1,000,000, k = 32).

The pattern is a closed form so that nothing has to be deduplicated and the expected CSR is known without
sorting: entry t sits in row t // 1074 at column q*931 + (row*7919 mod 931), q = t mod 1074 (columns ascend
within a row, distinct by construction; the last row is cut short and the rows after it are empty).  Every
row is longer than one segment, every column has about 2,148 entries.  Checked: CSR arrays bit for bit
against the closed form, the CSC arrays and perm through their defining properties over all 2^31 - 1
positions, and one step on sampled rows and columns against the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import relerr
from paper_2608_00977_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

M, N, K = 2_000_000, 1_000_000, 32
NNZ = 2**31 - 1
PER_ROW, STRIDE, MULT = 1074, 931, 7919
CHUNK = 1 << 25


def _pattern():
    rows = torch.empty(NNZ, dtype=torch.int32, device=DEV)
    cols = torch.empty(NNZ, dtype=torch.int32, device=DEV)
    vals = torch.empty(NNZ, dtype=torch.float32, device=DEV)
    for a in range(0, NNZ, CHUNK):
        b = min(NNZ, a + CHUNK)
        t = torch.arange(a, b, dtype=torch.int64, device=DEV)
        r = t // PER_ROW
        q = t - r * PER_ROW
        rows[a:b] = r.to(torch.int32)
        cols[a:b] = (q * STRIDE + (r * MULT) % STRIDE).to(torch.int32)
        vals[a:b] = (((t * 2654435761) >> 13) % 5 + 1).to(torch.float32)
    return rows, cols, vals


def test_largest_admissible_template():
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info(0)
    cfg = B.make_config(M, N, K, NNZ, precision=B.TSID_BF16_SHADOW, path=B.TSID_PATH_SPARSE, eta=0.05, lam=0.03,
                        xi=0.1, clip=B.TSID_CLIP_ASYM_STEP, norm_p=B.TSID_NORM_COUNT, norm_q=B.TSID_NORM_COUNT,
                        flags=B.TSID_VALIDATE)
    need = B.tsid_workspace_bytes(cfg) + 12 * NNZ + 24 * (1 << 30)
    if free < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of free device memory, {free / 2**30:.0f} GiB free")
    rows, cols, vals = _pattern()
    assert int(cols.max()) < N and int(rows[-1]) < M
    T = B.Template(cfg, rows, cols, vals)
    T.tsid_check()
    row_ptr, col_idx, val_csr, col_ptr, row_idx, val_csc, perm = T.tsid_get_layout(copy=False)

    # CSR: the input is already in (row, column) order
    assert torch.equal(col_idx, cols) and torch.equal(val_csr, vals)
    expect = torch.clamp(torch.arange(M + 1, dtype=torch.int64, device=DEV) * PER_ROW, max=NNZ)
    assert torch.equal(row_ptr, expect)
    del expect

    # CSC and perm, over every position: the entry perm points at has this row, this value and the column
    # whose segment holds the position; (column, row) ascends strictly, so perm repeats no entry
    assert int(col_ptr[0]) == 0 and int(col_ptr[-1]) == NNZ and bool((col_ptr[1:] >= col_ptr[:-1]).all())
    last_key = -1
    for a in range(0, NNZ, CHUNK):
        b = min(NNZ, a + CHUNK)
        p = perm[a:b].long() & 0xFFFFFFFF
        assert torch.equal(rows[p], row_idx[a:b])
        assert torch.equal(vals[p], val_csc[a:b])
        col_of_pos = torch.searchsorted(col_ptr, torch.arange(a, b, dtype=torch.int64, device=DEV), right=True) - 1
        assert torch.equal(cols[p].long(), col_of_pos)
        key = col_of_pos * (1 << 21) + row_idx[a:b].long()
        assert int(key[0]) > last_key and bool((key[1:] > key[:-1]).all())
        last_key = int(key[-1])
    del p, col_of_pos, key, row_ptr, col_idx, val_csr, col_ptr, row_idx, val_csc, perm

    # one step, sampled rows and columns against the oracle
    g = torch.Generator(device="cpu").manual_seed(31)
    P = (torch.randn(M, K, generator=g) * K ** -0.25).to(DEV)
    Q = (torch.randn(N, K, generator=g) * K ** -0.25).to(DEV)
    P0, Q0 = P.cpu().numpy(), Q.cpu().numpy()
    GP, GQ = torch.empty_like(P), torch.empty_like(Q)
    T.tsid_grad_step(P, Q, GP, GQ)
    T.tsid_check()
    last_row = (NNZ - 1) // PER_ROW
    rng = np.random.default_rng(31)
    for side, idx_all, other, nrow, Xg, G, Xnew, fixed in (
            ("rows", rows, cols, M, (P0, Q0), GP, P, [0, last_row, last_row + 1, M - 1]),
            ("cols", cols, rows, N, (Q0, P0), GQ, Q, [0, N - 1])):
        sample = np.unique(np.concatenate([np.asarray(fixed), rng.choice(nrow, 40, replace=False)]))
        lut = torch.full((nrow,), -1, dtype=torch.int32, device=DEV)
        lut[torch.as_tensor(sample, device=DEV)] = torch.arange(len(sample), dtype=torch.int32, device=DEV)
        loc = lut.index_select(0, idx_all)
        keep = loc >= 0
        sub_r = loc[keep].cpu().numpy(); sub_c = other[keep].cpu().numpy(); sub_v = vals[keep].cpu().numpy()
        del loc, keep
        st = oracle.grad_step(len(sample), Xg[1].shape[0], K, sub_r, sub_c, sub_v, Xg[0][sample], Xg[1], 0.05, 0.03,
                              0.1, oracle.CLIP_ASYM_STEP, oracle.NORM_COUNT, oracle.NORM_NONE, bf16_emulate=True)
        sel = torch.as_tensor(sample, device=DEV).long()
        assert relerr(G[sel].cpu().numpy(), st.GP) <= 1e-4, side
        assert relerr(Xnew[sel].cpu().numpy(), st.P) <= 1e-4, side
    # the empty rows behind the cut only decay
    empty = torch.arange(last_row + 1, M, device=DEV)
    assert not bool(GP[empty].any())
    T.tsid_destroy()
    del T, rows, cols, vals, P, Q, GP, GQ
    torch.cuda.empty_cache()
