"""Layout pass parity (bit-exact integers and values) against the oracle's sort, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import np_coo, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check(m, n, rows, cols, vals, flags=0, k=8):
    rows_t = torch.as_tensor(rows, dtype=torch.int32, device=DEV)
    cols_t = torch.as_tensor(cols, dtype=torch.int32, device=DEV)
    vals_t = torch.as_tensor(vals, dtype=torch.float32, device=DEV)
    cfg = B.make_config(m, n, k, len(rows), flags=flags)
    T = B.Template(cfg, rows_t, cols_t, vals_t)
    got = [x.cpu().numpy() for x in T.tsid_get_layout()]
    ref = oracle.layout(m, n, rows, cols, vals)
    names = ["row_ptr", "col_idx", "val_csr", "col_ptr", "row_idx", "val_csc", "perm"]
    for g, nm in zip(got, names):
        r = getattr(ref, nm)
        if nm == "perm":
            g = g.view(np.uint32)
        assert g.dtype == r.dtype and g.shape == r.shape, nm
        assert np.array_equal(g.view(np.uint8), r.view(np.uint8)), nm   # bit-exact, floats included
    T.tsid_destroy()


@pytest.mark.parametrize("order", ["sorted", "shuffled"])
def test_layout_c1(order):
    tpl = W.make_template(W.C1, DEV, order=order)
    r, c, v = np_coo(tpl)
    _check(W.C1.m, W.C1.n, r, c, v)


@pytest.mark.parametrize("m,n,nnz,pos", [(5000, 2000, 300_000, "zipf"), (300, 70_000, 250_000, "zipf"),
                                         (70_000, 300, 250_000, "zipf"), (1, 4000, 3000, "uniform"),
                                         (4000, 1, 3000, "uniform"), (40, 50, 2000, "uniform")])
def test_layout_shapes(m, n, nnz, pos):
    w = small_workload("lay", m, n, 8, nnz, positions=pos, seed=m + n)
    tpl = W.make_template(w, DEV, order="shuffled")
    r, c, v = np_coo(tpl)
    _check(m, n, r, c, v)


@pytest.mark.parametrize("m,n", [(20_000_000, 130), (130, 20_000_000), (17_000_000, 17_000_000)])
def test_layout_four_pass_sorts(m, n):
    """More than 2^24 rows or columns: four radix passes per sort, so the sorts end in the other buffer set
    than with the three passes of the workload sizes."""
    rng = np.random.default_rng(m % 1000 + n % 1000)
    nnz = 120_000
    key = np.unique(rng.integers(0, m, nnz).astype(np.int64) * n + rng.integers(0, n, nnz))
    key = key[rng.permutation(len(key))]
    rows, cols = (key // n).astype(np.int32), (key % n).astype(np.int32)
    _check(m, n, rows, cols, rng.standard_normal(len(key)).astype(np.float32), k=4)


def test_layout_degenerate_cases():
    _check(7, 5, np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.float32))     # empty Omega
    _check(7, 5, np.array([3], np.int32), np.array([4], np.int32), np.array([2.5], np.float32))
    # rows 0 and 6 and column 2 empty; one full row
    rows = np.array([5, 1, 5, 5, 2, 5, 5, 1], np.int32); cols = np.array([4, 0, 0, 3, 1, 1, 2, 4], np.int32)
    _check(7, 5, rows, cols, np.arange(8, dtype=np.float32))
    # duplicates are kept in input order when not validated
    rows = np.array([1, 0, 1, 1, 0], np.int32); cols = np.array([2, 0, 2, 1, 0], np.int32)
    _check(2, 3, rows, cols, np.array([10, 20, 30, 40, 50], np.float32))
    # row-sorted promise on sorted input
    rows = np.array([0, 0, 1, 3], np.int32); cols = np.array([1, 2, 0, 3], np.int32)
    _check(4, 4, rows, cols, np.ones(4, np.float32), flags=B.TSID_INPUT_ROW_SORTED)


def test_layout_full_size_c2_invariants_and_samples():
    """Full C2 size: the oracle's qsort of 10M triples takes seconds, so compare everything."""
    tpl = W.make_template(W.C2, DEV, order="shuffled")
    r, c, v = np_coo(tpl)
    _check(W.C2.m, W.C2.n, r, c, v, k=32)


def test_create_errors():
    rows = torch.tensor([0, 1, 2], dtype=torch.int32, device=DEV)
    cols = torch.tensor([0, 1, 5], dtype=torch.int32, device=DEV)
    vals = torch.ones(3, device=DEV)
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(3, 5, 8, 3), rows, cols, vals)
    assert e.value.status == B.TSID_ERR_INDEX_RANGE
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(3, 6, 8, 3), -rows - 1, cols, vals)
    assert e.value.status == B.TSID_ERR_INDEX_RANGE
    dr = torch.tensor([2, 0, 2], dtype=torch.int32, device=DEV); dc = torch.tensor([1, 0, 1], dtype=torch.int32, device=DEV)
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(3, 6, 8, 3, flags=B.TSID_VALIDATE), dr, dc, vals)
    assert e.value.status == B.TSID_ERR_DUPLICATE
    B.Template(B.make_config(3, 6, 8, 3), dr, dc, vals).tsid_destroy()          # accepted without VALIDATE
    with pytest.raises(B.TsidError) as e:
        B.Template(B.make_config(3, 6, 8, 3, flags=B.TSID_INPUT_ROW_SORTED), dr, dc, vals)
    assert e.value.status == B.TSID_ERR_UNSORTED
    # workspace too small
    import ctypes as C
    cfg = B.make_config(3, 6, 8, 3)
    ws = torch.empty(4096, dtype=torch.uint8, device=DEV)
    cfg.workspace = (ws.data_ptr() + 255) & ~255
    cfg.workspace_bytes = 1024
    h = C.c_void_p(None)
    st = B.lib().tsid_template_create(C.byref(cfg), dr.data_ptr(), dc.data_ptr(), vals.data_ptr(), C.byref(h))
    assert st == B.TSID_ERR_OOM and h.value is None
