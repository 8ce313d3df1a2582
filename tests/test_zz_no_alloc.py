"""tsid_sse_noalloc: the loss entry point for callers that may not allocate device memory.

Such callers (a hook inside a process whose framework has reserved the whole GPU, a real-time loop, a
plug-in that only receives pointers and a stream) cannot build a workspace for tsid_loss.  The variant
keeps its reduction scratch in a fixed array inside the library.  Here it is called through the C ABI
twice in a row (the second call finds the first call's leftovers in the scratch) and compared with what
tsid_loss returns for the same template and with the CPU oracle's loss, at the tolerance the loss tests
use (1e-5 relative).

This file sorts last on purpose, so that a run that stops at the first failure has already run the rest.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from helpers import np_coo, small_workload
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _sse_noalloc(w, tpl, P, Q):
    out = torch.full((1,), -1.0, dtype=torch.float64, device=DEV)
    B.tsid_sse_noalloc(w.m, w.n, w.k, tpl.rows, tpl.cols, tpl.vals, P, Q, out)
    return float(out.item())


def test_noalloc_sse_matches_tsid_loss_on_two_calls_in_a_row():
    big = small_workload("na-big", 3000, 2500, 64, 700_003, positions="zipf", seed=21, values="ratings", noise_var=0.25)
    small = small_workload("na-small", 400, 300, 20, 5_001, seed=22)
    refs, got = [], []
    tpls = [W.make_template(big, DEV, order="shuffled"), W.make_template(small, DEV, order="shuffled")]
    for w, tpl in zip((big, small), tpls):
        T = B.template_from_workload(tpl, precision=B.TSID_F32)
        refs.append(T.tsid_loss(tpl.P0, tpl.Q0)[0])
        T.tsid_destroy()
    # first call fills 684 scratch slots, the second (smaller) one reuses the first five of them
    for w, tpl in zip((big, small), tpls):
        got.append(_sse_noalloc(w, tpl, tpl.P0, tpl.Q0))
    # and once more in the opposite order, with different factors
    P2, Q2 = tpls[0].P0 * 0.5, tpls[0].Q0 * 0.5
    T = B.template_from_workload(tpls[0], precision=B.TSID_F32)
    ref2 = T.tsid_loss(P2, Q2)[0]
    T.tsid_destroy()
    got2 = _sse_noalloc(big, tpls[0], P2, Q2)
    for g, r in zip(got + [got2], refs + [ref2]):
        assert r > 0 and abs(g - r) / r <= 1e-5, (g, r)
    # and against the CPU oracle's loss (double sums over the COO triples), at the same tolerance
    orc = []
    for w, tpl, scale in ((big, tpls[0], 1.0), (small, tpls[1], 1.0), (big, tpls[0], 0.5)):
        r, c, v = np_coo(tpl)
        orc.append(oracle.loss(w.m, w.n, w.k, r, c, v, tpl.P0.cpu().numpy() * np.float32(scale),
                               tpl.Q0.cpu().numpy() * np.float32(scale), 0.0)[0])
    for g, r in zip(got + [got2], orc):
        assert r > 0 and abs(g - r) / r <= 1e-5, (g, r)
    # deterministic: the same call again gives the same bits
    assert _sse_noalloc(big, tpls[0], P2, Q2) == got2


def test_noalloc_limits_and_errors():
    L = B.lib()
    w = small_workload("na-err", 64, 48, 16, 500, seed=1)
    tpl = W.make_template(w, DEV)
    out = torch.zeros(1, dtype=torch.float64, device=DEV)
    args = lambda nnz, k=16, P=tpl.P0.data_ptr(): (w.m, w.n, k, nnz, tpl.rows.data_ptr(), tpl.cols.data_ptr(),
                                                   tpl.vals.data_ptr(), P, tpl.Q0.data_ptr(), None, out.data_ptr())
    assert L.tsid_sse_noalloc(*args((1 << 26) + 1)) == B.TSID_ERR_TOO_LARGE      # beyond the built-in scratch
    assert L.tsid_sse_noalloc(*args(500, k=6)) == B.TSID_ERR_UNSUPPORTED
    assert L.tsid_sse_noalloc(*args(500, P=None)) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_sse_noalloc(*args(500, P=tpl.P0.data_ptr() + 4)) == B.TSID_ERR_INVALID_ARG
    assert L.tsid_sse_noalloc(*args(0)) == B.TSID_OK                              # empty template: SSE = 0
    torch.cuda.synchronize()
    assert out.item() == 0.0
