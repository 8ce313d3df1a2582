"""Template sampling: oracle pins (CPU) and GPU parity through the C ABI."""
import os

import numpy as np
import pytest

import oracle
from conftest import ROOT


def _vectors():
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", "splitmix64.txt")) as f:
        for line in f:
            if line.startswith("#") or ":" not in line:
                continue
            k, v = line.split(":")
            out[int(k.strip()[4:])] = [int(x, 0) for x in v.split()]
    return out


def test_keys_are_the_splitmix64_stream():
    for seed, outs in _vectors().items():
        for i, want in enumerate(outs):
            assert oracle.splitmix64_at(seed, i + 1) == want


def _coo(m, n, nnz, seed):
    rng = np.random.default_rng(seed)
    ids = rng.choice(m * n, nnz, replace=False)
    rows, cols = (ids // n).astype(np.int32), (ids % n).astype(np.int32)
    return rows, cols, rng.standard_normal(nnz).astype(np.float32)


@pytest.mark.parametrize("n,alpha", [(50, 0.1), (50, 0.5), (7, 0.3), (33, 1.0), (1, 0.2), (1000, 0.001)])
def test_sample_size_map_and_membership(n, alpha):
    m = 40
    rows, cols, vals = _coo(m, n, min(m * n, 600), n)
    colmap, ro, co, vo, d = oracle.sample_template(m, n, rows, cols, vals, alpha, 42)
    assert d == int(np.ceil(alpha * n)) and 1 <= d <= n
    chosen = np.nonzero(colmap >= 0)[0]
    assert len(chosen) == d and np.array_equal(colmap[chosen], np.arange(d))     # ranks in ascending column order
    # the chosen set is the d smallest (key, column) pairs, by brute force in Python integers
    keys = sorted((oracle.splitmix64_at(42, j + 1), j) for j in range(n))
    assert sorted(j for _, j in keys[:d]) == chosen.tolist()
    keep = np.isin(cols, chosen)
    assert np.array_equal(ro, rows[keep]) and np.array_equal(vo, vals[keep])      # input order preserved
    assert np.array_equal(chosen[co], cols[keep])
    if alpha == 1.0:
        assert np.array_equal(co, cols) and d == n


def test_sampling_is_uniform_over_columns():
    n, alpha, trials = 20, 0.3, 3000
    cnt = np.zeros(n)
    r = c = np.zeros(0, np.int32); v = np.zeros(0, np.float32)
    for s in range(trials):
        colmap = oracle.sample_template(3, n, r, c, v, alpha, 1000 + s)[0]
        cnt += colmap >= 0
    freq = cnt / trials
    assert np.all(np.abs(freq - 0.3) < 4.5 * np.sqrt(0.3 * 0.7 / trials)), freq
    assert cnt.sum() == trials * 6


@pytest.mark.gpu
@pytest.mark.parametrize("m,n,nnz,alpha,seed", [(300, 200, 9000, 0.1, 1), (64, 5000, 40_000, 0.5, 2), (500, 37, 3000, 0.3, 3),
                                               (100, 100, 0, 0.2, 4), (2000, 1500, 150_000, 1.0, 5), (50, 3, 120, 0.01, 6),
                                               (900, 300_000, 700_000, 0.37, 7),      # several tiles per block
                                               (40, 2_500_000, 60_000, 0.5, 8)])      # bitmap too large for shared memory
def test_gpu_sampling_is_bit_exact(m, n, nnz, alpha, seed):
    import torch
    from paper_2608_00977_b200 import binding as B
    rows, cols, vals = _coo(m, n, nnz, seed)
    dev = "cuda:0"
    got = B.tsid_sample_template(m, n, torch.tensor(rows, device=dev), torch.tensor(cols, device=dev),
                                 torch.tensor(vals, device=dev), alpha, 7000 + seed)
    ref = oracle.sample_template(m, n, rows, cols, vals, alpha, 7000 + seed)
    assert got[4] == ref[4]
    for g, r in zip(got[:4], ref[:4]):
        g = g.cpu().numpy()
        assert g.dtype == r.dtype and g.shape == r.shape and np.array_equal(g.view(np.uint8), r.view(np.uint8))


@pytest.mark.gpu
def test_gpu_sample_then_factorize_end_to_end():
    """R -> template -> (P, Q): the sampled triples feed tsid_template_create with n = d."""
    import torch
    from paper_2608_00977_b200 import binding as B
    from paper_2608_00977_b200 import workloads as W
    dev = "cuda:0"
    tpl = W.make_template(W.scaled(W.C2, "full-matrix", 4000, 6000, 400_000), dev, order="shuffled")
    colmap, r, c, v, d = B.tsid_sample_template(4000, 6000, tpl.rows, tpl.cols, tpl.vals, 0.25, 99)
    assert d == 1500 and 0 < r.numel() < tpl.nnz
    ref = oracle.sample_template(4000, 6000, tpl.rows.cpu().numpy(), tpl.cols.cpu().numpy(), tpl.vals.cpu().numpy(), 0.25, 99)
    assert np.array_equal(c.cpu().numpy(), ref[2])
    cfg = B.make_config(4000, d, 32, r.numel(), B.TSID_F32, B.TSID_PATH_SPARSE, 0.05, 0.03, 0.1, 1, 1, 1)
    T = B.Template(cfg, r.contiguous(), c.contiguous(), v.contiguous())
    P, Q = tpl.P0.clone(), tpl.Q0[:d].clone().contiguous()
    h = T.tsid_fit(P, Q, 10, loss_every=10)
    assert h[1] < h[0]
    bad = torch.full((5,), 6000, dtype=torch.int32, device=dev)
    with pytest.raises(B.TsidError) as e:
        B.tsid_sample_template(10, 6000, bad, bad, torch.ones(5, device=dev), 0.5, 1)
    assert e.value.status == B.TSID_ERR_INDEX_RANGE
