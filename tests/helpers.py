"""Shared helpers of the GPU parity tests (comparison metrics, oracle calls on workload templates)."""
import numpy as np
import torch

import oracle
from paper_2608_00977_b200 import binding as B
from paper_2608_00977_b200 import workloads as W

# max relative error in the infinity norm: max|a - ref| / max|ref|  (fp32 path bar: 1e-4)
F32_TOL = 1e-4


def relerr(a, ref):
    a = np.asarray(a, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    den = np.max(np.abs(ref)) if ref.size else 1.0
    if den == 0.0:
        den = 1.0
    return float(np.max(np.abs(a - ref)) / den) if ref.size else 0.0


def rowwise_relerr(a, ref, counts):
    """Per-row check: max_i |a_i - ref_i|_inf / max(|ref_i|_inf, floor_i).  The whole-matrix metric above lets the
    most populated rows set the scale; here every row is held to its own size.  A row whose terms cancel has no
    relative accuracy of its own, so the denominator never goes below the size a sum of count_i random-sign
    terms has: floor_i = sqrt(max(count_i, 1)) * t, t = the median over rows of |ref_i|_inf / sqrt(count_i)."""
    a = np.asarray(a, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    c = np.sqrt(np.maximum(np.asarray(counts, dtype=np.float64), 1.0))
    mag = np.max(np.abs(ref), axis=1)
    t = np.median((mag / c)[mag > 0]) if np.any(mag > 0) else 1.0
    return float(np.max(np.max(np.abs(a - ref), axis=1) / np.maximum(mag, c * t)))


def np_coo(tpl):
    return (tpl.rows.cpu().numpy(), tpl.cols.cpu().numpy(), tpl.vals.cpu().numpy())


def oracle_step(tpl, P, Q, bf16_emulate=False):
    w = tpl.w
    r, c, v = np_coo(tpl)
    return oracle.grad_step(w.m, w.n, w.k, r, c, v, P, Q, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q,
                            bf16_emulate=bf16_emulate)


def gpu_step(tpl, precision=None, path=B.TSID_PATH_SPARSE, flags=0):
    """One tsid_grad_step on copies of the template's initial factors.  Returns (T, P1, Q1, GP, GQ) as numpy."""
    T = B.template_from_workload(tpl, path=path, flags=flags, precision=precision)
    P = tpl.P0.clone(); Q = tpl.Q0.clone()
    GP = torch.empty_like(P); GQ = torch.empty_like(Q)
    T.tsid_grad_step(P, Q, GP, GQ)
    T.tsid_check()
    return T, P.cpu().numpy(), Q.cpu().numpy(), GP.cpu().numpy(), GQ.cpu().numpy()


def small_workload(name, m, n, k, nnz, positions="uniform", precision="f32", seed=7, **kw):
    base = dict(values="lowrank", noise_var=1e-4, eta=0.01, lam=0.0, xi=0.1, clip=W.CLIP_NONE,
                norm_p=W.NORM_NONE, norm_q=W.NORM_NONE, epochs=5, zipf_s=1.1)
    base.update(kw)
    return W.Workload(name, m, n, k, nnz, positions, precision=precision, seed=seed, **base)
