"""One rank of the two-process row-sharded step test (started by tests/test_gpu_sharded.py, not collected by pytest).

Both ranks share the one GPU; the process group is gloo (host-side exchange of CUDA tensors, every collective
bounded by the group's timeout), so no kernel of one rank ever waits for a kernel of the other.  Each rank owns a
block of rows, runs RowShard.step - tsid_grad, all-reduce (sum) of G_Q, tsid_apply - three times, and rank 0
compares the assembled factors with the oracle's full-batch steps on the whole template.
"""
import datetime
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
from helpers import small_workload  # noqa: E402
from paper_2608_00977_b200 import binding as B  # noqa: E402
from paper_2608_00977_b200 import sharded as S  # noqa: E402
from paper_2608_00977_b200 import workloads as W  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    precision = sys.argv[1]
    dist.init_process_group("gloo", timeout=datetime.timedelta(seconds=60))
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    m, n, k, nnz, steps = 1500, 700, 32, 120_000, 3       # even m: gloo gathers equal blocks
    w = small_workload("shard2p-" + precision, m, n, k, nnz, positions="zipf", seed=29, precision=precision, eta=0.05,
                       lam=0.03, xi=0.1, clip=W.CLIP_ASYM_STEP, norm_p=W.NORM_COUNT, norm_q=W.NORM_COUNT)
    tpl = W.make_template(w, dev, order="shuffled")          # the same seeded template on both ranks
    r0, r1 = S.row_block(m, rank, world)
    rows, cols, vals = S.shard_coo(tpl.rows, tpl.cols, tpl.vals, r0, r1)
    prec = B.TSID_BF16_SHADOW if precision == "bf16" else B.TSID_F32
    sh = S.RowShard(r1 - r0, n, k, rows, cols, vals, precision=prec, eta=w.eta, lam=w.lam, xi=w.xi, clip=w.clip,
                    norm_p=w.norm_p, norm_q=w.norm_q, dist=dist)
    P, Q = tpl.P0[r0:r1].clone().contiguous(), tpl.Q0.clone()
    for _ in range(steps):
        sh.step(P.view(-1), Q.view(-1))
        sh.T.tsid_check()
    sse = sh.sse(P.view(-1), Q.view(-1))
    # assemble P on rank 0; the Q replicas must be bitwise equal
    parts = [torch.empty(S.row_block(m, r, world)[1] - S.row_block(m, r, world)[0], k, device=dev) for r in range(world)]
    dist.all_gather(parts, P)
    qs = [torch.empty_like(Q) for _ in range(world)]
    dist.all_gather(qs, Q)
    ok = all(torch.equal(q, qs[0]) for q in qs)
    if rank == 0:
        rr, cc, vv = (x.cpu().numpy() for x in (tpl.rows, tpl.cols, tpl.vals))
        Pr, Qr, hist = oracle.fit(m, n, k, rr, cc, vv, tpl.P0.cpu().numpy(), tpl.Q0.cpu().numpy(), steps, w.eta, w.lam, w.xi,
                                  w.clip, w.norm_p, w.norm_q, bf16_emulate=(precision == "bf16"))
        Pg = torch.cat(parts).cpu().numpy()
        ep = float(np.max(np.abs(Pg - Pr)) / np.max(np.abs(Pr)))
        eq = float(np.max(np.abs(qs[0].cpu().numpy() - Qr)) / np.max(np.abs(Qr)))
        es = abs(sse - hist[-1]) / hist[-1]
        print("rank0 errs P %.3e Q %.3e sse %.3e replicas_equal %s" % (ep, eq, es, ok), flush=True)
        ok = ok and ep <= 5e-4 and eq <= 5e-4 and es <= 1e-4
    sh.destroy()
    dist.barrier()
    dist.destroy_process_group()
    sys.exit(0 if ok else 1)


if __name__ == "__main__":
    main()
