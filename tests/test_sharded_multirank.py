"""Host logic of the sharded query on CPU ranks (gloo, world size 2): record layout and the
single all-gather.  The CUDA kernels are not involved; the merge of the gathered records
is redone with numpy to check that every rank sees every rank's record, in rank order."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2608_03839_b200 import sharded as S
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lay = S.RecordLayout(nq=3, k=4, L=5)
    buf = torch.zeros(lay.nbytes, dtype=torch.uint8)
    gidx, rec = lay.views(buf)
    # rank r pretends to have found rows 100*r + j with scores 0.9 - 0.1*j - 0.05*r
    for q in range(3):
        for j in range(4):
            gidx[q, j] = 100 * rank + 10 * q + j
            rec.score[q, j] = 0.9 - 0.1 * j - 0.05 * rank
            rec.cont_len[q, j] = j
            rec.cont_tok[q, j, :] = 1000 * rank + 10 * j
    g = S.all_gather_records(buf)
    assert g.shape == (world, lay.nbytes)
    merged = []
    for r in range(world):
        gi, rr = lay.views(g[r])
        assert gi[0, 0] == 100 * r and int(rr.cont_tok[1, 2, 0]) == 1000 * r + 20
        merged += [(-float(rr.score[0, j]), int(gi[0, j])) for j in range(4)]
    merged.sort()
    out.put((rank, [m[1] for m in merged[:4]]))
    dist.barrier()
    dist.destroy_process_group()


def test_records_travel_in_one_all_gather_and_arrive_in_rank_order():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # scores: rank0 .9 .8 .7 .6 ; rank1 .85 .75 .65 .55 -> interleaved, same on both ranks
    assert res[0][1] == res[1][1] == [0, 100, 1, 101]


def test_layout_is_aligned_and_disjoint():
    sys.path.insert(0, ROOT)
    from paper_2608_03839_b200 import sharded as S
    for nq, k, L in [(1, 1, 1), (3, 5, 7), (256, 64, 16), (8, 8, 32)]:
        lay = S.RecordLayout(nq, k, L)
        offs = [lay.off_gidx, lay.off_score, lay.off_len, lay.off_tok, lay.off_idx, lay.off_fired,
                lay.nbytes]
        assert offs == sorted(offs) and lay.off_gidx % 8 == 0 and lay.nbytes % 8 == 0
        assert lay.off_score - lay.off_gidx == nq * k * 8 and lay.off_idx - lay.off_tok == nq * k * L * 4
        buf = torch.zeros(lay.nbytes, dtype=torch.uint8)
        gidx, rec = lay.views(buf)
        gidx.fill_(-1); rec.score.fill_(1.0); rec.cont_len.fill_(2); rec.cont_tok.fill_(3)
        rec.idx.fill_(4); rec.fired.fill_(5)
        g2, r2 = lay.views(buf)
        assert torch.all(g2 == -1) and torch.all(r2.score == 1.0) and torch.all(r2.cont_len == 2)
        assert torch.all(r2.cont_tok == 3) and torch.all(r2.idx == 4) and torch.all(r2.fired == 5)
