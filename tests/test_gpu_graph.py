"""A lookup captured in a CUDA graph and replayed.

Between two request ends the pool does not change (a trace joins it when its request is
over), so a serving loop can capture one lookup (query states in a fixed buffer, results in
fixed buffers) and replay it at every decoding step.  The entry points only enqueue work on
the caller's stream, which is what makes them capturable; the replays must give what direct
calls give, for every scan path."""
import numpy as np
import pytest
import torch

from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query, fill_both

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nq,path,rows", [(1, B.PATH_GEMV, 6000), (8, B.PATH_MMA, 6000),
                                          (16, B.PATH_TENSOR, 6000), (160, B.PATH_TENSOR, 76000)])
def test_captured_lookup_replays_like_direct_calls(nq, path, rows):
    w = W.C1.scaled(n_rows=rows, d=256, nq=nq, k=8, cont_len=4, rows_per_trace=500, seed=60 + nq)
    pool, ora = fill_both(w, max_nq=256)
    pr = B.QueryParams(k=8, theta=-2.0, depth_mode=B.DEPTH_FIXED, cont_len=4, path=path)
    q_buf = torch.zeros(nq, w.d, dtype=torch.bfloat16, device="cuda")
    out = B.QueryOut.empty(nq, 8, 4, "cuda")
    qs = [w.queries("cuda", nq=nq, step=s)[0] for s in range(4)]
    q_buf.copy_(qs[0])
    pool.query(q_buf, pr, out=out)                       # warm (nothing is loaded lazily, but be plain)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        pool.query(q_buf, pr, out=out)
    for s in range(4):
        q_buf.copy_(qs[s])
        g.replay()
        torch.cuda.synchronize()
        check_query(out, ora, W.to_bits(qs[s]), pr)
        direct = pool.query(qs[s], pr).cpu()
        got = out.cpu()
        assert torch.equal(got.idx, direct.idx) and torch.equal(got.score, direct.score)
        assert torch.equal(got.cont_tok, direct.cont_tok)
    assert pool.stats()["stalled"] == 0
