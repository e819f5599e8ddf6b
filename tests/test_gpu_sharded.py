"""Row sharding on one GPU: G pools stand for G ranks, their records are stacked by hand
instead of all-gathered, and the merged answer must be what one pool with all rows gives
(checked against the CPU oracle holding every row at its global position)."""
import numpy as np
import pytest
import torch

from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import sharded as S
from paper_2608_03839_b200 import workloads as W
from parity import check_query

pytestmark = pytest.mark.gpu


def build(w, n_shards, route):
    shards = [S.ShardedPool(w.d, w.n_rows) for _ in range(n_shards)]
    ora = OraclePool(w.d)
    g = 0
    for t, (st, tk, tag) in enumerate(w.traces("cuda")):
        shards[route(t)].append(st, tk, global_row=g, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)       # global order
        g += st.shape[0]
    return shards, ora


def sharded_query(shards, q, pr):
    recs, lay = [], None
    for sh in shards:
        buf, lay = sh.local_record(q, pr)
        recs.append(buf.clone())
    return S.merge_gathered(torch.stack(recs), lay, pr.theta)


@pytest.mark.parametrize("n_shards", [1, 2, 3, 8])
@pytest.mark.parametrize("kind", ["clustered", "separated"])
def test_sharded_query_equals_single_pool(n_shards, kind):
    w = W.C1.scaled(n_rows=4096, nq=5, k=16, cont_len=6, d=512)
    if kind == "separated":
        w = w.separated()
    shards, ora = build(w, n_shards, lambda t: (t * 7 + 3) % n_shards)
    q, _ = w.queries("cuda")
    for theta, mode in ((0.8, B.DEPTH_FIXED), (-2.0, B.DEPTH_TIERED), (0.999, B.DEPTH_FIXED)):
        pr = B.QueryParams(k=w.k, theta=theta, depth_mode=mode, cont_len=w.cont_len)
        out = sharded_query(shards, q, pr)
        as_single = B.QueryOut(out.gidx.to(torch.int32), out.score, out.fired, out.cont_len,
                               out.cont_tok)
        check_query(as_single, ora, W.to_bits(q), pr)
    # a single unsharded pool gives the very same answer
    one = B.Pool(w.d, w.n_rows)
    for st, tk, tag in w.traces("cuda"):
        one.append(st, tk, tag=tag)
    pr = B.QueryParams(k=w.k, theta=0.8, depth_mode=B.DEPTH_FIXED, cont_len=w.cont_len)
    a, b = one.query(q, pr).cpu(), sharded_query(shards, q, pr)
    assert torch.equal(a.idx.to(torch.int64), b.gidx.cpu())
    assert torch.equal(a.cont_tok, b.cont_tok.cpu()) and torch.equal(a.fired, b.fired.cpu())
    assert torch.allclose(a.score, b.score.cpu(), atol=1e-6)
    # depth by rank is a matter of the merged order: a shard cannot assign it
    with pytest.raises(ValueError):
        sharded_query(shards, q, B.QueryParams(k=w.k, depth_mode=B.DEPTH_RANKED, cont_len=w.cont_len))


def test_exact_ties_across_shards_resolve_to_the_lowest_global_position():
    d = 64
    shards = [S.ShardedPool(d, 64) for _ in range(3)]
    row = torch.randn(1, d, device="cuda").to(torch.bfloat16)
    other = torch.randn(4, d, device="cuda").to(torch.bfloat16)
    tok = lambda n, b: torch.arange(b, b + n, dtype=torch.int32, device="cuda")
    # the same state stored at global positions 9 (shard 2), 4 (shard 0) and 20 (shard 1)
    shards[2].append(torch.cat([other[:1], row, other[1:2]]), tok(3, 80), global_row=8)
    shards[0].append(torch.cat([row, other[2:]]), tok(3, 40), global_row=4)
    shards[1].append(torch.cat([other[:2], row]), tok(3, 180), global_row=18)
    pr = B.QueryParams(k=3, theta=0.8, depth_mode=B.DEPTH_FIXED, cont_len=2, offset=1)
    out = sharded_query(shards, row, pr)
    assert out.gidx[0].tolist() == [4, 9, 20]
    assert out.score[0, 0] == out.score[0, 1] == out.score[0, 2]
    assert out.cont_tok[0].tolist() == [[41, 42], [82, -1], [-1, -1]] and out.fired[0] == 1
    assert out.cont_len[0].tolist() == [2, 1, 0]
    # not fired: neighbours are still reported, nothing is copied
    cold = sharded_query(shards, other[3:4].contiguous(),
                         B.QueryParams(k=3, theta=1.5, depth_mode=B.DEPTH_FIXED, cont_len=2))
    assert cold.fired[0] == 0 and torch.all(cold.cont_len == 0) and torch.all(cold.cont_tok == -1)
    assert cold.gidx[0, 0] >= 0


def test_fewer_rows_than_k_and_empty_shards():
    d = 64
    shards = [S.ShardedPool(d, 16) for _ in range(4)]
    st = torch.randn(3, d, device="cuda").to(torch.bfloat16)
    shards[1].append(st[:2].contiguous(), torch.tensor([5, 6], dtype=torch.int32, device="cuda"), 0)
    shards[3].append(st[2:].contiguous(), torch.tensor([7], dtype=torch.int32, device="cuda"), 2)
    out = sharded_query(shards, st[2:3].contiguous(),
                        B.QueryParams(k=5, theta=-2.0, depth_mode=B.DEPTH_FIXED, cont_len=2))
    assert out.gidx[0, 0] == 2 and sorted(out.gidx[0, :3].tolist()) == [0, 1, 2]
    assert out.gidx[0, 3:].tolist() == [-1, -1] and torch.all(torch.isinf(out.score[0, 3:]))
