"""oilbird_query_static: the query entry point that allocates nothing.

It exists for hosts that hold all device memory themselves (a serving engine that took
the whole GPU at start-up, say) and therefore cannot let this library allocate its
scratch: the candidate lists live in a fixed array inside the library instead.  The test
calls it through the C-ABI on pool arrays held in torch tensors and requires the very
same results as oilbird_pool_query on the same pool, on two calls in a row (the second
with other sizes, so that contents left by the first call would show), and checks the same
results against the CPU oracle directly.  The file is named so that pytest collects it
last; it passes alone in a fresh process and after the others.
"""
import numpy as np
import pytest
import torch

from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query

pytestmark = pytest.mark.gpu

FIELDS = ("idx", "score", "fired", "cont_len", "cont_tok")


def test_static_query_matches_pool_query_on_two_calls_in_a_row():
    w = W.C1.scaled(n_rows=3000, d=512, nq=2, seed=77)
    pool, ora = B.Pool(w.d, w.n_rows), OraclePool(w.d)
    for st, tk, tag in w.traces("cuda"):
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    # the caller's own copy of the pool arrays, in the layout append produces
    keys, tok, tid = pool.read_rows()
    _, ends, _ = pool.traces()
    keys_t = torch.from_numpy(keys.view(np.int16)).view(torch.bfloat16).cuda()
    tok_t, tid_t = torch.from_numpy(tok).cuda(), torch.from_numpy(tid).cuda()
    end_t = torch.from_numpy(ends.astype(np.int32)).cuda()
    q, _ = w.queries("cuda")
    calls = [
        (q, B.QueryParams(k=64, theta=-2.0, depth_mode=B.DEPTH_FIXED, cont_len=12,
                          path=B.PATH_GEMV)),
        (q[1:2].contiguous(), B.QueryParams(k=8, cont_len=48, path=B.PATH_GEMV)),   # paper defaults
    ]
    for qq, pr in calls:
        want = pool.query(qq, pr).cpu()
        out = B.QueryOut.empty(qq.shape[0], pr.k, pr.cont_len, "cuda")
        for t in (out.idx, out.fired, out.cont_len, out.cont_tok):
            t.fill_(-7)                                  # every output word must be written
        got = B.query_static(keys_t, tok_t, tid_t, end_t, qq, pr, out=out)
        check_query(got, ora, W.to_bits(qq), pr)           # the oracle, not only the other entry point
        got = got.cpu()
        for f in FIELDS:
            a, b = getattr(got, f), getattr(want, f)
            if f == "score":
                assert torch.allclose(a, b, atol=5e-5, rtol=0) and torch.equal(a, b)
            else:
                assert torch.equal(a, b), f


def test_static_query_rejects_what_does_not_fit():
    keys = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(64, dtype=torch.int32, device="cuda")
    end = torch.tensor([64], dtype=torch.int32, device="cuda")
    q3 = torch.zeros(3, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OilbirdError) as e:
        B.query_static(keys, z, z, end, q3, B.QueryParams(k=8, cont_len=4))
    assert e.value.code == B.EINVAL and "at most 2 queries" in str(e.value)
    with pytest.raises(B.OilbirdError) as e:
        B.query_static(keys, z, z, end, q3[:1].contiguous(), B.QueryParams(k=129, cont_len=4))
    assert e.value.code == B.EINVAL and "neighbours" in str(e.value)
    # an empty pool is legal: no neighbours
    out = B.query_static(keys[:0], z[:0], z[:0], end, q3[:1].contiguous(),
                         B.QueryParams(k=4, cont_len=4)).cpu()
    assert torch.all(out.idx == -1) and out.fired[0] == 0 and torch.all(out.cont_tok == -1)
