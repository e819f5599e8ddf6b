"""Full-size benchmark configurations on the GPU against the CPU oracle.

C3 and C4 are checked with the whole pool in the oracle (C4 on a subset of its 64
queries: the oracle needs about a second per query at a million rows).  C5 (17-34 GB of
keys) is checked on sampled rows: the oracle is run, unchanged, on a small pool made of
the rows the GPU returned, the planted rows and a random sample of the rest; every
property that holds for the full pool restricted to those rows is asserted.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import GAP, SCORE_BUG, check_query, fill_both, oracle_params

pytestmark = pytest.mark.gpu


def fixed(k, L, theta=0.8, **kw):
    return B.QueryParams(k=k, theta=theta, depth_mode=B.DEPTH_FIXED, cont_len=L, **kw)


@pytest.mark.parametrize("key_format", ["bf16", "e4m3"])
def test_c2_full_size_in_the_launch_configuration_the_bench_times(key_format):
    # bench.py's step on its default workload: oilbird_pool_step on the full C2 pool, the
    # 8 rows committed since the last step appended inside the scan kernel, one query, path
    # chosen by the library.  Every step's output is checked against the oracle, and the
    # stored rows at the end.
    w = W.C2
    pool, ora = fill_both(w, spare_rows=256, max_nq=w.nq, max_k=w.k, max_append=8,
                          key_format=key_format)
    q, meta = w.queries("cuda")
    g = torch.Generator(device="cuda").manual_seed(2)
    launches0 = pool.launch_count
    for step in range(6):
        st = torch.randn(8, w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, w.vocab, (8,), generator=g, device="cuda", dtype=torch.int32)
        qs = q.clone()
        if step % 2:
            qs[0] = st[5]                       # every other step asks for a row of this step
        pr = fixed(w.k, w.cont_len, theta=(0.8 if step < 3 else -2.0))
        out = pool.step(st, tk, qs, pr, tag=1_000_000 + step)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=1_000_000 + step)
        check_query(out, ora, W.to_bits(qs), pr)
        if step % 2:
            assert int(out.idx[0, 0]) == len(pool) - 3
        elif "planted_row" in meta:
            assert int(out.idx[0, 0]) == meta["planted_row"]
    assert len(pool) == w.n_rows + 48 and pool.stats()["stalled"] == 0
    assert pool.launch_count - launches0 == 12      # two kernels per step: scan, merge + gather
    _, tok, tid = pool.read_rows(w.n_rows, 48)
    assert np.array_equal(tok, ora.tokens[w.n_rows:]) and np.array_equal(tid, ora.trace_ids[w.n_rows:])
    if key_format == "bf16":
        keys, _, _ = pool.read_rows(w.n_rows, 48)
        assert np.array_equal(keys, ora.keys[w.n_rows:])
    else:
        codes, scales = pool.read_codes(w.n_rows, 48)
        assert np.array_equal(codes, ora.codes[w.n_rows:])
        assert np.array_equal(scales.view(np.uint32), ora.scales[w.n_rows:].view(np.uint32))


def test_c3_tool_calling_shape_full_size():
    w = W.C3
    pool, ora = fill_both(w)
    q, meta = w.queries("cuda")
    for theta in (0.8, -2.0):
        pr = fixed(w.k, w.cont_len, theta=theta)
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr)
    o = pool.query(q, fixed(w.k, w.cont_len, theta=-2.0)).cpu()
    # recall of the planted same-(template, position) rows and matched continuation length
    hits = tot = 0
    matched = []
    for i, rows in enumerate(meta["planted_rows"]):
        got = set(o.idx[i].tolist())
        hits += len(set(rows) & got)
        tot += min(len(rows), w.k)
        ttok, slot = meta["template_tokens"][i]
        pos = meta["pos"][i]
        want = ttok[pos + 2: pos + 2 + w.cont_len]
        ok = (o.cont_tok[i, 0, : len(want)] == want) | slot[pos + 2: pos + 2 + w.cont_len]
        matched.append(int(ok.sum()))
    assert hits / tot > 0.9
    # away from slot positions the continuation is the template's own next tokens
    assert np.mean(matched) > 0.9 * w.cont_len
    assert pool.stats()["stalled"] == 0


def test_c4_batched_shared_pool_full_size_sampled_queries():
    w = W.C4
    pool, ora = fill_both(w)
    q, meta = w.queries("cuda")
    pr = fixed(w.k, w.cont_len, theta=-2.0)
    out = pool.query(q, pr)                     # all 64 queries on the tensor path
    o = out.cpu()
    assert o.idx[0, 0] == meta["planted_row"]
    sel = [0, 1, 31, 63]                        # the oracle scores these four
    sub = B.QueryOut(o.idx[sel], o.score[sel], o.fired[sel], o.cont_len[sel], o.cont_tok[sel])
    st = check_query(sub, ora, W.to_bits(q)[sel], pr)
    assert st["max_score_err"] < SCORE_BUG
    # the CUDA-core path agrees on one of them
    one = pool.query(q[1:2].contiguous(), fixed(w.k, w.cont_len, theta=-2.0, path=B.PATH_GEMV))
    check_query(one, ora, W.to_bits(q)[1:2], pr)
    # separated variant: index sets must be identical
    del pool, ora
    torch.cuda.empty_cache()
    ws = w.scaled(n_rows=262144).separated()
    pool, ora = fill_both(ws)
    q, _ = ws.queries("cuda")
    st = check_query(pool.query(q, fixed(ws.k, ws.cont_len)), ora, W.to_bits(q), fixed(ws.k, ws.cont_len))
    assert st["strict_sets"] >= ws.nq // 2       # most rank-k gaps exceed the tie band
    assert pool.stats()["stalled"] == 0


def sampled_check(pool, w, C, q, out, n_rows, extra_rows, rng, params):
    """Oracle on {returned rows} U extra_rows U random sample; see module docstring."""
    o = out.cpu()
    idx = o.idx.numpy()
    nq, k = idx.shape
    rows = set(idx[idx >= 0].tolist()) | set(extra_rows)
    rows |= set(rng.integers(0, n_rows, size=1500).tolist())
    rows = np.array(sorted(rows))
    ora = OraclePool(w.d)
    by_trace = {}
    for r in rows:
        by_trace.setdefault(int(r) // w.rows_per_trace, []).append(int(r))
    hits_by_trace = {}
    for qi in range(nq):
        for j in range(k):
            if idx[qi, j] >= 0 and o.fired[qi]:
                hits_by_trace.setdefault(int(idx[qi, j]) // w.rows_per_trace, []).append((qi, j))
    order = []
    for t, rr in sorted(by_trace.items()):
        st, tk, tag = w.trace(t, "cuda", C)
        loc = torch.tensor([r - t * w.rows_per_trace for r in rr], device="cuda")
        ora.append(W.to_bits(st[loc]), tk[loc].cpu().numpy(), tag=tag)
        order += rr
        # gather is checked against the regenerated token stream of the neighbour's trace
        tk_host = tk.cpu().tolist()
        for qi, j in hits_by_trace.get(t, ()):
            s0 = int(idx[qi, j]) - t * w.rows_per_trace + params.offset
            want = tk_host[s0: s0 + params.cont_len]          # clipped at the trace end
            assert o.cont_len[qi, j] == len(want)
            assert o.cont_tok[qi, j].tolist() == want + [-1] * (params.cont_len - len(want))
    order = np.array(order)
    # keys of the sampled rows are bit-identical to the oracle's
    pos = {int(g): i for i, g in enumerate(order)}
    for g in list(idx[0, :4]) + list(extra_rows)[:4]:
        keys, _, _ = pool.read_rows(int(g), 1)
        assert np.array_equal(keys[0], ora.keys[pos[int(g)]])
    ref = ora.query(W.to_bits(q), oracle_params(params), want_all_scores=True)
    for qi in range(nq):
        s_loc = ref.all_scores[qi]
        got = idx[qi]
        loc = np.array([pos[int(g)] for g in got])
        err = np.abs(o.score[qi].numpy() - s_loc[loc])
        assert err.max() < SCORE_BUG
        # nothing in the sample beats the k-th returned score by more than the tie band
        kth = float(o.score[qi, -1])
        better = order[np.where(s_loc > kth + GAP)[0]]
        assert set(better.tolist()) <= set(got.tolist())
        assert np.all(np.diff(o.score[qi].numpy()) <= 0)
        assert len(set(got.tolist())) == k


@pytest.mark.parametrize("nq", [1, 8, 64, 256])
def test_c5_streaming_large_width(nq):
    w = W.C5
    steps_a, steps_b = 6, 6
    n_start, n_end = W.C5_START_ROWS, w.n_rows
    pool = B.Pool(w.d, n_end, max_nq=nq, max_k=w.k, max_traces=w.num_traces + 8)
    C = w._centroids("cuda")
    rng = np.random.default_rng(nq)
    g = torch.Generator(device="cuda").manual_seed(1000 + nq)
    pr = fixed(w.k, w.cont_len)
    t = 0

    def append_trace():
        nonlocal t
        st, tk, tag = w.trace(t, "cuda", C)
        pool.append(st, tk, tag=tag)
        t += 1
        return st

    def step(check):
        st = append_trace()
        n_rows = len(pool)
        q, _ = w.queries("cuda", nq=nq, step=t)
        r = int(rng.integers(0, st.shape[0]))
        q[nq - 1] = (st[r].float() + 0.05 * torch.randn(w.d, generator=g, device="cuda")).to(
            torch.bfloat16)
        out = pool.query(q, pr)                               # no synchronisation in between
        assert out.cpu().idx[nq - 1, 0] == n_rows - st.shape[0] + r, "appended row not visible"
        if check:
            extra = [n_rows - st.shape[0] + r]
            sampled_check(pool, w, C, q, out, n_rows, extra, rng, pr)

    while len(pool) < n_start:
        append_trace()
    for i in range(steps_a):
        step(check=(i in (0, steps_a - 1)))
    while len(pool) < n_end - steps_b * w.rows_per_trace:
        append_trace()
    for i in range(steps_b):
        step(check=(i == steps_b - 1))
    assert len(pool) == n_end
    assert pool.stats() == dict(degenerate_rows=0, nonfinite_queries=0, stalled=0)
