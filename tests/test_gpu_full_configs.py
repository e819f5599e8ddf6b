"""Full-size benchmark configurations on the GPU against the CPU oracle.

Every configuration is checked with the WHOLE pool in the oracle: C3 all queries, C4 on 16
of its 64 queries (the oracle needs about a second per query at a million rows), C5 (17 GB
of keys growing to 34 GB) on one to four queries of every batch size of its sweep at the
start of the stream and at its far end.  Where the host cannot hold a second copy of the C5
pool, and as a cross-check where it can, the oracle is also run, unchanged, on a small pool
made of the rows the GPU returned, ALL rows drawn around the query's centroid (the only rows
that can reach the top-k, see siblings_check) and a random sample of the rest.
"""
import numpy as np
import psutil
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
    sel = [0, 1, 2, 7, 8, 15, 16, 17, 31, 32, 33, 47, 48, 55, 62, 63]   # the oracle scores these
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


def take(out: B.QueryOut, sel) -> B.QueryOut:
    o = out.cpu()
    return B.QueryOut(o.idx[sel], o.score[sel], o.fired[sel], o.cont_len[sel], o.cont_tok[sel])


def siblings_check(pool, w, C, q, out, sel, q_centroid, assign, n_rows, extra_rows, rng, params):
    """The oracle on a sub-pool that holds every row that can matter.

    A clustered pool's rows are centroid + 0.2 * noise: two rows of the same centroid have
    cosine ~0.96, rows of different centroids ~N(0, 1/d) (sigma 0.011 at d = 8192).  The k
    best of a query are therefore rows of its own centroid as long as that centroid has at
    least k rows, and a row of another centroid would have to sit ~80 sigma out to reach
    them.  The sub-pool is: ALL rows of the selected queries' centroids (from the
    generator's labels, without materialising the pool), the rows the GPU returned, the rows
    in extra_rows and 1,500 random rows.  On it the unchanged oracle must reproduce the GPU's
    answer under the full acceptance rule (so a sibling the scan dropped fails the test),
    and the random rows must stay far below the k-th score (which is what makes the
    restriction to siblings exact rather than sampled).
    """
    o = take(out, sel)
    idx = o.idx.numpy()
    k = idx.shape[1]
    lab = torch.cat(assign)[:n_rows].cpu().numpy()
    rows = set(idx[idx >= 0].tolist()) | set(int(r) for r in extra_rows)
    sib = {}
    for j, qi in enumerate(sel):
        sib[j] = np.nonzero(lab == q_centroid[qi])[0]
        assert len(sib[j]) >= k, "centroid with fewer than k rows: the argument above does not apply"
        rows |= set(sib[j].tolist())
    rnd = rng.integers(0, n_rows, size=1500)
    rows |= set(rnd.tolist())
    rows = np.array(sorted(rows))
    ora = OraclePool(w.d)
    by_trace = {}
    for r in rows:
        by_trace.setdefault(int(r) // w.rows_per_trace, []).append(int(r))
    toks = {}
    for t, rr in sorted(by_trace.items()):
        st, tk, tag = w.trace(t, "cuda", C)
        loc = torch.tensor([r - t * w.rows_per_trace for r in rr], device="cuda")
        # one trace per sampled trace: a continuation never crosses into the next one
        ora.append(W.to_bits(st[loc]), tk[loc].cpu().numpy(), tag=tag)
        toks[t] = tk.cpu().tolist()
    pos = {int(g): i for i, g in enumerate(rows)}
    # stored keys of a few of those rows are bit-identical to the oracle's
    for g in list(idx[0, :3]) + [int(r) for r in list(extra_rows)[:2]]:
        keys, _, _ = pool.read_rows(int(g), 1)
        assert np.array_equal(keys[0], ora.keys[pos[int(g)]])
    # the GPU's answer, renumbered into the sub-pool (the order of rows is kept, so ties
    # break the same way), checked by the same rule as everywhere else but for the gather,
    # which is compared with the regenerated token stream of the neighbour's own trace
    ref = ora.query(W.to_bits(q)[sel], oracle_params(params), want_all_scores=True)
    for j, qi in enumerate(sel):
        s_loc = ref.all_scores[j]
        got = idx[j]
        loc = np.array([pos[int(g)] for g in got])
        assert np.abs(o.score[j].numpy() - s_loc[loc]).max() < SCORE_BUG
        assert len(set(got.tolist())) == k and np.all(np.diff(o.score[j].numpy()) <= 0)
        s_k = float(ref.score[j, k - 1])
        assert np.all(s_loc[loc] >= s_k - GAP), "a returned row is not among the k best"
        must = rows[np.where(s_loc > s_k + GAP)[0]]
        assert set(must.tolist()) <= set(got.tolist()), "a row that beats the k-th by more than the tie band is missing"
        # every row of another centroid in the sample is far below the k-th score
        other = np.array([pos[int(r)] for r in rnd if int(lab[int(r)]) != q_centroid[qi]])
        assert s_k - float(s_loc[other].max()) > 0.5
        for jj in range(k):
            t, r0 = divmod(int(got[jj]), w.rows_per_trace)
            want = (toks[t][r0 + params.offset: r0 + params.offset + params.cont_len]
                    if o.fired[j] else [])                    # clipped at the trace end
            assert o.cont_len[j, jj] == len(want)
            assert o.cont_tok[j, jj].tolist() == want + [-1] * (params.cont_len - len(want))


def test_c5_streaming_large_width_whole_pool_in_the_oracle():
    w = W.C5
    n_start, n_end = W.C5_START_ROWS, w.n_rows
    pr = fixed(w.k, w.cont_len)
    # the oracle keeps its own copy of the keys (uint16): 17 GB at the start, 34 GB at the end
    need = n_end * w.d * 2
    full = psutil.virtual_memory().available > need + (12 << 30)
    pool = B.Pool(w.d, n_end, max_nq=256, max_k=w.k, max_traces=w.num_traces + 8)
    ora = OraclePool(w.d) if full else None
    C = w._centroids("cuda")
    rng = np.random.default_rng(5)
    g = torch.Generator(device="cuda").manual_seed(1005)
    assign = []
    t = 0

    def append_trace():
        nonlocal t
        st, tk, tag = w.trace(t, "cuda", C)
        pool.append(st, tk, tag=tag)
        if ora is not None:
            ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
        assign.append(w.trace_assign(t, "cuda"))
        t += 1
        return st

    def step(nq, n_oracle):
        """One step of the stream (256 rows appended, nq queries, no synchronisation in
        between); n_oracle of the queries are checked against the whole-pool oracle."""
        st = append_trace()
        n_rows = len(pool)
        q, meta = w.queries("cuda", nq=nq, step=t)
        cent = list(meta["centroid"])
        r = int(rng.integers(0, st.shape[0]))
        q[nq - 1] = (st[r].float() + 0.05 * torch.randn(w.d, generator=g, device="cuda")).to(
            torch.bfloat16)
        cent[nq - 1] = int(assign[-1][r])
        out = pool.query(q, pr)
        assert out.cpu().idx[nq - 1, 0] == n_rows - st.shape[0] + r, "appended row not visible"
        if n_oracle == 0:
            return
        sel = sorted({nq - 1, 0, nq // 3, (2 * nq) // 3})[-n_oracle:]
        if ora is not None:
            assert len(ora) == n_rows
            stt = check_query(take(out, sel), ora, W.to_bits(q)[sel], pr)
            assert stt["max_score_err"] < SCORE_BUG
        extra = [n_rows - st.shape[0] + r]
        if meta["planted_row"] < n_rows:              # (drawn over the final size of the pool)
            extra.append(meta["planted_row"])
        siblings_check(pool, w, C, q, out, sel, cent, assign, n_rows, extra, rng, pr)

    while len(pool) < n_start:
        append_trace()
    # the start of the stream (N = 2^20 + a few steps): every batch size of the sweep
    for nq, n_oracle in ((1, 1), (8, 4), (64, 4), (256, 4), (1, 0), (256, 0)):
        step(nq, n_oracle)
    while len(pool) < n_end - 4 * w.rows_per_trace:
        append_trace()
    # the far end (N -> 2^21): the compact-list path (nq = 256, k = 64) where it is used,
    # and the single-request scan over 34 GB
    for nq, n_oracle in ((64, 2), (8, 0), (256, 4), (1, 1)):
        step(nq, n_oracle)
    assert len(pool) == n_end
    assert pool.stats() == dict(degenerate_rows=0, nonfinite_queries=0, stalled=0)
    print(f"C5: whole-pool oracle {'used' if full else 'NOT used (host memory)'}; "
          f"host memory available at start {psutil.virtual_memory().available / 2**30:.0f} GiB")
