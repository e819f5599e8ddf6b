"""GPU parity for the coarse index: the CUDA index against oracle/index.py on the same pool,
centroids and queries.  Assignments and lists are integers and must be identical (the
workloads keep the best two centroids of every row well apart, so accumulation order
cannot decide); answers go through the acceptance rule of every other query test, applied to
the oracle's candidate-restricted scores."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OraclePool
from oracle.index import OracleIndex
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import GAP, SCORE_BUG, fill_both, oracle_params

pytestmark = pytest.mark.gpu


def fixed(k, L, theta=-2.0, **kw):
    return B.QueryParams(k=k, theta=theta, depth_mode=B.DEPTH_FIXED, cont_len=L, **kw)


def check_index_query(out, oidx: OracleIndex, q_bits, n_probe, params, exclude=None):
    """check_query's rule with the oracle's scores masked to the candidate rows."""
    o = out.cpu()
    idx, score = o.idx.numpy(), o.score.numpy()
    ref = oidx.query(q_bits, n_probe, oracle_params(params, exclude), want_all_scores=True)
    nq, k = idx.shape
    for q in range(nq):
        s_all = ref.all_scores[q]
        kk = min(k, int(np.sum(np.isfinite(s_all))))
        got = idx[q]
        assert np.all(got[kk:] == -1) and np.all(np.isneginf(score[q, kk:]))
        assert len(set(got[:kk].tolist())) == kk
        if kk:
            assert np.all(np.isfinite(s_all[got[:kk]])), "a row outside the probed lists was returned"
            err = np.abs(score[q, :kk].astype(np.float64) - s_all[got[:kk]])
            assert err.max() <= SCORE_BUG
            s_k = float(ref.score[q, kk - 1])
            assert np.all(s_all[got[:kk]] >= s_k - GAP)
            must = np.where(s_all > s_k + GAP)[0]
            assert set(must.tolist()) <= set(got[:kk].tolist())
            for j in range(1, kk):
                assert score[q, j - 1] > score[q, j] or (score[q, j - 1] == score[q, j] and got[j - 1] < got[j])
            if abs(float(ref.score[q, 0]) - params.theta) > GAP:
                assert o.fired[q] == ref.fired[q]
        for j in range(k):
            dep = 0
            if o.fired[q] and got[j] >= 0:
                dep = (params.cont_len if params.depth_mode == B.DEPTH_FIXED
                       else oracle.depth_by_rank(j, params.tier_depth) if params.depth_mode == B.DEPTH_RANKED
                       else oracle.depth(float(score[q, j]), params.tier_thr, params.tier_depth))
            tok, n = oidx.pool.gather_one(int(got[j]), dep, params.offset, params.cont_len)
            assert o.cont_len[q, j] == n and np.array_equal(o.cont_tok[q, j].numpy(), tok)
    return ref


def build_both(w, n_lists, seed=0, **pool_kw):
    pool, ora = fill_both(w, **pool_kw)
    # centroids: stored states of the pool, drawn at random (a sample of traffic)
    g = np.random.default_rng(seed)
    rows = np.sort(g.choice(w.n_rows, n_lists, replace=False))
    raw = []
    for r in rows:
        t, i = divmod(int(r), w.rows_per_trace)
        raw.append(w.trace(t, "cuda")[0][i])
    cent = torch.stack(raw).contiguous()
    gix, oix = B.Index(pool, cent), OracleIndex(ora, W.to_bits(cent))
    return pool, ora, gix, oix


def same_lists(gix, oix):
    a, off, rows = gix.read()
    assert np.array_equal(a, oix.assign.astype(np.int32))
    want = oix.lists()
    assert off[0] == 0 and off[-1] == oix.n_indexed
    for l in range(oix.n_lists):
        assert sorted(rows[off[l]:off[l + 1]].tolist()) == want[l].tolist()


@pytest.mark.parametrize("d,n_lists", [(256, 24), (1024, 64)])
def test_lists_and_answers_match_the_oracle(d, n_lists):
    w = W.C1.scaled(n_rows=6000, d=d, nq=5, k=8, cont_len=4, n_centroids=40, rows_per_trace=500)
    pool, ora, gix, oix = build_both(w, n_lists, spare_rows=600)
    gix.refresh(); oix.refresh()
    assert len(gix) == 6000
    same_lists(gix, oix)
    q, _ = w.queries("cuda")
    for n_probe in (1, 3, n_lists, n_lists + 7):
        for k in (1, 8, 40):
            pr = fixed(k, 4, theta=0.8 if k == 8 else -2.0)
            check_index_query(gix.query(q, n_probe, pr), oix, W.to_bits(q), n_probe, pr)
    # every list probed: the full scan's own answer, bit for bit
    pr = fixed(8, 4)
    a, b = gix.query(q, n_lists, pr).cpu(), pool.query(q, pr).cpu()
    assert torch.equal(a.idx, b.idx) and torch.equal(a.cont_tok, b.cont_tok)
    assert torch.allclose(a.score, b.score, atol=SCORE_BUG, rtol=0)
    # rows appended after the refresh are found without one (the tail), then move into lists
    g = torch.Generator(device="cuda").manual_seed(3)
    st = torch.randn(300, d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(300, dtype=torch.int32, device="cuda")
    pool.append(st, tk, tag=77)
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=77)
    q2 = torch.cat([st[17:18], q[:2]]).contiguous()
    out = gix.query(q2, 1, fixed(4, 4))
    assert int(out.idx[0, 0]) == 6017
    check_index_query(out, oix, W.to_bits(q2), 1, fixed(4, 4))
    gix.refresh(); oix.refresh()
    assert len(gix) == 6300
    same_lists(gix, oix)
    check_index_query(gix.query(q2, 2, fixed(4, 4)), oix, W.to_bits(q2), 2, fixed(4, 4))
    # exclusion tags
    ex = np.array([77, 0, 3], dtype=np.uint64)
    pr = fixed(6, 4, exclude_tag=torch.from_numpy(ex.view(np.int64)).cuda())
    check_index_query(gix.query(q2, 4, pr), oix, W.to_bits(q2), 4, pr, exclude=ex)
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("nq", [1, 2, 3, 4])
def test_lookups_in_one_launch_match_the_oracle_and_the_separate_launches(nq):
    # a single query's lookup is one launch (centroids, probes, candidates, merge and gather);
    # batches, and an explicit scan path, take the separate launches
    w = W.C1.scaled(n_rows=9000, d=512, nq=nq, k=8, cont_len=4, n_centroids=40, rows_per_trace=500, seed=21)
    pool, ora, gix, oix = build_both(w, 48, seed=5, spare_rows=400, max_k=128)
    gix.refresh(); oix.refresh()
    g = torch.Generator(device="cuda").manual_seed(8)
    st = torch.randn(130, 512, generator=g, device="cuda").to(torch.bfloat16)     # a tail
    tk = torch.arange(130, dtype=torch.int32, device="cuda")
    pool.append(st, tk, tag=99)
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=99)
    q, _ = w.queries("cuda")
    q[nq - 1] = st[11]                                       # one query whose best row is in the tail
    launches = pool.launch_count
    for n_probe in (1, 3, 31, 48):
        for k in (1, 8, 40, 100):
            pr = fixed(k, 4, theta=0.8 if k == 8 else -2.0)
            one = gix.query(q, n_probe, pr)
            check_index_query(one, oix, W.to_bits(q), n_probe, pr)
            sep = gix.query(q, n_probe, fixed(k, 4, theta=pr.theta, path=B.PATH_GEMV))
            a, b = one.cpu(), sep.cpu()
            assert torch.equal(a.idx, b.idx) and torch.equal(a.cont_tok, b.cont_tok)
            assert torch.equal(a.fired, b.fired) and torch.equal(a.cont_len, b.cont_len)
            assert torch.allclose(a.score, b.score, atol=SCORE_BUG, rtol=0)
    assert int(gix.query(q, 1, fixed(4, 4)).idx[nq - 1, 0]) == 9011
    # a single query is one launch per lookup up to 32 probes (12 above, one here); more
    # probes, batches, and lookups that name a scan path are two on this pool (+ two on the
    # centroids' own)
    fused = 1 if nq == 1 else 2
    assert pool.launch_count - launches == (12 + 1) * fused + 4 * 2 + 16 * 2, "the one-launch form was not taken"
    # exclusion tags and a query that is not finite
    ex = np.zeros(nq, dtype=np.uint64); ex[0] = 99; ex[-1] = 99
    pr = fixed(6, 4, exclude_tag=torch.from_numpy(ex.view(np.int64)).cuda())
    check_index_query(gix.query(q, 4, pr), oix, W.to_bits(q), 4, pr, exclude=ex)
    bad = q.clone(); bad[0, 5] = float("nan")
    out = gix.query(bad, 4, fixed(8, 4)).cpu()
    assert out.idx[0].tolist() == [-1] * 8 and int(out.fired[0]) == 0 and out.cont_len[0].sum() == 0
    if nq > 1:
        good = gix.query(q, 4, fixed(8, 4)).cpu()
        assert torch.equal(out.idx[1:], good.idx[1:])
    # the words the CTAs of a lookup meet at are left clear: the same lookup as a CUDA graph,
    # replayed, gives the same answer every time
    pr = fixed(8, 4)
    want = gix.query(q, 3, pr).cpu()
    out = gix.query(q, 3, pr)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        gix.query(q, 3, pr, out=out)
        s.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=s):
            for _ in range(3):
                gix.query(q, 3, pr, out=out)
        for _ in range(4):
            out.idx.fill_(-7)
            gr.replay()
            s.synchronize()
            assert torch.equal(out.idx.cpu(), want.idx) and torch.equal(out.cont_tok.cpu(), want.cont_tok)
    assert pool.stats()["stalled"] == 0 and pool.status() == B.OK


@pytest.mark.parametrize("key_format", ["bf16", "e4m3"])
def test_one_launch_lookup_at_the_widest_rows_and_longest_lists(key_format):
    # d = 8192 (a row is more than one round of a lane's loads), k up to 128 (four registers of
    # list per lane), 32 probes (the most the one-launch form takes)
    w = W.C1.scaled(n_rows=3000, d=8192, nq=1, k=8, cont_len=4, n_centroids=40, rows_per_trace=500, seed=23)
    pool, ora, gix, oix = build_both(w, 40, seed=6, spare_rows=100, max_k=128, key_format=key_format)
    gix.refresh(); oix.refresh()
    same_lists(gix, oix)
    q, _ = w.queries("cuda")
    launches = pool.launch_count
    for n_probe, k in ((1, 64), (7, 128), (32, 128), (32, 33)):
        pr = fixed(k, 4)
        one = gix.query(q, n_probe, pr)
        check_index_query(one, oix, W.to_bits(q), n_probe, pr)
        sep = gix.query(q, n_probe, fixed(k, 4, path=B.PATH_GEMV)).cpu()
        assert torch.equal(one.cpu().idx, sep.idx) and torch.equal(one.cpu().score, sep.score)
    assert pool.launch_count - launches == 4 * (1 + 2)
    assert pool.stats()["stalled"] == 0


def test_index_after_eviction_needs_a_reset():
    w = W.C1.scaled(n_rows=2000, d=128, nq=3, k=4, cont_len=2, rows_per_trace=250)
    pool, ora, gix, oix = build_both(w, 16, spare_rows=1000)
    gix.refresh(); oix.refresh()
    pool.evict_oldest(2); ora.evict_oldest(2)
    q, _ = w.queries("cuda")
    with pytest.raises(B.OilbirdError) as e:
        gix.query(q, 2, fixed(4, 2))
    assert e.value.code == B.EINVAL
    # growing back past the indexed size does not make the old row numbers right again
    g = torch.Generator(device="cuda").manual_seed(8)
    for tag in (501, 502, 503):
        st = torch.randn(250, w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.arange(250, dtype=torch.int32, device="cuda")
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    assert len(pool) > len(gix)
    for call in (lambda: gix.query(q, 2, fixed(4, 2)), gix.refresh):
        with pytest.raises(B.OilbirdError) as e:
            call()
        assert e.value.code == B.EINVAL
    gix.reset(); oix.reset()
    # everything is tail now: the full scan's answer whatever is probed
    pr = fixed(4, 2)
    a, b = gix.query(q, 1, pr).cpu(), pool.query(q, pr).cpu()
    assert torch.equal(a.idx, b.idx)
    gix.refresh(); oix.refresh()
    same_lists(gix, oix)
    check_index_query(gix.query(q, 3, pr), oix, W.to_bits(q), 3, pr)


def test_c2_shaped_pool_recall_and_candidate_volume():
    # the single-request configuration at a quarter of its size: 512 centroids' worth of
    # traffic, 256 lists from a sample of stored states
    w = W.C2.scaled(n_rows=16384)
    pool, ora, gix, oix = build_both(w, 256)
    gix.refresh(); oix.refresh()
    same_lists(gix, oix)
    q, meta = w.queries("cuda", nq=4)
    pr = fixed(w.k, w.cont_len)
    exact = pool.query(q, pr).cpu()
    hits = []
    for n_probe in (1, 4, 16, 256):
        out = gix.query(q, n_probe, pr)
        check_index_query(out, oix, W.to_bits(q), n_probe, pr)
        o = out.cpu()
        hits.append(np.mean([len(set(o.idx[i].tolist()) & set(exact.idx[i].tolist())) / w.k
                             for i in range(4)]))
    assert hits == sorted(hits) and hits[-1] == 1.0


def test_bad_arguments_are_refused():
    cent = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    pool = B.Pool(64, 100)
    with pytest.raises(B.OilbirdError) as e:
        B.Index(pool, torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda"))   # no lists
    assert e.value.code == B.EINVAL
    ix = B.Index(pool, cent)
    q = torch.zeros(1, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OilbirdError):
        ix.query(q, 0, fixed(4, 2))                          # at least one probe
    out = ix.query(q, 2, fixed(4, 2)).cpu()                  # an empty pool is legal
    assert torch.all(out.idx == -1) and out.fired[0] == 0


def test_index_over_an_8bit_pool_matches_the_oracle():
    """Codes and scales in place of keys: rows are assigned through their dequantised form
    (fp32(value(code) * scale), rounded to bf16 as a query), candidates are scored by the 8-bit
    pool's own rule, training takes the means of the dequantised elements."""
    w = W.C1.scaled(n_rows=6000, nq=5, d=256, k=8, cont_len=4, n_centroids=24, rows_per_trace=500, seed=41)
    pool, ora = fill_both(w, key_format="e4m3", spare_rows=300, max_nq=16, max_k=128)
    assign = np.concatenate([w.trace_assign(t, "cuda").cpu().numpy() for t in range(w.num_traces)])[: w.n_rows]
    first = [int(np.nonzero(assign == c)[0][0]) for c in range(24)]      # one row of every cluster
    keys_raw = torch.cat([st for st, _, _ in w.traces("cuda")])[: w.n_rows]
    cent = keys_raw[first].contiguous()
    gix, oix = B.Index(pool, cent), OracleIndex(ora, W.to_bits(cent))
    gix.refresh(); oix.refresh()
    assert len(gix) == 6000
    same_lists(gix, oix)
    q, _ = w.queries("cuda")
    for n_probe in (1, 3, 24, 30):
        for k in (1, 8, 40):
            pr = fixed(k, 4, theta=0.8 if k == 8 else -2.0)
            check_index_query(gix.query(q, n_probe, pr), oix, W.to_bits(q), n_probe, pr)
    # every list probed: the 8-bit pool's own full scan (single queries share its arithmetic)
    pr = fixed(8, 4)
    for i in range(2):
        a, b = gix.query(q[i:i + 1].contiguous(), 24, pr).cpu(), pool.query(q[i:i + 1].contiguous(), pr).cpu()
        assert torch.equal(a.idx, b.idx) and torch.equal(a.score, b.score) and torch.equal(a.cont_tok, b.cont_tok)
    # a single query's lookup is one launch here too: same neighbours as the separate launches
    launches = pool.launch_count
    for n_probe in (1, 3, 30):
        for k in (1, 8, 100):
            q1 = q[2:3].contiguous()
            one = gix.query(q1, n_probe, fixed(k, 4))
            check_index_query(one, oix, W.to_bits(q1), n_probe, fixed(k, 4))
            sep = gix.query(q1, n_probe, fixed(k, 4, path=B.PATH_GEMV)).cpu()
            assert torch.equal(one.cpu().idx, sep.idx) and torch.equal(one.cpu().score, sep.score)
            assert torch.equal(one.cpu().cont_tok, sep.cont_tok)
    assert pool.launch_count - launches == 9 * (1 + 2)
    # the tail, then a refresh; exclusion tags
    g = torch.Generator(device="cuda").manual_seed(3)
    st = torch.randn(200, w.d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(200, dtype=torch.int32, device="cuda")
    pool.append(st, tk, tag=77)
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=77)
    q2 = torch.cat([st[17:18], q[:2]]).contiguous()
    out = gix.query(q2, 1, fixed(4, 4))
    assert int(out.idx[0, 0]) == 6017
    check_index_query(out, oix, W.to_bits(q2), 1, fixed(4, 4))
    gix.refresh(); oix.refresh()
    same_lists(gix, oix)
    ex = np.array([77, 0, 3], dtype=np.uint64)
    pr = fixed(6, 4, exclude_tag=torch.from_numpy(ex.view(np.int64)).cuda())
    check_index_query(gix.query(q2, 4, pr), oix, W.to_bits(q2), 4, pr, exclude=ex)
    # training: raw centroids, assignments and lists identical after one and three iterations
    done = 0
    for upto in (1, 3):
        gix.train(upto - done); oix.train(upto - done)
        done = upto
        assert np.array_equal(gix.centroids(), oix.cent_raw)
        same_lists(gix, oix)
    check_index_query(gix.query(q, 3, fixed(8, 4)), oix, W.to_bits(q), 3, fixed(8, 4))
    assert pool.stats()["stalled"] == 0


def test_training_matches_the_oracle_bit_for_bit():
    """Lloyd's iterations: raw centroids, assignments and lists identical to the oracle's after
    one, two and five iterations (one starting centroid in each cluster of the recipe, so
    that no row sits between two centroids), then answers under the acceptance rule."""
    w = W.C1.scaled(n_rows=6000, nq=6, d=256, n_centroids=24, rows_per_trace=500, seed=31)
    pool, ora = fill_both(w, max_nq=16)
    assign = np.concatenate([w.trace_assign(t, "cuda").cpu().numpy() for t in range(w.num_traces)])[: w.n_rows]
    first = [int(np.nonzero(assign == c)[0][0]) for c in range(24)]      # one row of every cluster
    keys_raw = torch.cat([st for st, _, _ in w.traces("cuda")])[: w.n_rows]
    cent = keys_raw[first].contiguous()
    gix, oix = B.Index(pool, cent), OracleIndex(ora, W.to_bits(cent))
    assert np.array_equal(gix.centroids(), oix.cent_raw)
    done = 0
    for upto in (1, 2, 5):
        gix.train(upto - done)
        oix.train(upto - done)
        done = upto
        assert np.array_equal(gix.centroids(), oix.cent_raw)
        same_lists(gix, oix)
        assert len(gix) == len(pool)
    q, _ = w.queries("cuda")
    for n_probe in (1, 3, 24):
        pr = fixed(8, 4)
        check_index_query(gix.query(q, n_probe, pr), oix, W.to_bits(q), n_probe, pr)
    # zero iterations only rebuild the lists; an empty pool has nothing to learn from
    gix.train(0)
    same_lists(gix, oix)
    empty = B.Pool(w.d, 64)
    eix = B.Index(empty, cent)
    eix.train(3)
    assert len(eix) == 0 and np.array_equal(eix.centroids(), W.to_bits(cent))


def test_training_on_fewer_lists_than_clusters_keeps_the_index_exact_and_helps_recall():
    w = W.C1.scaled(n_rows=20000, nq=32, k=8, d=128, n_centroids=96, rows_per_trace=1000, seed=32)
    pool, ora, gix, oix = build_both(w, 20, seed=3, max_nq=32)
    q, _ = w.queries("cuda")
    pr = fixed(8, 4)
    exact = pool.query(q, fixed(8, 4, path=B.PATH_GEMV)).cpu()    # (the index scores on the CUDA cores)
    gix.refresh()

    def recall(n_probe):
        got = gix.query(q, n_probe, pr).cpu().idx.numpy()
        return float(np.mean([len(set(got[i]) & set(exact.idx[i].tolist())) / 8 for i in range(32)]))

    r_before = recall(1)
    gix.train(6)
    a, off, rows = gix.read()
    assert len(gix) == len(pool) and off[-1] == len(pool)
    assert sorted(rows.tolist()) == list(range(len(pool)))             # a partition of the rows
    full = gix.query(q, 20, pr).cpu()                                   # every list probed: the full scan
    assert torch.equal(full.idx, exact.idx) and torch.equal(full.score, exact.score)
    assert recall(1) >= r_before - 0.02
    # the same training twice gives the same centroids (nothing depends on scheduling)
    c1 = gix.centroids()
    pool2, _, gix2, _ = build_both(w, 20, seed=3, max_nq=32)
    gix2.train(6)
    assert np.array_equal(c1, gix2.centroids())
    assert pool.stats()["stalled"] == 0
