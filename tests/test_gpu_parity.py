"""GPU parity tests: the CUDA pool (through the C-ABI) against the CPU oracle on the same
seeded inputs.  Integer results bit-exact, scores within the stated tolerances (see
tests/parity.py for the acceptance rule)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query, fill_both

pytestmark = pytest.mark.gpu

P1, M1 = 0x3F80, 0xBF80


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def fixed(k, L, theta=0.8, **kw):
    return B.QueryParams(k=k, theta=theta, depth_mode=B.DEPTH_FIXED, cont_len=L, **kw)


# ----------------------------------------------------------------- append (a1) ----

@pytest.mark.parametrize("d", [8, 200, 256, 4096, 8192])
def test_append_matches_oracle_bit_for_bit(d):
    g = torch.Generator(device="cuda").manual_seed(d)
    n = 300
    st = (torch.randn(n, d, generator=g, device="cuda") * 3).to(torch.bfloat16)
    st[7] = 0                                   # zero row
    st[11, d // 2] = float("inf")               # non-finite rows are stored as zero keys
    st[13, 0] = float("nan")
    # rows that leave the normal-number fast path of the normalisation: a subnormal element,
    # a negative zero, finite values near the top of the range (sum of squares above 2^256),
    # a row of subnormals only
    sub = torch.tensor([1, 0x7f, 0x8003], dtype=torch.int32).to(torch.int16).view(torch.bfloat16).cuda()
    st[20, 1] = sub[0]
    st[21, 0] = -0.0
    st[22] = 3.0e38
    st[22, d - 1] = -1.5e38
    st[23] = sub[1]
    st[23, d // 3] = sub[2]
    tk = torch.randint(0, 50000, (n,), generator=g, device="cuda", dtype=torch.int32)
    pool, ora = B.Pool(d, 1000), OraclePool(d)
    # three traces, the second extended in two pieces, one empty append in between
    cuts = [(0, 100, 5, True), (100, 101, 6, True), (101, 101, 0, False), (101, 250, 0, False),
            (250, 300, 7, True)]
    for lo, hi, tag, new in cuts:
        pool.append(st[lo:hi].contiguous(), tk[lo:hi].contiguous(), tag=tag, new_trace=new)
        ora.append(W.to_bits(st[lo:hi]), tk[lo:hi].cpu().numpy(), tag=tag, new_trace=new)
    keys, tok, tid = pool.read_rows()
    assert np.array_equal(keys, ora.keys)
    assert np.array_equal(tok, ora.tokens) and np.array_equal(tid, ora.trace_ids)
    s, e, t = pool.traces()
    assert s.tolist() == ora.trace_starts.tolist() and e.tolist() == ora.trace_ends.tolist()
    assert t.tolist() == ora.trace_tags.tolist()
    assert pool.stats()["degenerate_rows"] == ora.degenerate_rows == 3
    assert np.all(keys[[7, 11, 13]] == 0)


@pytest.mark.parametrize("d", [200, 4096, 4104, 8192, 12288])
def test_bulk_append_matches_oracle_bit_for_bit(d):
    # thousands of rows per call take the prefetching kernel (a few rows per resident block);
    # row counts that are not a multiple of the grid, rows held in registers in part only
    g = torch.Generator(device="cuda").manual_seed(100 + d)
    n = 3011
    st = (torch.randn(n, d, generator=g, device="cuda") * 2).to(torch.bfloat16)
    st[5] = 0
    st[n - 1, d - 1] = float("inf")
    st[1500, 3] = float("nan")
    st[201] = 0                                  # one row of a pair of rows leaves the fast path
    st[300] = 0                                  # both rows of a pair do
    st[301] = 0
    st[400, 7] = 0                               # a single zero element
    tk = torch.randint(0, 50000, (n,), generator=g, device="cuda", dtype=torch.int32)
    pool, ora = B.Pool(d, n + 200), OraclePool(d)
    for lo, hi, tag in ((0, 100, 3), (100, n, 4)):          # a small call, then a bulk one
        pool.append(st[lo:hi].contiguous(), tk[lo:hi].contiguous(), tag=tag, new_trace=True)
        ora.append(W.to_bits(st[lo:hi]), tk[lo:hi].cpu().numpy(), tag=tag, new_trace=True)
    keys, tok, tid = pool.read_rows()
    assert np.array_equal(keys, ora.keys)
    assert np.array_equal(tok, ora.tokens) and np.array_equal(tid, ora.trace_ids)
    s, e, t = pool.traces()
    assert e.tolist() == ora.trace_ends.tolist() and t.tolist() == ora.trace_tags.tolist()
    assert pool.stats()["degenerate_rows"] == ora.degenerate_rows == 6


def test_append_capacity_and_argument_errors():
    pool = B.Pool(64, 10, max_traces=2)
    st = torch.randn(8, 64, device="cuda").to(torch.bfloat16)
    tk = torch.zeros(8, dtype=torch.int32, device="cuda")
    pool.append(st, tk, tag=1)
    with pytest.raises(B.OilbirdError) as e:
        pool.append(st, tk, tag=2)              # 16 rows > capacity 10
    assert e.value.code == B.ECAPACITY and len(pool) == 8 and pool.num_traces == 1
    pool.append(st[:1].contiguous(), tk[:1].contiguous(), tag=2)
    with pytest.raises(B.OilbirdError) as e:
        pool.append(st[:1].contiguous(), tk[:1].contiguous(), tag=3)   # third trace
    assert e.value.code == B.ECAPACITY
    q = st[:1].contiguous()
    for bad in (dict(k=0), dict(k=65), dict(cont_len=0), dict(cont_len=129), dict(offset=-1)):
        pr = fixed(4, 4)
        for key, val in bad.items():
            setattr(pr, key, val)
        with pytest.raises(B.OilbirdError) as e:
            pool.query(q, pr)
        assert e.value.code == B.EINVAL
    with pytest.raises(B.OilbirdError):
        B.Pool(12, 10)                           # d not a multiple of 8
    pool.reset()
    assert len(pool) == 0 and pool.num_traces == 0


# ------------------------------------------------ closed-form pools on the GPU ----

@pytest.mark.parametrize("d", [16, 256, 1024, 4096])
@pytest.mark.parametrize("path", [B.PATH_GEMV, B.PATH_TENSOR])
def test_hamming_pool_exact_scores_and_tie_order(d, path):
    rng = np.random.default_rng(d)
    base = rng.choice([-1, 1], size=d)
    hs = list(rng.integers(1, min(d, 40), size=300))
    hs[5] = hs[19] = 0                           # planted exact duplicates of the query
    rows = np.stack([np.where(np.arange(d) < h, -base, base) for h in hs])
    bits = np.where(rows > 0, P1, M1).astype(np.uint16)
    pool, ora = B.Pool(d, 512), OraclePool(d)
    tk = np.arange(300, dtype=np.int32)
    pool.append(bits_to_dev(bits), torch.from_numpy(tk).cuda(), tag=1)
    ora.append(bits, tk, tag=1)
    qb = np.where(base > 0, P1, M1).astype(np.uint16)
    pr = fixed(32, 4, path=path)
    out = pool.query(bits_to_dev(qb[None]), pr)
    ref = ora.query(qb, __import__("parity").oracle_params(pr))
    o = out.cpu()
    # every score is an exact dyadic rational: results are identical, ties included
    assert o.idx.numpy().tolist() == ref.idx.tolist()
    assert np.array_equal(o.score.numpy(), ref.score)
    assert o.idx[0, :2].tolist() == [5, 19] and o.score[0, 0] == 1.0
    assert np.array_equal(o.cont_tok.numpy(), ref.cont_tok)
    assert np.array_equal(o.cont_len.numpy(), ref.cont_len)


def test_theta_and_depth_tiers_on_exact_scores():
    d = 1024
    base = np.ones(d, np.int64)
    for h, fired, dep in [(51, 1, 48), (52, 1, 8), (92, 1, 8), (93, 1, 0), (102, 1, 0),
                          (103, 0, 0)]:
        rows = np.stack([np.where(np.arange(d) < h, -base, base)] + [-base] * 60)
        bits = np.where(rows > 0, P1, M1).astype(np.uint16)
        pool = B.Pool(d, 64)
        pool.append(bits_to_dev(bits), torch.arange(61, dtype=torch.int32).cuda(), tag=1)
        out = pool.query(bits_to_dev(np.full((1, d), P1, np.uint16)), B.QueryParams()).cpu()
        assert out.score[0, 0] == 1.0 - 2.0 * h / d
        assert out.fired[0] == fired and out.cont_len[0, 0] == dep
        assert out.cont_tok[0, 0, :dep].tolist() == list(range(2, 2 + dep))
        assert torch.all(out.cont_tok[0, 0, dep:] == -1)
        assert torch.all(out.idx[0, 1:] >= 1)    # theta is not a floor inside the top-k


def test_depth_by_rank_on_exact_scores_and_on_every_scan_path():
    # by hand, as the oracle's pin: scores .609 .9219 .8145 .8828 .414 -> neighbours 1 3 2 0 4
    d = 1024
    base = np.ones(d, np.int64)
    rows = np.stack([np.where(np.arange(d) < h, -base, base) for h in (200, 40, 95, 60, 300)] + [-base] * 60)
    bits = np.where(rows > 0, P1, M1).astype(np.uint16)
    pool = B.Pool(d, 80)
    pool.append(bits_to_dev(bits), torch.arange(65, dtype=torch.int32).cuda(), tag=1)
    q = bits_to_dev(np.full((1, d), P1, np.uint16))
    out = pool.query(q, B.QueryParams(k=5, cont_len=48, depth_mode=B.DEPTH_RANKED)).cpu()
    assert out.idx[0].tolist() == [1, 3, 2, 0, 4] and int(out.fired[0]) == 1
    assert out.cont_len[0].tolist() == [48, 8, 8, 8, 8]
    assert out.cont_tok[0, 0, :3].tolist() == [3, 4, 5] and out.cont_tok[0, 3, :8].tolist() == list(range(2, 10))
    pr = B.QueryParams(k=5, cont_len=12, depth_mode=B.DEPTH_RANKED, tier_thr=(0.0, 0.0, 0.0), tier_depth=(20, 0, 3))
    assert pool.query(q, pr).cpu().cont_len[0].tolist() == [12, 0, 3, 3, 3]
    out = pool.query(q, B.QueryParams(k=5, theta=0.95, cont_len=48, depth_mode=B.DEPTH_RANKED)).cpu()
    assert int(out.fired[0]) == 0 and int(out.cont_len.sum()) == 0 and torch.all(out.cont_tok == -1)
    with pytest.raises(B.OilbirdError):
        pool.query(q, B.QueryParams(k=5, cont_len=12, depth_mode=3))
    # against the oracle on a benchmark-shaped pool, every scan path, several queries
    w = W.C1.scaled(nq=6, k=12, n_rows=3000, d=512, cont_len=24)
    big, ora = fill_both(w)
    qs, _ = w.queries("cuda")
    for path in (B.PATH_GEMV, B.PATH_MMA, B.PATH_TENSOR):
        for tiers in ((48, 8), (5, 4, 3, 2)):
            pr = B.QueryParams(k=8, theta=-2.0, cont_len=24, depth_mode=B.DEPTH_RANKED, path=path,
                               tier_thr=(0.0,) * len(tiers), tier_depth=tiers)
            check_query(big.query(qs, pr), ora, W.to_bits(qs), pr)


# ------------------------------------------------------------- benchmark shapes ----

def run_workload(w, n_rows=None, nq=None, paths=(B.PATH_AUTO,), thetas=(0.8, -2.0), **kw):
    pool, ora = fill_both(w, n_rows=n_rows, **kw)
    q, meta = w.queries("cuda", nq=nq)
    stats = []
    for path in paths:
        for theta in thetas:
            pr = fixed(w.k, w.cont_len, theta=theta, path=path)
            out = pool.query(q, pr)
            stats.append(check_query(out, ora, W.to_bits(q), pr))
            o = out.cpu()
            if "planted_row" in meta and (n_rows is None or meta["planted_row"] < n_rows):
                assert o.idx[0, 0] == meta["planted_row"]
    assert pool.stats()["stalled"] == 0
    return pool, ora, q, meta, stats


def test_c1_tiny_config_and_separated_variant():
    run_workload(W.C1, paths=(B.PATH_GEMV, B.PATH_TENSOR))
    _, _, _, _, st = run_workload(W.C1.separated(), paths=(B.PATH_GEMV, B.PATH_TENSOR))
    assert all(s["strict_sets"] == 1 for s in st)


@pytest.mark.parametrize("n_rows", [1, 31, 32, 33, 127, 129, 1000, 4095])
def test_ragged_pool_sizes(n_rows):
    run_workload(W.C1.scaled(nq=3), n_rows=n_rows, paths=(B.PATH_GEMV, B.PATH_TENSOR))


@pytest.mark.parametrize("nq,k", [(1, 1), (2, 5), (5, 64), (8, 8), (17, 33), (64, 32)])
def test_nq_and_k_combinations(nq, k):
    w = W.C1.scaled(nq=nq, k=k, n_rows=3000, d=512, cont_len=5)
    run_workload(w, paths=(B.PATH_GEMV, B.PATH_TENSOR))
    run_workload(w.separated(), paths=(B.PATH_GEMV, B.PATH_TENSOR))


def test_c2_single_request_decode_full_size():
    _, _, _, _, st = run_workload(W.C2)
    run_workload(W.C2.separated())


def test_c3_tool_calling_shape_scaled():
    w = W.C3.scaled(n_rows=30000, n_templates=20)
    pool, ora, q, meta, _ = run_workload(w)
    out = pool.query(q, fixed(w.k, w.cont_len, theta=-2.0)).cpu()
    # retrieved rows are dominated by the same (template, position) rows of earlier traces
    hits = tot = 0
    for i, rows in enumerate(meta["planted_rows"]):
        want = set(rows)
        got = set(out.idx[i].tolist())
        hits += len(want & got)
        tot += min(len(want), w.k)
    assert hits / tot > 0.9


def test_exclusion_tags():
    w = W.C1.scaled(nq=4, n_rows=2048)
    pool, ora = fill_both(w)
    q, _ = w.queries("cuda")
    ex = np.array([0, 3, 5, 999], dtype=np.uint64)          # tags are 1 + trace number
    for path in (B.PATH_GEMV, B.PATH_TENSOR):
        pr = fixed(16, 4, theta=-2.0, path=path,
                   exclude_tag=torch.from_numpy(ex.view(np.int64)).cuda())
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr, exclude=ex)
        tid = ora.trace_ids
        o = out.cpu()
        assert not np.any(tid[o.idx[1].numpy()] == 2) and not np.any(tid[o.idx[2].numpy()] == 4)


def test_empty_pool_k_above_rows_and_bad_queries():
    d = 64
    pool, ora = B.Pool(d, 100), OraclePool(d)
    q = torch.randn(3, d, device="cuda").to(torch.bfloat16)
    pr = fixed(8, 4, theta=-2.0)
    out = pool.query(q, pr).cpu()
    assert torch.all(out.idx == -1) and torch.all(out.fired == 0) and torch.all(out.cont_tok == -1)
    st = torch.randn(5, d, device="cuda").to(torch.bfloat16)
    tk = torch.arange(5, dtype=torch.int32, device="cuda")
    pool.append(st, tk, tag=1)
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=1)
    q[1] = 0                                      # zero query: all scores 0, lowest rows first
    q[2, 3] = float("nan")                        # NaN query: no neighbours
    for path in (B.PATH_GEMV, B.PATH_TENSOR):
        pr = fixed(8, 4, theta=-2.0, path=path)
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr)
        o = out.cpu()
        assert o.idx[1].tolist() == [0, 1, 2, 3, 4, -1, -1, -1]
        assert torch.all(o.idx[2] == -1) and o.fired[2] == 0
    assert pool.stats()["nonfinite_queries"] == 2


# ------------------------------------------------------------------ invariants ----

def test_batched_equals_single_and_is_deterministic():
    w = W.C1.scaled(nq=8, n_rows=4096, d=1024, k=16)
    pool, ora = fill_both(w)
    q, _ = w.queries("cuda")
    for path in (B.PATH_GEMV, B.PATH_TENSOR):
        pr = fixed(16, 8, theta=-2.0, path=path)
        a = pool.query(q, pr).cpu()
        b = pool.query(q, pr).cpu()
        for f in ("idx", "score", "fired", "cont_len", "cont_tok"):
            assert torch.equal(getattr(a, f), getattr(b, f)), "same inputs, different outputs"
        for i in range(w.nq):
            s = pool.query(q[i:i + 1].contiguous(), pr).cpu()
            assert torch.equal(s.idx[0], a.idx[i]) and torch.equal(s.cont_tok[0], a.cont_tok[i])
            assert torch.allclose(s.score[0], a.score[i], atol=1e-6)


def test_gemv_and_tensor_paths_agree():
    w = W.C1.scaled(nq=8, n_rows=5000, d=2048, k=16).separated()
    pool, ora = fill_both(w)
    q, _ = w.queries("cuda")
    a = pool.query(q, fixed(16, 8, path=B.PATH_GEMV)).cpu()
    b = pool.query(q, fixed(16, 8, path=B.PATH_TENSOR)).cpu()
    assert torch.allclose(a.score, b.score, atol=2e-5)
    assert torch.equal(a.idx[:, :8], b.idx[:, :8])


def test_query_scale_invariance_and_chunked_append():
    w = W.C1.scaled(n_rows=2000, nq=2)
    pool, ora = fill_both(w)
    q, _ = w.queries("cuda")
    pr = fixed(8, 8, theta=-2.0)
    a, b = pool.query(q, pr).cpu(), pool.query((q.float() * 4).to(torch.bfloat16), pr).cpu()
    assert torch.equal(a.idx, b.idx) and torch.equal(a.score, b.score)
    # the same rows appended in other pieces give a bit-identical pool
    pool2 = B.Pool(w.d, w.n_rows)
    for st, tk, tag in w.traces("cuda"):
        pool2.append(st[:100].contiguous(), tk[:100].contiguous(), tag=tag, new_trace=True)
        pool2.append(st[100:].contiguous(), tk[100:].contiguous(), new_trace=False)
    for x, y in zip(pool.read_rows(), pool2.read_rows()):
        assert np.array_equal(x, y)
    c = pool2.query(q, pr).cpu()
    assert torch.equal(a.idx, c.idx) and torch.equal(a.cont_tok, c.cont_tok)


def test_rows_visible_in_stream_order_and_reset():
    w = W.C1.scaled(n_rows=1024)
    pool, ora = fill_both(w, spare_rows=64)
    g = torch.Generator(device="cuda").manual_seed(7)
    for step in range(4):
        st = torch.randn(16, w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 100, (16,), generator=g, device="cuda", dtype=torch.int32)
        pool.append(st, tk, tag=100 + step)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=100 + step)
        q = (st[9:10].float() + 0.05 * torch.randn(1, w.d, generator=g, device="cuda")).to(
            torch.bfloat16)
        pr = fixed(4, 4)
        out = pool.query(q, pr)                   # no synchronisation in between
        assert out.cpu().idx[0, 0] == 1024 + 16 * step + 9
        check_query(out, ora, W.to_bits(q), pr)
    pool.reset()
    ora.reset()
    for st, tk, tag in w.traces("cuda"):
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    q, _ = w.queries("cuda")
    check_query(pool.query(q, fixed(8, 8)), ora, W.to_bits(q), fixed(8, 8))


# -------------------------------------------------------- other entry points ----

def test_gather_entry_point_bit_exact():
    w = W.C1.scaled(n_rows=2048)
    pool, ora = fill_both(w)
    rng = np.random.default_rng(3)
    nq, k, L = 6, 8, 12
    idx = rng.integers(-1, 2048, size=(nq, k)).astype(np.int32)
    idx[0, 0], idx[1, 0], idx[2, 0] = 255, 254, 2047       # trace ends (256-row traces)
    score = np.sort(rng.uniform(0.7, 1.0, size=(nq, k)).astype(np.float32), axis=1)[:, ::-1].copy()
    for pr in (B.QueryParams(k=k, cont_len=L), fixed(k, L), fixed(k, L, offset=1),
               B.QueryParams(k=k, cont_len=L, theta=0.95)):
        out = pool.gather(torch.from_numpy(idx).cuda(), torch.from_numpy(score).cuda(), pr).cpu()
        for q in range(nq):
            f = int(idx[q, 0] >= 0 and score[q, 0] >= np.float32(pr.theta))
            assert out.fired[q] == f
            for j in range(k):
                dep = 0
                if f and idx[q, j] >= 0:
                    dep = L if pr.depth_mode == B.DEPTH_FIXED else oracle.depth(float(score[q, j]))
                tok, n = ora.gather_one(int(idx[q, j]), dep, pr.offset, L)
                assert out.cont_len[q, j] == n and out.cont_tok[q, j].tolist() == tok.tolist()


def test_host_buffer_entry_points_match_device_ones():
    w = W.C1.scaled(n_rows=1024, nq=3)
    pool, ora = fill_both(w, spare_rows=32)
    st = torch.randn(8, w.d).to(torch.bfloat16).pin_memory()
    tk = torch.arange(8, dtype=torch.int32).pin_memory()
    pool.append_host(st, tk, tag=77)
    ora.append(W.to_bits(st), tk.numpy(), tag=77)
    q, _ = w.queries("cuda")
    pr = fixed(8, 8, theta=-2.0)
    a = pool.query(q, pr).cpu()
    b = pool.query_host(q.cpu().contiguous(), pr)
    for f in ("idx", "score", "fired", "cont_len", "cont_tok"):
        assert torch.equal(getattr(a, f), getattr(b, f))
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)


def test_caller_provided_arena():
    w = W.C1.scaled(n_rows=512)
    pool, ora = fill_both(w, use_torch_arena=True)
    q, _ = w.queries("cuda")
    check_query(pool.query(q, fixed(8, 8)), ora, W.to_bits(q), fixed(8, 8))


@pytest.mark.parametrize("nq,path", [(1, "gemv"), (2, "gemv"), (4, "tensor"), (3, "mma"), (8, "mma"),
                                     (11, "mma")])
def test_step_is_append_plus_query(nq, path):
    # the fused step lets the scan run next to its own append; results must not change,
    # and the rows appended in the same step must be found
    w = W.C1.scaled(n_rows=4096, nq=nq)
    pool, ora = fill_both(w, spare_rows=512)
    pool2, _ = fill_both(w, spare_rows=512)
    g = torch.Generator(device="cuda").manual_seed(11)
    pr = fixed(8, 8, theta=-2.0)
    pr.path = {"gemv": B.PATH_GEMV, "tensor": B.PATH_TENSOR, "mma": B.PATH_MMA}[path]
    for step in range(8):
        n = [8, 1, 0, 33, 64, 100, 8, 2][step]      # up to 64 rows ride inside the scan kernel
        st = torch.randn(n, w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 100, (n,), generator=g, device="cuda", dtype=torch.int32)
        q = torch.randn(nq, w.d, generator=g, device="cuda").to(torch.bfloat16)
        if n > 0:
            q[0] = st[n - 1]          # the newest row is the best neighbour of query 0
        a = pool.step(st, tk, q, pr, tag=70 + step)
        pool2.append(st, tk, tag=70 + step)
        b = pool2.query(q, pr)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=70 + step)
        for f in ("idx", "score", "fired", "cont_len", "cont_tok"):
            assert torch.equal(getattr(a, f), getattr(b, f)), (step, f)
        if n > 0:
            assert int(a.idx[0, 0]) == len(pool) - 1
        check_query(a, ora, W.to_bits(q), pr)
    assert len(pool) == len(pool2) == 4096 + 216
    assert pool.stats()["stalled"] == 0
    keys, tok, _ = pool.read_rows()
    assert np.array_equal(keys, ora.keys) and np.array_equal(tok, ora.tokens)


def test_step_with_exclusion_tags_sees_the_new_rows_tags():
    # the rows a fused step appends carry a tag; a query of the same step that excludes that
    # tag must not return them, and one that excludes another tag must
    w = W.C1.scaled(n_rows=4096, nq=2)
    pool, ora = fill_both(w, spare_rows=512)
    g = torch.Generator(device="cuda").manual_seed(21)
    for step in range(6):
        n = 8
        st = torch.randn(n, w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 100, (n,), generator=g, device="cuda", dtype=torch.int32)
        q = torch.stack([st[3], st[5]]).contiguous()           # both queries equal new rows
        tag = 9000 + step
        ex = torch.tensor([tag, 12345], dtype=torch.int64, device="cuda")
        pr = fixed(4, 4, theta=-2.0)
        pr.exclude_tag = ex
        out = pool.step(st, tk, q, pr, tag=tag, new_trace=(step % 2 == 0))
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag, new_trace=(step % 2 == 0))
        first_new = len(pool) - n
        if step % 2 == 0:                                     # a new trace with the excluded tag
            assert all(int(r) < first_new for r in out.idx[0].tolist())
        assert int(out.idx[1, 0]) == first_new + 5
        check_query(out, ora, W.to_bits(q), pr, exclude=ex.cpu().numpy().astype(np.uint64))


def test_step_back_to_back_and_small_pools():
    # 300 fused steps without a host synchronisation in between: every step must find the
    # row it has just appended; then a pool too small to host the append inside the scan
    w = W.C1.scaled(n_rows=8192, nq=1)
    pool, ora = fill_both(w, spare_rows=4096)
    g = torch.Generator(device="cuda").manual_seed(3)
    pr = fixed(4, 4, theta=-2.0)
    steps = 300
    st = torch.randn(steps, 8, w.d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.randint(0, 100, (steps, 8), generator=g, device="cuda", dtype=torch.int32)
    outs = [B.QueryOut.empty(1, 4, 4, "cuda") for _ in range(steps)]
    for s in range(steps):
        pool.step(st[s], tk[s], st[s, 7:8].contiguous(), pr, out=outs[s], tag=500 + s,
                  new_trace=(s % 3 == 0))
    torch.cuda.synchronize()
    for s in range(steps):
        assert int(outs[s].idx[0, 0]) == 8192 + 8 * s + 7, s
        assert abs(float(outs[s].score[0, 0]) - 1.0) < 2e-2
    for s in range(steps):
        ora.append(W.to_bits(st[s]), tk[s].cpu().numpy(), tag=500 + s, new_trace=(s % 3 == 0))
    keys, tok, tid = pool.read_rows()
    assert np.array_equal(keys, ora.keys) and np.array_equal(tok, ora.tokens)
    check_query(pool.query(st[0, :1].contiguous(), pr), ora, W.to_bits(st[0, :1]), pr)
    assert pool.stats()["stalled"] == 0

    small = B.Pool(w.d, 256)
    osm = oracle.OraclePool(w.d)
    for s in range(4):
        out = small.step(st[s], tk[s], st[s, 3:4].contiguous(), pr, tag=s)
        osm.append(W.to_bits(st[s]), tk[s].cpu().numpy(), tag=s)
        assert int(out.idx[0, 0]) == 8 * s + 3
    keys, tok, _ = small.read_rows()
    assert np.array_equal(keys, osm.keys) and np.array_equal(tok, osm.tokens)


def test_step_host_is_append_host_plus_query_host():
    w = W.C1.scaled(n_rows=1024, nq=2)
    pool, ora = fill_both(w, spare_rows=64)
    pool2, _ = fill_both(w, spare_rows=64)
    g = torch.Generator().manual_seed(5)
    q, _ = w.queries("cuda")
    qh = q.cpu().contiguous()
    pr = fixed(8, 8, theta=-2.0)
    for step in range(3):
        st = torch.randn(8, w.d, generator=g).to(torch.bfloat16)
        tk = torch.randint(0, 100, (8,), generator=g, dtype=torch.int32)
        a = B.QueryOut.empty(2, 8, 8, "cpu")
        pool.step_host(st, tk, qh, pr, a, tag=50 + step)
        pool2.append_host(st, tk, tag=50 + step)
        b = pool2.query_host(qh, pr)
        ora.append(W.to_bits(st), tk.numpy(), tag=50 + step)
        for f in ("idx", "score", "fired", "cont_len", "cont_tok"):
            assert torch.equal(getattr(a, f), getattr(b, f))
    assert len(pool) == len(pool2) == 1024 + 24
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)


def test_host_steps_in_flight_two_deep_equal_the_oracle_step_by_step():
    """step_host_begin / step_host_end: two steps in flight, each step's answer is the oracle's
    answer on the pool as it was after that step's own append (and before the next one's);
    a busy slot and an idle slot are refused and change nothing."""
    w = W.C1.scaled(n_rows=1024, nq=2)
    pool, ora = fill_both(w, spare_rows=200)
    g = torch.Generator().manual_seed(11)
    pr = fixed(8, 8, theta=-2.0)
    sizes = [8, 1, 0, 16, 8, 3, 8]
    steps = []
    for n in sizes:
        st = torch.randn(n, w.d, generator=g).to(torch.bfloat16)
        qh = torch.randn(2, w.d, generator=g).to(torch.bfloat16)
        if n:
            qh[0] = st[n // 2]                   # the first query repeats one of the step's own rows
        steps.append((st, torch.randint(0, 100, (n,), generator=g, dtype=torch.int32), qh.contiguous()))
    outs = [B.QueryOut.empty(2, 8, 8, "cpu") for _ in steps]
    with pytest.raises(B.OilbirdError) as e:
        pool.step_host_end(0, outs[0])           # nothing in flight yet
    assert e.value.code == B.EINVAL

    for s, (st, tk, qh) in enumerate(steps):
        if s >= 2:
            pool.step_host_end(s % 2, outs[s - 2])   # frees the slot this step takes
        st_in, tk_in, qh_in = st.clone(), tk.clone(), qh.clone()
        pool.step_host_begin(st_in, tk_in, qh_in, pr, slot=s % 2, tag=70 + s)
        st_in.zero_(); tk_in.zero_(); qh_in.zero_()  # the caller's buffers are free after begin
        if s == 0:
            rows = len(pool)
            with pytest.raises(B.OilbirdError) as e:
                pool.step_host_begin(st, tk, qh, pr, slot=0, tag=999)   # slot 0 is busy
            assert e.value.code == B.EINVAL and "in flight" in str(e.value) and len(pool) == rows
    pool.step_host_end((len(steps) - 1) % 2, outs[-1])   # any order
    pool.step_host_end((len(steps) - 2) % 2, outs[-2])
    for s, (st, tk, qh) in enumerate(steps):
        ora.append(W.to_bits(st), tk.numpy(), tag=70 + s)
        check_query(outs[s], ora, W.to_bits(qh), pr)
        if sizes[s]:
            assert int(outs[s].idx[0, 0]) == len(ora) - sizes[s] + sizes[s] // 2
    assert len(pool) == len(ora) == 1024 + sum(sizes)
    # a synchronous call beside a step in flight uses the free slot
    qh = steps[0][2]
    pool.step_host_begin(torch.empty(0, w.d, dtype=torch.bfloat16), torch.empty(0, dtype=torch.int32),
                         qh, pr, slot=0, new_trace=False)
    b = pool.query_host(qh, pr)
    a = pool.step_host_end(0, B.QueryOut.empty(2, 8, 8, "cpu"))
    for f in ("idx", "score", "fired", "cont_len", "cont_tok"):
        assert torch.equal(getattr(a, f), getattr(b, f))


@pytest.mark.parametrize("nq,k", [(256, 128), (100, 128), (256, 64), (33, 100)])
def test_largest_nq_and_k(nq, k):
    """Per-query lists for nq*k beyond shared memory: the tensor path keeps them in global
    memory (its slice of the scan's output) and still scans the keys once."""
    w = W.C1.scaled(nq=nq, k=k, n_rows=2500, d=256, cont_len=3)
    pool, ora = fill_both(w, max_k=128, max_nq=256)
    q, _ = w.queries("cuda")
    pr = fixed(k, 3, theta=-2.0, path=B.PATH_TENSOR)
    out = pool.query(q, pr)
    check_query(out, ora, W.to_bits(q), pr)
    ws = w.scaled(n_rows=max(2500, 2 * nq * (k + 4))).separated()   # room for the planted rows
    pool, ora = fill_both(ws, max_k=128, max_nq=256)
    q, _ = ws.queries("cuda")
    st = check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    if k <= 100:
        gem = pool.query(q[:2].contiguous(), fixed(k, 3, theta=-2.0, path=B.PATH_GEMV))
        check_query(gem, ora, W.to_bits(q)[:2], pr)


@pytest.mark.parametrize("nq,k", [(129, 8), (160, 64), (200, 16), (256, 64), (256, 128), (131, 1)])
def test_pairs_of_ctas_on_batches_above_128_queries(nq, k):
    """More than 128 queries on a pool of at least four tiles per SM: two CTAs share each
    tile of 256 rows (one MMA over both, each loading half of the query rows).  Ragged last
    tile whose second half is empty or partly filled, query counts that are no multiple of
    32, rows beyond the pool's size inside the last tile."""
    for n_rows in (148 * 128 * 4 + 77, 148 * 128 * 4 + 128 + 5):
        w = W.C1.scaled(nq=nq, k=k, n_rows=n_rows, d=192, cont_len=3, n_centroids=2048,
                        rows_per_trace=1024, seed=40 + k)
        pool, ora = fill_both(w, max_k=128, max_nq=256)
        q, meta = w.queries("cuda")
        pr = fixed(k, 3, theta=-2.0, path=B.PATH_TENSOR)
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr)
        assert int(out.idx[0, 0]) == meta["planted_row"]
        assert pool.stats()["stalled"] == 0
        # which candidates reach the lists depends on when the CTAs' bounds arrive; the
        # answer must not: three more runs, bit for bit
        a = out.cpu()
        for _ in range(3):
            b = pool.query(q, pr).cpu()
            assert torch.equal(a.idx, b.idx) and torch.equal(a.score, b.score)
            assert torch.equal(a.cont_tok, b.cont_tok) and torch.equal(a.cont_len, b.cont_len)
    ws = w.separated()
    pool, ora = fill_both(ws, max_k=128, max_nq=256)
    q, _ = ws.queries("cuda")
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    # exclusion tags: every query skips the trace that holds its best neighbour
    best = pool.query(q, pr).cpu().idx[:, 0].numpy()
    ex = np.array([ws.trace_tag(int(b) // ws.rows_per_trace) for b in best], dtype=np.int64)
    pr_ex = fixed(k, 3, theta=-2.0, path=B.PATH_TENSOR, exclude_tag=torch.from_numpy(ex).cuda())
    check_query(pool.query(q, pr_ex), ora, W.to_bits(q), pr_ex, exclude=ex.astype(np.uint64))
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("nq,k", [(97, 8), (128, 64), (120, 1), (160, 16), (224, 64), (129, 8),
                                  (256, 64), (241, 128)])
def test_pairs_of_ctas_with_two_tiles_each_from_97_to_256_queries(nq, k):
    """97 to 256 queries on a pool of at least eight tiles per SM: a pair of CTAs takes macro
    tiles of 512 rows (two MMAs over both CTAs per query tile), with two accumulator sets up
    to 128 queries and one above.  Last macro tile with one, two and three of its four
    sub-tiles (partly) filled."""
    sizes = (148 * 128 * 8 + 77, 148 * 128 * 8 + 128 + 5, 148 * 128 * 8 + 3 * 128 - 1)
    if (nq, k) not in ((128, 64), (160, 16)):   # the other batch sizes take one ragged size each
        sizes = sizes[(nq + k) % 3:][:1]
    for n_rows in sizes:
        w = W.C1.scaled(nq=nq, k=k, n_rows=n_rows, d=128, cont_len=3, n_centroids=2048,
                        rows_per_trace=1024, seed=80 + k)
        pool, ora = fill_both(w, max_k=128, max_nq=256)
        q, meta = w.queries("cuda")
        pr = fixed(k, 3, theta=-2.0, path=B.PATH_TENSOR)
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr)
        assert int(out.idx[0, 0]) == meta["planted_row"]
        assert pool.stats()["stalled"] == 0
        a = out.cpu()
        for _ in range(2):
            b = pool.query(q, pr).cpu()
            assert torch.equal(a.idx, b.idx) and torch.equal(a.score, b.score)
    ws = w.separated()
    pool, ora = fill_both(ws, max_k=128, max_nq=256)
    q, _ = ws.queries("cuda")
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    best = pool.query(q, pr).cpu().idx[:, 0].numpy()
    ex = np.array([ws.trace_tag(int(b) // ws.rows_per_trace) for b in best], dtype=np.int64)
    pr_ex = fixed(k, 3, theta=-2.0, path=B.PATH_TENSOR, exclude_tag=torch.from_numpy(ex).cuda())
    check_query(pool.query(q, pr_ex), ora, W.to_bits(q), pr_ex, exclude=ex.astype(np.uint64))
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("nq,k,n_rows", [(16, 16, 40000), (64, 64, 40000), (256, 64, 148 * 128 * 8 + 77),
                                         (200, 128, 148 * 128 * 8 + 77)])
def test_rows_that_keep_getting_better_overflow_the_candidate_queues(nq, k, n_rows):
    """A pool whose every row is closer to the queries than the rows before it: every score
    is a candidate, the per-query queues of the tensor scan's epilogue fill up in every round
    and the tiles go the long way (round-wide queues, sorted batches).  Same answers."""
    d = 128
    g = torch.Generator(device="cuda").manual_seed(90 + nq)
    base = torch.randn(1, d, generator=g, device="cuda")
    noise = torch.randn(n_rows, d, generator=g, device="cuda")
    wgt = torch.linspace(3.0, 0.2, n_rows, device="cuda").unsqueeze(1)
    st = (base + wgt * noise).to(torch.bfloat16)
    pool = B.Pool(d, n_rows, max_nq=256, max_k=128, max_traces=64)
    ora = OraclePool(d)
    per = 8192
    for i in range(0, n_rows, per):
        rows = st[i:i + per].contiguous()
        tk = torch.arange(i, i + rows.shape[0], dtype=torch.int32, device="cuda")
        pool.append(rows, tk, tag=i // per + 1)
        ora.append(W.to_bits(rows), tk.cpu().numpy(), tag=i // per + 1)
    q = (base + 0.05 * torch.randn(nq, d, generator=g, device="cuda")).to(torch.bfloat16)
    pr = fixed(k, 3, theta=-2.0, path=B.PATH_TENSOR)
    out = pool.query(q, pr)
    check_query(out, ora, W.to_bits(q), pr)
    assert int(out.idx[:, 0].min()) > n_rows - 4000          # the best rows are the last ones
    a = out.cpu()
    b = pool.query(q, pr).cpu()
    assert torch.equal(a.idx, b.idx) and torch.equal(a.score, b.score)
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("d", [8, 72, 200, 1000])
def test_key_widths_that_are_not_multiples_of_the_k_block(d):
    w = W.C1.scaled(nq=3, k=8, n_rows=1500, d=d, cont_len=4, sigma=0.3)
    run_workload(w, paths=(B.PATH_GEMV, B.PATH_TENSOR))
    run_workload(w.separated(), paths=(B.PATH_GEMV, B.PATH_TENSOR))


def test_exact_ties_spread_over_all_ctas_keep_the_lowest_rows():
    """Many rows with identical scores, spread over every CTA of the tensor scan: the
    thresholds the CTAs exchange must never drop a tied row that has a lower position."""
    d, n = 64, 148 * 128 * 4 + 77
    rng = np.random.default_rng(5)
    base = rng.choice([-1, 1], size=d)
    hs = rng.choice([0, 1, 2, 3, 20, 21, 22, 30], size=n, p=[.002, .004, .004, .01, .2, .2, .28, .3])
    rows = np.tile(base, (n, 1))
    for h in np.unique(hs):
        rows[hs == h, :h] *= -1
    bits = np.where(rows > 0, P1, M1).astype(np.uint16)
    tk = np.arange(n, dtype=np.int32)
    pool, ora = B.Pool(d, n, max_k=128), OraclePool(d)
    pool.append(bits_to_dev(bits), torch.from_numpy(tk).cuda(), tag=1)
    ora.append(bits, tk, tag=1)
    qb = np.stack([np.where(base > 0, P1, M1).astype(np.uint16)] * 3)
    qb[1, :2] = np.where(base[:2] > 0, M1, P1)              # a second, slightly different query
    # the same three queries 50 times over: the two-CTA form of the tensor scan (> 128 queries)
    qmany = np.concatenate([qb] * 50)
    pool.close()
    pool = B.Pool(d, n, max_k=128, max_nq=256)
    pool.append(bits_to_dev(bits), torch.from_numpy(tk).cuda(), tag=1)
    for k in (8, 128):
        pr = fixed(k, 2, theta=-2.0, path=B.PATH_TENSOR)
        out = pool.query(bits_to_dev(qmany), pr).cpu()
        ref = ora.query(qb, __import__("parity").oracle_params(pr))
        for r in range(50):
            assert out.idx.numpy()[3 * r:3 * r + 3].tolist() == ref.idx.tolist(), (k, r)
            assert np.array_equal(out.score.numpy()[3 * r:3 * r + 3], ref.score)
    for k in (1, 8, 64, 128):
        for path in (B.PATH_TENSOR, B.PATH_GEMV):
            pr = fixed(k, 2, theta=-2.0, path=path)
            out = pool.query(bits_to_dev(qb), pr).cpu()
            ref = ora.query(qb, __import__("parity").oracle_params(pr))
            assert out.idx.numpy().tolist() == ref.idx.tolist(), (k, path)
            assert np.array_equal(out.score.numpy(), ref.score)
