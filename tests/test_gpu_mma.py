"""GPU parity for the warp-level tensor-core scan (OILBIRD_PATH_MMA: batches of 3 to 8 queries
on pools of the paper's size) against the CPU oracle, under the acceptance rule of
tests/parity.py, and against the other two scans."""
import numpy as np
import pytest
import torch

from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query, fill_both, oracle_params

pytestmark = pytest.mark.gpu

P1, M1 = 0x3F80, 0xBF80


def fixed(k, L, theta=0.8, **kw):
    return B.QueryParams(k=k, theta=theta, depth_mode=B.DEPTH_FIXED, cont_len=L, **kw)


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("d", [256, 1024, 4096])
def test_hamming_pool_exact_scores_and_tie_order(d):
    # +-1 keys and queries: every product and partial sum is an exact dyadic number, so the
    # scores, the order and the planted ties must come out identical to the oracle's
    rng = np.random.default_rng(d)
    base = rng.choice([-1, 1], size=d)
    hs = list(rng.integers(1, min(d, 40), size=300))
    hs[5] = hs[19] = 0
    rows = np.stack([np.where(np.arange(d) < h, -base, base) for h in hs])
    bits = np.where(rows > 0, P1, M1).astype(np.uint16)
    pool, ora = B.Pool(d, 512, max_nq=8), OraclePool(d)
    tk = np.arange(300, dtype=np.int32)
    pool.append(bits_to_dev(bits), torch.from_numpy(tk).cuda(), tag=1)
    ora.append(bits, tk, tag=1)
    qb = np.stack([np.where(base > 0, P1, M1), np.where(base > 0, M1, P1),
                   bits[7], bits[100], bits[299]]).astype(np.uint16)
    pr = fixed(32, 4, path=B.PATH_MMA)
    o = pool.query(bits_to_dev(qb), pr).cpu()
    ref = ora.query(qb, oracle_params(pr))
    assert o.idx.numpy().tolist() == ref.idx.tolist()
    assert np.array_equal(o.score.numpy(), ref.score)
    assert o.idx[0, :2].tolist() == [5, 19] and o.score[0, 0] == 1.0
    assert np.array_equal(o.cont_tok.numpy(), ref.cont_tok)
    assert np.array_equal(o.cont_len.numpy(), ref.cont_len)


@pytest.mark.parametrize("nq,k", [(1, 8), (3, 8), (5, 32), (8, 16), (8, 33), (9, 8), (11, 64), (16, 16), (17, 5), (35, 40)])
def test_nq_and_k_combinations(nq, k):
    # 9 to 16 queries take two 8-query tiles per pass, more run in several passes over the
    # keys; k above 32 uses two registers per lane
    w = W.C1.scaled(nq=nq, k=k, n_rows=3000, d=512, cont_len=5)
    for wl in (w, w.separated()):
        pool, ora = fill_both(wl)
        q, _ = wl.queries("cuda")
        for theta in (0.8, -2.0):
            pr = fixed(k, 5, theta=theta, path=B.PATH_MMA)
            check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
        assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("n_rows", [1, 15, 16, 17, 127, 129, 1000, 4095])
def test_ragged_pool_sizes(n_rows):
    w = W.C1.scaled(nq=6)
    pool, ora = fill_both(w, n_rows=n_rows)
    q, _ = w.queries("cuda")
    pr = fixed(w.k, w.cont_len, theta=-2.0, path=B.PATH_MMA)
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)


def test_exclusion_tags_bad_queries_and_agreement_with_the_other_scans():
    w = W.C1.scaled(nq=7, n_rows=2048)
    pool, ora = fill_both(w)
    q, _ = w.queries("cuda")
    q = q.clone()
    q[2, 3] = float("nan")                       # finds nothing, is counted
    q[4] = 0                                     # legal: scores 0 against every row
    ex = np.array([0, 3, 5, 999, 2, 0, 1], dtype=np.uint64)       # tags are 1 + trace number
    outs = {}
    for path in (B.PATH_GEMV, B.PATH_TENSOR, B.PATH_MMA):
        pr = fixed(16, 4, theta=-2.0, path=path,
                   exclude_tag=torch.from_numpy(ex.view(np.int64)).cuda())
        outs[path] = pool.query(q, pr).cpu()
    pr = fixed(16, 4, theta=-2.0, path=B.PATH_MMA,
               exclude_tag=torch.from_numpy(ex.view(np.int64)).cuda())
    o = outs[B.PATH_MMA]
    qb = W.to_bits(q)
    keep = [0, 1, 3, 4, 5, 6]
    assert torch.all(o.idx[2] == -1) and int(o.fired[2]) == 0
    assert pool.stats()["nonfinite_queries"] == 3          # once per path
    tid = ora.trace_ids
    assert not np.any(tid[o.idx[1].numpy()] == 2) and not np.any(tid[o.idx[4].numpy()] == 1)
    # the three scans normalise a query to the same bf16 vector and differ only in the order
    # of the fp32 accumulation: same neighbours wherever the scores are not within rounding
    for other in (B.PATH_GEMV, B.PATH_TENSOR):
        assert torch.allclose(o.score, outs[other].score, atol=2e-5, rtol=0, equal_nan=True)
        same = (o.idx == outs[other].idx).float().mean()
        assert same > 0.95
    # and the oracle, query by query (the NaN query is covered above)
    for i in keep:
        pr_i = fixed(16, 4, theta=-2.0, path=B.PATH_MMA,
                     exclude_tag=torch.from_numpy(ex[i:i + 1].view(np.int64)).cuda())
        check_query(pool.query(q[i:i + 1].contiguous(), pr_i), ora, qb[i:i + 1], pr_i,
                    exclude=ex[i:i + 1])


def test_auto_path_uses_it_for_small_batches_only():
    w = W.C1.scaled(nq=8, n_rows=4096, d=256)
    pool, ora = fill_both(w)
    q, _ = w.queries("cuda")
    pr = fixed(8, 8, theta=-2.0)
    for nq, launches in ((1, 2), (2, 2), (3, 2), (8, 2)):    # scan + merge
        l0 = pool.launch_count
        out = pool.query(q[:nq].contiguous(), pr)
        assert pool.launch_count - l0 == launches
        check_query(out, ora, W.to_bits(q[:nq]), pr)
    big = B.Pool(256, 64, max_nq=16)
    big.append(torch.randn(64, 256, device="cuda").to(torch.bfloat16),
               torch.zeros(64, dtype=torch.int32, device="cuda"), tag=1)
    l0 = big.launch_count
    big.query(torch.randn(9, 256, device="cuda").to(torch.bfloat16), pr)
    assert big.launch_count - l0 == 2                        # sixteen queries per pass fit: still this scan
    big17 = B.Pool(256, 64, max_nq=32)
    big17.append(torch.randn(64, 256, device="cuda").to(torch.bfloat16),
                 torch.zeros(64, dtype=torch.int32, device="cuda"), tag=1)
    l0 = big17.launch_count
    big17.query(torch.randn(17, 256, device="cuda").to(torch.bfloat16), pr)
    assert big17.launch_count - l0 == 3                      # query normalisation + tcgen05 scan + merge
    # widths that are not a multiple of 128 and k above 64 stay on the other scans
    odd = B.Pool(200, 64, max_nq=8, max_k=128)
    odd.append(torch.randn(64, 200, device="cuda").to(torch.bfloat16),
               torch.zeros(64, dtype=torch.int32, device="cuda"), tag=1)
    odd.query(torch.randn(4, 200, device="cuda").to(torch.bfloat16), pr)
    with pytest.raises(B.OilbirdError) as e:
        odd.query(torch.randn(4, 200, device="cuda").to(torch.bfloat16), fixed(8, 8, path=B.PATH_MMA))
    assert e.value.code == B.EINVAL
    # 8-bit pools take it from widths that are multiples of 256 (tests/test_gpu_q8.py)
    q8 = B.Pool(128, 64, max_nq=8, key_format="e4m3")
    q8.append(torch.randn(64, 128, device="cuda").to(torch.bfloat16),
              torch.zeros(64, dtype=torch.int32, device="cuda"), tag=1)
    with pytest.raises(B.OilbirdError):
        q8.query(torch.randn(4, 128, device="cuda").to(torch.bfloat16), fixed(8, 8, path=B.PATH_MMA))


def test_paper_scale_pool_batch_of_eight_full_width():
    # a pool of the paper's own size (tens of thousands of rows at d = 4096), eight queries
    w = W.C2.scaled(n_rows=33000, nq=8)
    pool, ora = fill_both(w)
    q, meta = w.queries("cuda")
    for theta in (0.8, -2.0):
        pr = fixed(w.k, w.cont_len, theta=theta)             # auto: the warp-level tensor scan
        l0 = pool.launch_count
        out = pool.query(q, pr)
        assert pool.launch_count - l0 == 2
        check_query(out, ora, W.to_bits(q), pr)


def test_fused_step_appends_inside_the_scan_and_sees_the_new_rows_tags():
    # 3 to 8 queries and up to 64 new rows: the scan's first CTAs append the step's rows
    # (two launches per step); a query of the same step finds them, honours their tag, and the
    # stored rows equal the oracle's
    w = W.C1.scaled(n_rows=4096, nq=5)
    pool, ora = fill_both(w, spare_rows=1024)
    g = torch.Generator(device="cuda").manual_seed(33)
    for step in range(8):
        n = [8, 1, 64, 33, 8, 16, 2, 8][step]
        st = torch.randn(n, w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 100, (n,), generator=g, device="cuda", dtype=torch.int32)
        q = torch.randn(5, w.d, generator=g, device="cuda").to(torch.bfloat16)
        q[0] = st[n - 1]
        q[3] = st[0]
        tag = 9000 + step
        ex = torch.tensor([tag, 12345, 0, 0, tag], dtype=torch.int64, device="cuda")
        pr = fixed(4, 4, theta=-2.0)
        pr.exclude_tag = ex
        new_trace = step % 2 == 0
        l0 = pool.launch_count
        out = pool.step(st, tk, q, pr, tag=tag, new_trace=new_trace)
        assert pool.launch_count - l0 == 2
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag, new_trace=new_trace)
        first_new = len(pool) - n
        if new_trace:                                         # a new trace with the excluded tag
            assert all(int(r) < first_new for r in out.idx[0].tolist())
        assert int(out.idx[3, 0]) == first_new
        check_query(out, ora, W.to_bits(q), pr, exclude=ex.cpu().numpy().astype(np.uint64))
    assert pool.stats()["stalled"] == 0
    keys, tok, tid = pool.read_rows()
    assert np.array_equal(keys, ora.keys) and np.array_equal(tok, ora.tokens)
    assert np.array_equal(tid, ora.trace_ids)


@pytest.mark.parametrize("d", [6144, 8192])
def test_wide_rows(d):
    # the eight normalised queries of a CTA take 96 to 128 KB of shared memory here
    w = W.C1.scaled(n_rows=1500, nq=7, d=d, k=8)
    pool, ora = fill_both(w, spare_rows=64)
    q, _ = w.queries("cuda")
    for theta in (0.8, -2.0):
        pr = fixed(8, 8, theta=theta, path=B.PATH_MMA)
        check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    g = torch.Generator(device="cuda").manual_seed(d)
    st = torch.randn(8, d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.randint(0, 100, (8,), generator=g, device="cuda", dtype=torch.int32)
    qs = q.clone()
    qs[2] = st[6]
    pr = fixed(8, 8, theta=-2.0)
    l0 = pool.launch_count
    out = pool.step(st, tk, qs, pr, tag=777)
    assert pool.launch_count - l0 == 2
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=777)
    check_query(out, ora, W.to_bits(qs), pr)
    assert int(out.idx[2, 0]) == len(pool) - 2
    assert pool.stats()["stalled"] == 0
