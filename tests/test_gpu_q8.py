"""GPU parity for pools with 8-bit keys (FP8 E4M3 codes + one fp32 scale per row): stored
codes and scales bit-exact against the oracle, scores / neighbours / continuations under the
same acceptance rule as the 16-bit pool (tests/parity.py)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query, fill_both

pytestmark = pytest.mark.gpu


def fixed(k, L, theta=0.8, **kw):
    return B.QueryParams(k=k, theta=theta, depth_mode=B.DEPTH_FIXED, cont_len=L, **kw)


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("d", [16, 208, 256, 4096, 8192])
def test_codes_and_scales_match_oracle_bit_for_bit(d):
    g = torch.Generator(device="cuda").manual_seed(d)
    n = 300
    st = (torch.randn(n, d, generator=g, device="cuda") * 3).to(torch.bfloat16)
    st[7] = 0                                   # zero row
    st[11, d // 2] = float("inf")               # non-finite rows are stored as zero codes
    st[13, 0] = float("nan")
    st[17] = st[17] * 1e-30                     # tiny but usable
    st[19, 1:] = 0                              # one-hot: the peak is the only entry
    st[23] = torch.where(st[23].abs() < 2.0, torch.zeros_like(st[23]), st[23])   # many exact zeros
    st[29, : d // 2] *= 1e-3                    # half the row lands in the subnormal codes
    st[31] = -st[31].abs()                      # all negative
    tok = torch.arange(n, dtype=torch.int32, device="cuda")
    pool = B.Pool(d, n, key_format="e4m3")
    ora = OraclePool(d, "e4m3")
    pool.append(st[:100].contiguous(), tok[:100].contiguous(), tag=1)
    pool.append(st[100:].contiguous(), tok[100:].contiguous(), tag=2, new_trace=False)
    ora.append(W.to_bits(st), tok.cpu().numpy(), tag=1)
    codes, scales = pool.read_codes()
    assert np.array_equal(scales.view(np.uint32), ora.scales.view(np.uint32))
    assert np.array_equal(codes, ora.codes)
    _, tk, _ = pool.read_rows()
    assert np.array_equal(tk, ora.tokens)
    assert pool.stats()["degenerate_rows"] == 3
    assert not codes[7].any() and scales[7] == 0


@pytest.mark.parametrize("d", [64, 4096])
def test_rows_whose_elements_sit_on_code_boundaries(d):
    # x / peak = 3 * 2^-j or 5 * 2^-j / 7 ... : with a power-of-two peak, 448 x / peak = 21 * 2^m
    # lies exactly between two codes, and only the rounding of the stored scale (a different
    # one per row, through the norm) decides the side.  Elements far below the peak (a spread
    # of more than 2^40) and rows mixing all of it with ordinary values are in as well.
    rng = np.random.default_rng(7 + d)
    n = 400
    rows = np.zeros((n, d), np.float32)
    for r in range(n):
        peak = 2.0 ** rng.integers(-20, 20)
        j = rng.integers(2, 9, size=d)
        vals = np.where(rng.random(d) < 0.5, 3.0, 1.0) * 2.0 ** (-j) * peak
        vals *= rng.choice([-1.0, 1.0], size=d)
        if r % 3 == 1:                                   # ordinary values mixed in: moves the norm
            m = rng.random(d) < 0.3
            vals[m] = rng.standard_normal(m.sum()) * 0.05 * peak
        if r % 7 == 3:
            vals[rng.integers(0, d)] = peak * 2.0 ** -45  # far below the peak
        vals[rng.integers(0, d)] = peak
        rows[r] = vals
    st = torch.from_numpy(rows).to(torch.bfloat16).cuda()
    tok = torch.arange(n, dtype=torch.int32, device="cuda")
    pool = B.Pool(d, n, key_format="e4m3")
    ora = OraclePool(d, "e4m3")
    pool.append(st, tok, tag=1)
    ora.append(W.to_bits(st), tok.cpu().numpy(), tag=1)
    codes, scales = pool.read_codes()
    assert np.array_equal(scales.view(np.uint32), ora.scales.view(np.uint32))
    assert np.array_equal(codes, ora.codes)
    # the planted boundary values did land on both sides across the rows
    rb = st.float().cpu().numpy()
    c84 = codes[(np.abs(rb) == 0.1875 * np.abs(rb).max(1, keepdims=True))] & 0x7f
    assert len(set(c84.tolist())) >= 2


@pytest.mark.parametrize("d", [16, 64, 256, 1024, 4096])
def test_closed_form_pool_scores_are_exact(d):
    # +-1 rows: every code is +-448 and s = (1 - 2 Hamming / d) * (scale * 448 * sqrt(d)), the
    # partial sums are small integers times a power of two, so fp32 accumulation is exact too
    rng = np.random.default_rng(d)
    n = 600
    rows = rng.choice([-1.0, 1.0], size=(n, d)).astype(np.float32)
    q = rng.choice([-1.0, 1.0], size=(2, d)).astype(np.float32)
    rows[5] = q[0]; rows[300] = q[0]; rows[599] = q[0]        # a three-way tie at the top
    rows[17] = -q[1]
    pool = B.Pool(d, n, key_format="e4m3")
    ora = OraclePool(d, "e4m3")
    rb = oracle.f32_to_bf16_bits(rows)
    tok = np.arange(n, dtype=np.int32)
    pool.append(bits_to_dev(rb), torch.from_numpy(tok).cuda(), tag=1)
    ora.append(rb, tok, tag=1)
    qb = oracle.f32_to_bf16_bits(q)
    pr = fixed(8, 2, theta=-2.0)
    out = pool.query(bits_to_dev(qb), pr).cpu()
    ref = ora.query(qb, oracle.QueryParams(k=8, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=2))
    assert out.idx.numpy().tolist() == ref.idx.tolist()
    assert np.array_equal(out.score.numpy(), ref.score)
    assert out.idx[0, :3].tolist() == [5, 300, 599]
    assert np.array_equal(out.cont_tok.numpy(), ref.cont_tok)


@pytest.mark.parametrize("nq,k", [(1, 8), (2, 16), (5, 8), (3, 64), (2, 128)])
def test_query_matches_oracle(nq, k):
    w = W.C1.scaled(n_rows=6000, nq=nq)
    pool, ora = fill_both(w, key_format="e4m3", max_k=k)
    q, _ = w.queries("cuda", nq=nq)
    for pr in (fixed(k, 8), fixed(k, 8, theta=-2.0),
               B.QueryParams(k=k, cont_len=48)):               # the paper's tiers
        check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    assert pool.stats()["stalled"] == 0


def test_wide_rows_exclusion_tags_and_step():
    w = W.C2.scaled(n_rows=3000, nq=2)
    pool, ora = fill_both(w, key_format="e4m3", spare_rows=64)
    q, _ = w.queries("cuda", nq=2)
    tags = [t for _, _, t in w.traces("cpu")][:2]
    ex = torch.tensor([tags[0], 0], dtype=torch.int64, device="cuda")
    pr = fixed(16, 16, theta=-2.0)
    pr.exclude_tag = ex
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr, exclude=ex.cpu().numpy().astype(np.uint64))
    # one serving step: the newest row must be found (separate append kernel for 8-bit pools)
    g = torch.Generator(device="cuda").manual_seed(2)
    st = torch.randn(8, w.d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(8, dtype=torch.int32, device="cuda")
    pr2 = fixed(4, 4, theta=-2.0)
    out = pool.step(st, tk, st[7:8].contiguous(), pr2, tag=999)
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=999)
    assert int(out.idx[0, 0]) == len(pool) - 1
    check_query(out, ora, W.to_bits(st[7:8]), pr2)


def test_limits_of_8bit_pools():
    with pytest.raises(B.OilbirdError):
        B.Pool(24, 100, key_format="e4m3")                       # d must be a multiple of 16
    pool = B.Pool(64, 256, key_format="e4m3")
    st = torch.randn(40, 64, device="cuda").to(torch.bfloat16)
    pool.append(st, torch.arange(40, dtype=torch.int32, device="cuda"))
    pr = fixed(4, 4)
    pr.path = 7
    with pytest.raises(B.OilbirdError):
        pool.query(st[:4].contiguous(), pr)                      # no such scan
    keys, tok, tid = pool.read_rows()
    assert keys is None and tok.shape == (40,)
    pool16 = B.Pool(64, 256)
    pool16.append(st, torch.arange(40, dtype=torch.int32, device="cuda"))
    with pytest.raises(B.OilbirdError):
        pool16.read_codes()
    # half the key bytes: the arena of an 8-bit pool is smaller
    a8 = B.lib().oilbird_pool_arena_bytes
    import ctypes
    c16 = B.PoolConfig(d=4096, capacity_rows=100000, flags=0)
    c8 = B.PoolConfig(d=4096, capacity_rows=100000, flags=B.KEYS_E4M3)
    assert a8(ctypes.byref(c16)) - a8(ctypes.byref(c8)) >= 100000 * 4096 - 100000 * 4 - 4096


def test_retrieval_agrees_with_the_16bit_pool_on_separated_neighbours():
    # quantisation moves a score by < 0.02 here; neighbours that lead by more than that in
    # the 16-bit pool must also be found in the 8-bit one
    w = W.C2.scaled(n_rows=20000, nq=2)
    p8, _ = fill_both(w, key_format="e4m3")
    p16, _ = fill_both(w)
    q, _ = w.queries("cuda", nq=2)
    pr = fixed(16, 4, theta=-2.0)
    a, b = p8.query(q, pr).cpu(), p16.query(q, pr).cpu()
    for i in range(2):
        s16 = b.score[i].numpy()
        lead = [int(r) for r, s in zip(b.idx[i].tolist(), s16) if s > s16[-1] + 0.04]
        assert set(lead) <= set(a.idx[i].tolist())
        common = {int(r): float(s) for r, s in zip(b.idx[i].tolist(), s16)}
        for r, s in zip(a.idx[i].tolist(), a.score[i].tolist()):
            if r in common:
                assert abs(s - common[r]) < 0.02


def test_fused_steps_on_8bit_pool():
    # for nq <= 2 and up to 64 rows the 8-bit scan appends the step's rows itself
    w = W.C1.scaled(n_rows=8192, nq=1)
    pool, ora = fill_both(w, key_format="e4m3", spare_rows=8192)
    g = torch.Generator(device="cuda").manual_seed(4)
    pr = fixed(4, 4, theta=-2.0)
    steps = 120
    sizes = [8, 1, 64, 33, 100, 0]                         # 100 and 0: separate append / none
    outs, chunks = [], []
    for s in range(steps):
        n = sizes[s % len(sizes)]
        st = torch.randn(max(n, 1), w.d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 100, (max(n, 1),), generator=g, device="cuda", dtype=torch.int32)
        q = st[-1:].contiguous()
        st, tk = st[:n].contiguous(), tk[:n].contiguous()
        outs.append((n, pool.step(st, tk, q, pr, tag=700 + s, new_trace=(s % 2 == 0)), len(pool)))
        chunks.append((st, tk, s))
    torch.cuda.synchronize()
    for n, out, rows in outs:
        if n > 0:
            assert int(out.idx[0, 0]) == rows - 1
    for st, tk, s in chunks:
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=700 + s, new_trace=(s % 2 == 0))
    codes, scales = pool.read_codes()
    assert np.array_equal(codes, ora.codes) and np.array_equal(scales, ora.scales)
    _, tok, _ = pool.read_rows()
    assert np.array_equal(tok, ora.tokens)
    q = chunks[3][0][:1].contiguous()
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    assert pool.stats()["stalled"] == 0


# ------------------------------------------- warp-level tensor scan on 8-bit pools ----

@pytest.mark.parametrize("d", [256, 1024, 4096])
def test_mma_scan_closed_form_pool_scores_are_exact(d):
    # +-1 rows (codes +-448) and +-1 queries: f16 products and their sums are exact, so the
    # batch scan must return the oracle's scores, order and ties bit for bit
    rng = np.random.default_rng(d)
    n = 600
    rows = rng.choice([-1.0, 1.0], size=(n, d)).astype(np.float32)
    q = rng.choice([-1.0, 1.0], size=(5, d)).astype(np.float32)
    rows[5] = q[0]; rows[300] = q[0]; rows[599] = q[0]
    rows[17] = -q[1]
    pool = B.Pool(d, n, max_nq=8, key_format="e4m3")
    ora = OraclePool(d, "e4m3")
    rb = oracle.f32_to_bf16_bits(rows)
    tok = np.arange(n, dtype=np.int32)
    pool.append(bits_to_dev(rb), torch.from_numpy(tok).cuda(), tag=1)
    ora.append(rb, tok, tag=1)
    qb = oracle.f32_to_bf16_bits(q)
    pr = fixed(8, 2, theta=-2.0, path=B.PATH_MMA)
    l0 = pool.launch_count
    out = pool.query(bits_to_dev(qb), pr).cpu()
    assert pool.launch_count - l0 == 2
    ref = ora.query(qb, oracle.QueryParams(k=8, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=2))
    assert out.idx.numpy().tolist() == ref.idx.tolist()
    assert np.array_equal(out.score.numpy(), ref.score)
    assert out.idx[0, :3].tolist() == [5, 300, 599]


@pytest.mark.parametrize("nq,k", [(1, 8), (3, 8), (8, 16), (8, 40), (11, 8), (16, 64), (19, 5)])
def test_mma_scan_matches_oracle_and_the_cuda_core_scan(nq, k):
    w = W.C1.scaled(n_rows=6000, nq=nq, d=512)
    pool, ora = fill_both(w, key_format="e4m3", max_k=k, max_nq=32)
    q, _ = w.queries("cuda", nq=nq)
    for theta in (0.8, -2.0):
        pr = fixed(k, 8, theta=theta, path=B.PATH_MMA)
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr)
        ref = pool.query(q, fixed(k, 8, theta=theta, path=B.PATH_GEMV))
        assert torch.allclose(out.score, ref.score, atol=2e-5, rtol=0)
    # the automatic choice for three queries and more is this scan: one launch (its passes of
    # 8 or 16 queries run inside the kernel) plus the merge
    if nq >= 3:
        l0 = pool.launch_count
        pool.query(q, fixed(k, 8))
        assert pool.launch_count - l0 == 2
    assert pool.stats()["stalled"] == 0


def test_mma_scan_wide_rows_exclusion_and_ragged_sizes():
    w = W.C2.scaled(n_rows=3000, nq=6)
    pool, ora = fill_both(w, key_format="e4m3", spare_rows=64)
    q, _ = w.queries("cuda", nq=6)
    tags = [t for _, _, t in w.traces("cpu")][:2]
    ex = torch.tensor([tags[0], 0, tags[1], 0, 0, 12345], dtype=torch.int64, device="cuda")
    pr = fixed(16, 16, theta=-2.0)
    pr.exclude_tag = ex
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr, exclude=ex.cpu().numpy().astype(np.uint64))
    for n_rows in (1, 15, 17, 129, 1000):
        ws = W.C1.scaled(nq=4, d=256)
        pool2, ora2 = fill_both(ws, n_rows=n_rows, key_format="e4m3")
        q2, _ = ws.queries("cuda")
        pr2 = fixed(ws.k, ws.cont_len, theta=-2.0)
        check_query(pool2.query(q2, pr2), ora2, W.to_bits(q2), pr2)
    # a width that is not a multiple of 256 keeps the CUDA-core scan
    odd = B.Pool(384, 64, max_nq=8, key_format="e4m3")
    odd.append(torch.randn(64, 384, device="cuda").to(torch.bfloat16),
               torch.zeros(64, dtype=torch.int32, device="cuda"), tag=1)
    odd.query(torch.randn(4, 384, device="cuda").to(torch.bfloat16), fixed(8, 8))
    with pytest.raises(B.OilbirdError):
        odd.query(torch.randn(4, 384, device="cuda").to(torch.bfloat16), fixed(8, 8, path=B.PATH_MMA))


def test_mma_scan_appends_the_rows_of_a_step_itself():
    # three queries and more on an 8-bit pool: eight warps of the scan's first CTAs quantise
    # one row per CTA (two launches per step); codes and scales equal the oracle's, and a
    # query of the same step finds the new rows and honours their tag
    w = W.C1.scaled(n_rows=4096, nq=5, d=512)
    pool, ora = fill_both(w, key_format="e4m3", spare_rows=1024)
    g = torch.Generator(device="cuda").manual_seed(44)
    for step in range(8):
        n = [8, 1, 64, 33, 8, 16, 2, 8][step]
        st = torch.randn(n, w.d, generator=g, device="cuda").to(torch.bfloat16)
        if step == 3:
            st[5] = 0                                     # a zero row among the new ones
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
        if new_trace:
            assert all(int(r) < first_new for r in out.idx[0].tolist())
        assert int(out.idx[3, 0]) == first_new
        check_query(out, ora, W.to_bits(q), pr, exclude=ex.cpu().numpy().astype(np.uint64))
    assert pool.stats()["stalled"] == 0 and pool.stats()["degenerate_rows"] == 1
    codes, scales = pool.read_codes()
    assert np.array_equal(codes, ora.codes)
    assert np.array_equal(scales.view(np.uint32), ora.scales.view(np.uint32))
    _, tok, tid = pool.read_rows()
    assert np.array_equal(tok, ora.tokens) and np.array_equal(tid, ora.trace_ids)


# ---- tcgen05 scan of 8-bit pools: codes turned into f16 inside the kernel ---------------

@pytest.mark.parametrize("d", [16, 64, 256, 1024, 4096])
def test_tensor_scan_closed_form_pool_scores_are_exact(d):
    # +-1 rows (codes +-448) and +-1 queries: f16 products and their sums are exact, so the
    # scan must return the oracle's scores, order and ties bit for bit
    rng = np.random.default_rng(d + 1)
    n = 700
    rows = rng.choice([-1.0, 1.0], size=(n, d)).astype(np.float32)
    q = rng.choice([-1.0, 1.0], size=(12, d)).astype(np.float32)
    rows[5] = q[0]; rows[300] = q[0]; rows[699] = q[0]
    rows[17] = -q[1]
    pool = B.Pool(d, n, max_nq=16, key_format="e4m3")
    ora = OraclePool(d, "e4m3")
    rb = oracle.f32_to_bf16_bits(rows)
    tok = np.arange(n, dtype=np.int32)
    pool.append(bits_to_dev(rb), torch.from_numpy(tok).cuda(), tag=1)
    ora.append(rb, tok, tag=1)
    qb = oracle.f32_to_bf16_bits(q)
    pr = fixed(8, 2, theta=-2.0, path=B.PATH_TENSOR)
    l0 = pool.launch_count
    out = pool.query(bits_to_dev(qb), pr).cpu()
    assert pool.launch_count - l0 == 3                       # query preparation, scan, merge
    ref = ora.query(qb, oracle.QueryParams(k=8, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=2))
    assert out.idx.numpy().tolist() == ref.idx.tolist()
    assert np.array_equal(out.score.numpy(), ref.score)
    assert out.idx[0, :3].tolist() == [5, 300, 699]
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("nq,k", [(3, 8), (9, 8), (16, 64), (64, 16), (100, 8), (256, 64), (33, 128)])
def test_tensor_scan_matches_oracle_and_the_other_scans(nq, k):
    w = W.C1.scaled(n_rows=6000, nq=nq, d=512)
    pool, ora = fill_both(w, key_format="e4m3", max_k=128, max_nq=256)
    q, _ = w.queries("cuda", nq=nq)
    for theta in (0.8, -2.0):
        pr = fixed(k, 8, theta=theta, path=B.PATH_TENSOR)
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr)
        if k <= 64:
            ref = pool.query(q, fixed(k, 8, theta=theta, path=B.PATH_MMA))
            assert torch.allclose(out.score, ref.score, atol=2e-5, rtol=0)
        again = pool.query(q, pr).cpu()                      # bit-identical from run to run
        assert torch.equal(out.cpu().idx, again.idx) and torch.equal(out.cpu().score, again.score)
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("n_rows,d", [(148 * 128 * 2 + 77, 256), (148 * 128 * 3 + 128 + 5, 208),
                                      (1, 64), (127, 128), (129, 1024), (5000, 8192)])
def test_tensor_scan_tile_shapes_widths_and_exclusion(n_rows, d):
    # two key tiles per query tile (from two tiles per SM on), a ragged last tile, a width that
    # is not a multiple of the k-block (the codes beyond it read as zero), one row, wide rows
    w = W.C1.scaled(n_rows=max(n_rows, 2100), nq=24, k=16, d=d, cont_len=4, rows_per_trace=700,
                    n_centroids=512, seed=70 + d)
    pool, ora = fill_both(w, n_rows=n_rows, key_format="e4m3", max_k=64, max_nq=64)
    q, _ = w.queries("cuda")
    pr = fixed(16, 4, theta=-2.0, path=B.PATH_TENSOR)
    out = pool.query(q, pr)
    check_query(out, ora, W.to_bits(q), pr)
    if n_rows > 1000:
        ws = w.separated()
        pool, ora = fill_both(ws, key_format="e4m3", max_k=64, max_nq=64)
        q, _ = ws.queries("cuda")
        check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
        best = pool.query(q, pr).cpu().idx[:, 0].numpy()
        ex = np.array([ws.trace_tag(int(b) // ws.rows_per_trace) for b in best], dtype=np.int64)
        pr_ex = fixed(16, 4, theta=-2.0, path=B.PATH_TENSOR, exclude_tag=torch.from_numpy(ex).cuda())
        check_query(pool.query(q, pr_ex), ora, W.to_bits(q), pr_ex, exclude=ex.astype(np.uint64))
    assert pool.stats()["stalled"] == 0


def test_batches_on_larger_8bit_pools_take_the_tensor_scan_by_themselves():
    # more than 8 queries from 32 MB of codes on: query preparation + one scan + merge, where
    # the warp-level scan would read the codes once per 8 queries; a step adds its append
    w = W.C1.scaled(n_rows=70000, nq=20, k=8, d=512, cont_len=4, rows_per_trace=1000, seed=77)
    pool, ora = fill_both(w, key_format="e4m3", max_nq=32, spare_rows=64)
    q, _ = w.queries("cuda")
    pr = fixed(8, 4, theta=-2.0)
    l0 = pool.launch_count
    out = pool.query(q, pr)
    assert pool.launch_count - l0 == 3
    check_query(out, ora, W.to_bits(q), pr)
    g = torch.Generator(device="cuda").manual_seed(3)
    st = torch.randn(8, w.d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(8, dtype=torch.int32, device="cuda")
    q[0] = st[5]
    l0 = pool.launch_count
    out = pool.step(st, tk, q, pr, tag=4242)
    assert pool.launch_count - l0 == 4
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=4242)
    check_query(out, ora, W.to_bits(q), pr)
    assert int(out.idx[0, 0]) == len(pool) - 3
    small = pool.query(q[:8].contiguous(), pr)                   # 8 queries stay on the warp-level scan
    check_query(small, ora, W.to_bits(q[:8]), pr)
    assert pool.stats()["stalled"] == 0
