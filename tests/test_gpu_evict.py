"""GPU parity for eviction (bounded store): after dropping the oldest traces the CUDA pool
must hold exactly what the oracle holds after the same eviction, bit for bit, and keep
answering queries, steps and appends like it."""
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


def same_store(pool, ora):
    if pool.key_format == "bf16":
        keys, tok, tid = pool.read_rows()
        assert np.array_equal(keys, ora.keys)
    else:
        _, tok, tid = pool.read_rows()
        codes, scales = pool.read_codes()
        assert np.array_equal(codes, ora.codes) and np.array_equal(scales, ora.scales)
    assert np.array_equal(tok, ora.tokens) and np.array_equal(tid, ora.trace_ids)
    st, en, tg = pool.traces()
    assert np.array_equal(st, ora.trace_starts) and np.array_equal(en, ora.trace_ends)
    assert np.array_equal(tg, ora.trace_tags)
    assert len(pool) == len(ora) and pool.num_traces == ora.num_traces


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
@pytest.mark.parametrize("drop", [1, 5, 15, 16, 40])
def test_evict_matches_oracle(fmt, drop):
    w = W.C1.scaled(nq=4)                       # 16 traces of 256 rows
    pool, ora = fill_both(w, key_format=fmt, spare_rows=512)
    n0 = len(pool)
    dropped = pool.evict_oldest(drop)
    assert dropped == ora.evict_oldest(drop) == min(drop, 16) * 256
    assert len(pool) == n0 - dropped
    same_store(pool, ora)
    q, _ = w.queries("cuda")
    if len(pool):
        paths = (B.PATH_GEMV,) if fmt == "e4m3" else (B.PATH_GEMV, B.PATH_TENSOR)
        for path in paths:
            pr = fixed(8, 8, theta=-2.0, path=path)
            check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    # life goes on: a fused step, an append to the open trace, another eviction
    g = torch.Generator(device="cuda").manual_seed(drop)
    st = torch.randn(8, w.d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(8, dtype=torch.int32, device="cuda")
    pr = fixed(4, 4, theta=-2.0)
    out = pool.step(st, tk, st[5:6].contiguous(), pr, tag=4242)
    ora.append(W.to_bits(st), tk.cpu().numpy(), tag=4242)
    assert int(out.idx[0, 0]) == len(pool) - 3
    pool.append(st[:3].contiguous(), tk[:3].contiguous(), new_trace=False)
    ora.append(W.to_bits(st[:3]), tk[:3].cpu().numpy(), new_trace=False)
    same_store(pool, ora)
    pool.evict_oldest(1)
    ora.evict_oldest(1)
    same_store(pool, ora)
    assert pool.stats()["stalled"] == 0


def test_many_waves_a_short_trace_in_front_of_a_long_pool():
    # 3 rows dropped in front of ~5000 (a prefix far smaller than what remains)
    d = 64
    g = torch.Generator(device="cuda").manual_seed(1)
    pool, ora = B.Pool(d, 6000), OraclePool(d)
    for n, tag in ((3, 1), (2500, 2), (7, 3), (2490, 4)):
        st = torch.randn(n, d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 1000, (n,), generator=g, device="cuda", dtype=torch.int32)
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    assert pool.evict_oldest(1) == ora.evict_oldest(1) == 3
    same_store(pool, ora)
    assert pool.evict_oldest(2) == ora.evict_oldest(2) == 2507
    same_store(pool, ora)
    assert pool.evict_oldest(0) == 0 and pool.evict_oldest(9) == 2490
    assert len(pool) == 0 and pool.num_traces == 0
    # an emptied pool starts over
    st = torch.randn(5, d, generator=g, device="cuda").to(torch.bfloat16)
    pool.append(st, torch.arange(5, dtype=torch.int32, device="cuda"), tag=9)
    out = pool.query(st[2:3].contiguous(), fixed(1, 2, theta=-2.0))
    assert int(out.idx[0, 0]) == 2 and out.cont_tok[0, 0].tolist() == [4, -1]


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
def test_one_row_dropped_in_front_of_a_pool_of_several_waves(fmt):
    # a one-row trace in front of 20,000 rows: the fixed-size register-staged waves (about
    # 600,000 16-byte chunks each on a B200) pass several times, with a ragged last wave; the
    # barrier count must not depend on the size of the dropped prefix
    d = 1024
    g = torch.Generator(device="cuda").manual_seed(11)
    pool, ora = B.Pool(d, 21000, key_format=fmt), OraclePool(d, fmt)
    for n, tag in ((1, 1), (9000, 2), (2, 3), (10997, 4)):
        st = torch.randn(n, d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 1000, (n,), generator=g, device="cuda", dtype=torch.int32)
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    assert pool.evict_oldest(1) == ora.evict_oldest(1) == 1
    same_store(pool, ora)
    q = torch.randn(1, d, generator=g, device="cuda").to(torch.bfloat16)
    pr = fixed(8, 4, theta=-2.0)
    check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    assert pool.evict_oldest(2) == ora.evict_oldest(2) == 9002
    same_store(pool, ora)


def test_large_prefix_takes_the_streaming_form():
    # 1,700 rows of 8 KB in front (14 MB, more than one staged wave): waves of `head` rows
    d = 4096
    g = torch.Generator(device="cuda").manual_seed(12)
    pool, ora = B.Pool(d, 6000), OraclePool(d)
    for n, tag in ((1700, 1), (2100, 2), (1500, 3)):
        st = torch.randn(n, d, generator=g, device="cuda").to(torch.bfloat16)
        tk = torch.randint(0, 1000, (n,), generator=g, device="cuda", dtype=torch.int32)
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    assert pool.evict_oldest(1) == ora.evict_oldest(1) == 1700
    same_store(pool, ora)


def test_evicting_empty_traces_still_renumbers():
    d = 32
    g = torch.Generator(device="cuda").manual_seed(3)
    pool, ora = B.Pool(d, 100), OraclePool(d)
    empty = torch.empty(0, d, dtype=torch.bfloat16, device="cuda")
    none = torch.empty(0, dtype=torch.int32, device="cuda")
    for n, tag in ((0, 1), (0, 2), (9, 3), (0, 4), (5, 5)):
        st = torch.randn(n, d, generator=g, device="cuda").to(torch.bfloat16) if n else empty
        tk = torch.arange(n, dtype=torch.int32, device="cuda") if n else none
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st) if n else np.empty((0, d), np.uint16), tk.cpu().numpy(), tag=tag)
    assert pool.evict_oldest(2) == ora.evict_oldest(2) == 0        # two empty traces
    same_store(pool, ora)
    assert pool.evict_oldest(2) == ora.evict_oldest(2) == 9        # one full, one empty
    same_store(pool, ora)


def test_eviction_keeps_global_positions_of_a_shard():
    d = 32
    g = torch.Generator(device="cuda").manual_seed(2)
    pool = B.Pool(d, 1000)
    bases = [100, 5000, 70000]
    for i, gb in enumerate(bases):
        st = torch.randn(10, d, generator=g, device="cuda").to(torch.bfloat16)
        pool.append_global(st, torch.arange(10, dtype=torch.int32, device="cuda"), gb, tag=i + 1)
    pool.evict_oldest(1)
    idx = torch.tensor([0, 9, 10, 19, -1], dtype=torch.int32, device="cuda")
    assert pool.to_global(idx).tolist() == [5000, 5009, 70000, 70009, -1]


def fewest_traces_to_go(ora, n, capacity, max_traces, open_new):
    """The definition of OILBIRD_EVICT_TO_FIT, by trying every count in turn."""
    ends = ora.trace_ends.tolist()
    have = len(ends)
    may_go = have if open_new else have - 1
    for nt in range(0, may_go + 1):
        dropped = ends[nt - 1] if nt else 0
        if len(ora) - dropped + n <= capacity and (not open_new or have - nt < max_traces):
            return nt
    return None


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
def test_appends_and_steps_that_evict_to_fit(fmt):
    """A bounded store: appends and steps that do not fit drop the fewest oldest traces first,
    exactly as oilbird_pool_evict_oldest would; everything else is as after that eviction."""
    d, cap, max_traces = 256, 1000, 7
    pool = B.Pool(d, cap, max_traces=max_traces, max_nq=8, key_format=fmt)
    ora = OraclePool(d, fmt)
    g = torch.Generator(device="cuda").manual_seed(21)
    next_tag = [100]

    def rows(n):
        st = torch.randn(n, d, generator=g, device="cuda").to(torch.bfloat16)
        return st, torch.randint(0, 1000, (n,), generator=g, device="cuda", dtype=torch.int32)

    def both(n, new=True, step_nq=0, host=False):
        st, tk = rows(n)
        tag = next_tag[0]; next_tag[0] += 1
        nt = fewest_traces_to_go(ora, n, cap, max_traces, new or ora.num_traces == 0)
        assert nt is not None
        gen0 = pool.num_traces
        if step_nq:
            q = rows(step_nq)[0]
            if n:
                q[0] = st[n - 1]
            pr = fixed(4, 4, theta=-2.0)
            if host:
                out = B.QueryOut.empty(step_nq, 4, 4, "cpu")
                pool.step_host(st.cpu(), tk.cpu(), q.cpu(), pr, out, tag=tag, new_trace=new, evict_to_fit=True)
            else:
                out = pool.step(st, tk, q, pr, tag=tag, new_trace=new, evict_to_fit=True)
        elif host:
            pool.append_host(st.cpu(), tk.cpu(), tag=tag, new_trace=new, evict_to_fit=True)
        else:
            pool.append(st, tk, tag=tag, new_trace=new, evict_to_fit=True)
        ora.evict_oldest(nt)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag, new_trace=new)
        same_store(pool, ora)
        if step_nq:
            check_query(out, ora, W.to_bits(q), pr)
            if n:
                assert int(out.idx[0, 0]) == len(pool) - 1
        return nt

    for _ in range(5):
        assert both(200) == 0                     # 1,000 rows, 5 traces: full
    assert both(150) == 1                         # one trace goes: 950 rows
    assert both(50) == 0                          # fits exactly
    assert both(8, step_nq=1) == 1                # a fused step that has to make room
    assert both(100, new=False) == 0              # the open trace grows into the room left
    assert both(300, step_nq=3) >= 1              # a step with its own append kernel
    assert both(120, host=True) >= 0
    assert both(64, step_nq=2, host=True) >= 0
    # the trace table fills before the rows do: one-row traces
    for _ in range(2 * max_traces):
        both(1)
    assert pool.num_traces == max_traces
    # the open trace is never evicted: extending it beyond what the others can free is refused
    while ora.num_traces > 1:
        pool.evict_oldest(1); ora.evict_oldest(1)
    room = cap - len(ora)
    st, tk = rows(room + 1)
    before = (len(pool), pool.num_traces)
    with pytest.raises(B.OilbirdError) as e:
        pool.append(st, tk, new_trace=False, evict_to_fit=True)
    assert e.value.code == B.ECAPACITY and (len(pool), pool.num_traces) == before
    # ... but as a new trace the same rows fit once the old one has gone
    assert both(room + 1) == 1
    # more rows than the pool holds at all
    st, tk = rows(cap + 1)
    with pytest.raises(B.OilbirdError) as e:
        pool.append(st, tk, tag=1, evict_to_fit=True)
    assert e.value.code == B.ECAPACITY
    # a refused step evicts nothing
    both(600)
    before = (len(pool), pool.num_traces)
    st, tk = rows(700)
    with pytest.raises(B.OilbirdError) as e:
        pool.step(st, tk, st[:2].contiguous(), fixed(4, 4, path=9), tag=5, evict_to_fit=True)
    assert e.value.code == B.EINVAL and (len(pool), pool.num_traces) == before
    same_store(pool, ora)
    assert pool.stats()["stalled"] == 0
