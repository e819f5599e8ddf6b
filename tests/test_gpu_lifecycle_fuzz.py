"""Randomised life cycles: a seeded sequence of appends, fused steps, evictions, resets and
queries is applied to the CUDA pool and to the oracle alike; after every operation that
returns results they are compared under the acceptance rule, and at the end (and after every
eviction) the stored arrays must be identical bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query

pytestmark = pytest.mark.gpu


def fewest_traces_to_go(ora, n, capacity, max_traces, open_new):
    """OILBIRD_EVICT_TO_FIT by its definition: the first count that makes room."""
    ends = ora.trace_ends.tolist()
    have = len(ends)
    for nt in range(0, (have if open_new else have - 1) + 1):
        dropped = ends[nt - 1] if nt else 0
        if len(ora) - dropped + n <= capacity and (not open_new or have - nt < max_traces):
            return nt
    return None


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


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
@pytest.mark.parametrize("seed", range(8))
def test_random_life_cycle(fmt, seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 256, 1024]))
    cap = 6000
    pool = B.Pool(d, cap, max_nq=8, max_k=32, max_traces=400, max_append=256, key_format=fmt)
    ora = OraclePool(d, fmt)
    g = torch.Generator(device="cuda").manual_seed(seed)
    cent = torch.randn(16, d, generator=g, device="cuda")
    next_tag = [1]

    def rows(n):
        c = torch.randint(0, 16, (n,), generator=g, device="cuda")
        st = (cent[c] + 0.3 * torch.randn(n, d, generator=g, device="cuda")).to(torch.bfloat16)
        tk = torch.randint(0, 5000, (n,), generator=g, device="cuda", dtype=torch.int32)
        return st, tk

    def params(nq):
        k = int(rng.choice([1, 4, 8, 17, 32]))
        pr = B.QueryParams(k=k, theta=float(rng.choice([-2.0, 0.5, 0.8])),
                           depth_mode=int(rng.choice([B.DEPTH_FIXED, B.DEPTH_TIERED, B.DEPTH_RANKED])),
                           cont_len=int(rng.choice([1, 4, 16])), offset=int(rng.choice([0, 1, 2])))
        if fmt == "bf16" and nq >= 1:
            paths = [B.PATH_AUTO, B.PATH_GEMV, B.PATH_TENSOR] + ([B.PATH_MMA] * 2 if d % 128 == 0 else [])
            pr.path = int(rng.choice(paths))
        return pr

    for op_no in range(100):
        op = rng.choice(["append", "step", "step", "query", "evict", "reset"],
                        p=[0.25, 0.2, 0.2, 0.2, 0.12, 0.03])
        if op in ("append", "step"):
            n = int(rng.choice([0, 1, 7, 8, 40, 64, 65, 200]))
            fit = False
            if len(pool) + n > cap or pool.num_traces + 1 > 390:
                if rng.random() < 0.5:
                    fit = True                   # the call makes its own room
                else:
                    op, n = "evict", 0
        host = bool(rng.random() < 0.3)          # through the host-buffer entry points
        if op == "append":
            st, tk = rows(n)
            new = bool(rng.random() < 0.7) or len(pool) == 0 or fit
            tag = next_tag[0]; next_tag[0] += 1
            if host:
                pool.append_host(st.cpu(), tk.cpu(), tag=tag, new_trace=new, evict_to_fit=fit)
            else:
                pool.append(st, tk, tag=tag, new_trace=new, evict_to_fit=fit)
            if fit:
                ora.evict_oldest(fewest_traces_to_go(ora, n, cap, 400, True))
            ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag, new_trace=new)
        elif op == "step":
            st, tk = rows(n)
            nq = int(rng.choice([1, 1, 2, 3, 8]))
            q = rows(nq)[0]
            if n > 0:
                q[0] = st[n - 1]
            new = bool(rng.random() < 0.7) or len(pool) == 0 or fit
            tag = next_tag[0]; next_tag[0] += 1
            pr = params(nq)
            in_flight = host and bool(rng.random() < 0.5)   # the two-halves form of the host step
            if in_flight:
                out = B.QueryOut.empty(nq, pr.k, pr.cont_len, "cpu")
                slot = int(rng.integers(0, 2))
                pool.step_host_begin(st.cpu(), tk.cpu(), q.cpu(), pr, slot, tag=tag, new_trace=new,
                                     evict_to_fit=fit)
            elif host:
                out = B.QueryOut.empty(nq, pr.k, pr.cont_len, "cpu")
                pool.step_host(st.cpu(), tk.cpu(), q.cpu(), pr, out, tag=tag, new_trace=new,
                               evict_to_fit=fit)
            else:
                out = pool.step(st, tk, q, pr, tag=tag, new_trace=new, evict_to_fit=fit)
            if fit:
                ora.evict_oldest(fewest_traces_to_go(ora, n, cap, 400, True))
            ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag, new_trace=new)
            if in_flight:
                if len(ora) and rng.random() < 0.7:      # other lookups while the step is in flight
                    q2 = rows(2)[0]
                    pr2 = params(2)
                    o2 = pool.query_host(q2.cpu(), pr2) if rng.random() < 0.5 else pool.query(q2, pr2)
                    check_query(o2, ora, W.to_bits(q2), pr2)
                pool.step_host_end(slot, out)
            if len(ora):
                check_query(out, ora, W.to_bits(q), pr)
        elif op == "query":
            nq = int(rng.choice([1, 2, 5, 8]))
            q = rows(nq)[0]
            pr = params(nq)
            out = pool.query_host(q.cpu(), pr) if host else pool.query(q, pr)
            check_query(out, ora, W.to_bits(q), pr)
        elif op == "evict":
            nt = int(rng.integers(0, max(2, pool.num_traces // 2 + 1)))
            assert pool.evict_oldest(nt) == ora.evict_oldest(nt)
            same_store(pool, ora)
        else:
            pool.reset()
            ora.reset()
        assert len(pool) == len(ora) and pool.num_traces == ora.num_traces
    same_store(pool, ora)
    assert pool.stats()["stalled"] == 0


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
@pytest.mark.parametrize("seed", range(4))
def test_random_life_cycle_with_an_index(fmt, seed):
    """Appends, refreshes, lookups (one launch and separate launches), training, evictions and
    resets in a seeded order, the coarse index and its oracle side by side: lists identical
    after every refresh, answers under the acceptance rule on the candidate rows."""
    from oracle.index import OracleIndex
    from test_gpu_index import check_index_query, same_lists
    rng = np.random.default_rng(2000 + seed)
    d = int(rng.choice([128, 512]))
    cap, n_lists = 5000, 12
    pool = B.Pool(d, cap, max_nq=8, max_k=32, max_traces=200, key_format=fmt)
    ora = OraclePool(d, fmt)
    g = torch.Generator(device="cuda").manual_seed(50 + seed)
    cent = torch.randn(n_lists, d, generator=g, device="cuda")
    cent_bf = cent.to(torch.bfloat16).contiguous()
    gix, oix = B.Index(pool, cent_bf), OracleIndex(ora, W.to_bits(cent_bf))
    tag = [1]

    def rows(n):
        # well inside a cluster: the best two centroids of a row stay apart, so the lists
        # cannot depend on the accumulation order
        c = torch.randint(0, n_lists, (n,), generator=g, device="cuda")
        return (cent[c] + 0.15 * torch.randn(n, d, generator=g, device="cuda")).to(torch.bfloat16), \
            torch.randint(0, 5000, (n,), generator=g, device="cuda", dtype=torch.int32)

    for _ in range(45):
        op = rng.choice(["append", "refresh", "lookup", "lookup", "train", "evict", "reset"],
                        p=[0.3, 0.15, 0.2, 0.2, 0.05, 0.07, 0.03])
        if op == "append":
            n = int(rng.choice([1, 8, 60, 300]))
            if len(pool) + n > cap or pool.num_traces + 1 > 190:
                op = "evict"
            else:
                st, tk = rows(n)
                pool.append(st, tk, tag=tag[0])
                ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag[0])
                tag[0] += 1
        if op == "refresh":
            gix.refresh(); oix.refresh()
            assert len(gix) == len(pool)
            same_lists(gix, oix)
        elif op == "lookup" and len(ora):
            nq = int(rng.choice([1, 1, 2, 5]))
            q = rows(nq)[0]
            pr = B.QueryParams(k=int(rng.choice([1, 8, 32])), theta=float(rng.choice([-2.0, 0.8])),
                               depth_mode=int(rng.choice([B.DEPTH_FIXED, B.DEPTH_TIERED, B.DEPTH_RANKED])),
                               cont_len=int(rng.choice([2, 16])),
                               path=int(rng.choice([B.PATH_AUTO, B.PATH_AUTO, B.PATH_GEMV])))
            n_probe = int(rng.choice([1, 3, n_lists, 40]))
            check_index_query(gix.query(q, n_probe, pr), oix, W.to_bits(q), n_probe, pr)
        elif op == "train" and len(ora):
            gix.train(1); oix.train(1)
            assert np.array_equal(gix.centroids(), oix.cent_raw)
            same_lists(gix, oix)
        elif op == "evict" and pool.num_traces:
            nt = int(rng.integers(1, pool.num_traces + 1))
            assert pool.evict_oldest(nt) == ora.evict_oldest(nt)
            if len(gix) > 0:
                with pytest.raises(B.OilbirdError):
                    gix.refresh()                  # row numbers changed: a reset comes first
            gix.reset(); oix.reset()
            gix.refresh(); oix.refresh()
            same_lists(gix, oix)
        elif op == "reset":
            pool.reset(); ora.reset()
            gix.reset(); oix.reset()
    gix.refresh(); oix.refresh()
    same_lists(gix, oix)
    assert pool.stats()["stalled"] == 0 and pool.status() == B.OK
