"""Randomised configurations of the whole query path against the oracle: pool size, width,
nq, k, continuation length, offset, depth mode, tiers, theta, exclusion tags and scan
kernel are all drawn at random (seeded)."""
import numpy as np
import pytest
import torch

from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(24))
def test_random_configuration(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([8, 64, 136, 256, 520, 1024, 2048]))
    n_rows = int(rng.choice([1, 7, 130, 999, 4097, 20000, 60001]))
    rows_per_trace = int(rng.choice([1, 3, 50, 257, 1000]))
    nq = int(rng.choice([1, 2, 3, 9, 16, 40, 130]))
    k = int(rng.choice([1, 2, 8, 31, 32, 33, 64, 100]))
    L = int(rng.choice([1, 2, 7, 16, 48]))
    kind = str(rng.choice(["clustered", "separated"]))
    w = W.Workload(f"F{seed}", "clustered", d=d, n_rows=n_rows, rows_per_trace=rows_per_trace,
                   vocab=1000, nq=nq, k=k, cont_len=L, seed=500 + seed,
                   n_centroids=int(rng.choice([1, 4, 64])), sigma=float(rng.choice([0.05, 0.3, 1.0])))
    if kind == "separated" and n_rows >= nq * (k + 4):
        w = w.separated()
    pool = B.Pool(w.d, w.n_rows, max_k=128, max_nq=256, max_traces=w.num_traces + 1)
    ora = OraclePool(w.d)
    for t, (st, tk, _) in enumerate(w.traces("cuda")):
        tag = int(rng.integers(1, 4))                     # few tags: exclusion bites
        pool.append(st, tk, tag=tag)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
    q, _ = w.queries("cuda")
    ex = rng.integers(0, 4, nq).astype(np.uint64) if rng.random() < 0.5 else None
    mode = int(rng.integers(0, 2))
    tiers = sorted(rng.uniform(0.0, 1.0, int(rng.integers(0, 4))).tolist(), reverse=True)
    depths = [int(x) for x in rng.integers(0, 60, len(tiers))]
    pr = B.QueryParams(k=k, theta=float(rng.choice([-2.0, 0.0, 0.5, 0.8, 0.95])),
                       offset=int(rng.integers(0, 4)), depth_mode=mode, cont_len=L,
                       tier_thr=tuple(tiers), tier_depth=tuple(depths),
                       exclude_tag=None if ex is None else torch.from_numpy(ex.view(np.int64)).cuda())
    paths = [B.PATH_GEMV, B.PATH_TENSOR, B.PATH_AUTO]
    if d % 128 == 0 and k <= 64:
        paths.append(B.PATH_MMA)                         # the warp-level tensor scan takes these
    for path in paths:
        pr.path = path
        out = pool.query(q, pr)
        check_query(out, ora, W.to_bits(q), pr, exclude=ex)
    assert pool.stats()["stalled"] == 0
    # the same pool with 8-bit keys (widths that are multiples of 16), every scan it has
    if d % 16 == 0 and n_rows <= 20000:
        pool8 = B.Pool(w.d, w.n_rows, max_k=128, max_nq=256, max_traces=w.num_traces + 1,
                       key_format="e4m3")
        ora8 = OraclePool(w.d, "e4m3")
        rng2 = np.random.default_rng(1000 + seed)
        for t, (st, tk, _) in enumerate(w.traces("cuda")):
            tag = int(rng2.integers(1, 4))
            pool8.append(st, tk, tag=tag)
            ora8.append(W.to_bits(st), tk.cpu().numpy(), tag=tag)
        paths8 = [B.PATH_GEMV, B.PATH_AUTO] + ([B.PATH_MMA] if d % 256 == 0 and k <= 64 else [])
        for path in paths8:
            pr.path = path
            check_query(pool8.query(q, pr), ora8, W.to_bits(q), pr, exclude=ex)
        assert pool8.stats()["stalled"] == 0
