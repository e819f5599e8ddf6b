"""CPU oracle for the coarse index over the pool (test infrastructure).

The paper's Limitations section names "an index" as one of three ways to keep the cost of
the cosine lookup bounded as the store grows, and defines none.  The one built here is an
inverted file over centroids the caller supplies; what it computes, in the order the steps
are taken:

  assign   every stored row belongs to the list of the centroid that is the best neighbour
           of the row's STORED key taken as a query state (the lookup of Algorithm 1 with
           k = 1 against the centroids: cosine of the normalised vectors, ties to the lowest
           centroid);
  probe    a query's lists are the n_probe best centroids for the query state (the same
           lookup with k = n_probe);
  scan     the candidates are the rows of the probed lists plus every row appended since
           the index was last refreshed (the tail, which is always scanned); among them the
           answer is exactly Eq. 2 and Eq. 3: top-k by (score descending, row ascending),
           theta on the best, depth, continuation clipped at the trace end.

So the result is the brute-force result restricted to the candidate rows: with every list
probed it IS the brute-force result, which is the first pin.  Everything is built from
OraclePool (full scores in double, full sort); plain numpy and Python loops on purpose.

  train    Lloyd's iterations on the rows the pool holds (spherical k-means, the textbook
           procedure; the paper defines none).  One iteration: every row is assigned as
           above; then each centroid that has rows becomes the mean of its rows' stored
           keys, and a centroid without rows stays as it is.  So that the mean does not
           depend on the order of the rows it is taken in fixed point: element x of a stored
           key contributes trunc(x * 2^30) (an integer, |x| <= 1), the integers are summed
           exactly, and the new raw centroid element is bf16(float(double(sum) /
           (count * 2^30))), both roundings to nearest even.  The raw centroids then go
           through the same normalisation as at creation.  After the last iteration the lists
           are rebuilt from scratch.

8-bit pools (FP8 E4M3 codes with one fp32 scale per row).  The paper defines neither the
quantised store nor the index, so what a stored row IS, as a state, is a reading: element j of
row i is x = fp32(value(code_ij) * scale_i), the product rounded once to fp32.  Taken as a
query state (assign), the row is those elements rounded to bf16, like any state the library
is handed, and goes through the query normalisation.  In the training means the element
contributes trunc(x * 2^30) with the fp32 x itself.  Scoring, and so the scan step, is the
8-bit pool's own (OraclePool with key_format "e4m3").
"""
from __future__ import annotations

import numpy as np

from . import (DEPTH_FIXED, DEPTH_RANKED, OraclePool, QueryParams, QueryResult, depth as oracle_depth,
               depth_by_rank)


class OracleIndex:
    def __init__(self, pool: OraclePool, centroids_bits: np.ndarray):
        """centroids_bits: raw bf16 states [n_lists, d] (uint16 bit patterns)."""
        c = np.ascontiguousarray(centroids_bits, dtype=np.uint16).reshape(-1, pool.d)
        self.pool = pool
        self.n_lists = c.shape[0]
        self.cent_raw = c.copy()                       # raw centroid states (bf16 bit patterns)
        self._build_centroids()
        self.assign = np.empty(0, dtype=np.int64)      # list of every indexed row

    def _build_centroids(self) -> None:
        self.cent = OraclePool(self.pool.d)
        self.cent.append(self.cent_raw, np.arange(self.n_lists, dtype=np.int32), tag=0)

    @property
    def n_indexed(self) -> int:
        return int(self.assign.shape[0])

    def reset(self) -> None:
        self.assign = np.empty(0, dtype=np.int64)

    def _stored_f32(self, lo: int, hi: int) -> np.ndarray:
        """Rows lo..hi of the store as fp32 elements (see the header for 8-bit pools)."""
        from . import bf16_bits_to_f32, e4m3_decode
        if self.pool.key_format == "bf16":
            return bf16_bits_to_f32(self.pool.keys[lo:hi])
        value = np.array([e4m3_decode(c) for c in range(256)], dtype=np.float64)
        value[~np.isfinite(value)] = 0.0               # NaN codes are never stored
        codes, scales = self.pool.codes[lo:hi], self.pool.scales[lo:hi]
        return (value[codes] * scales.astype(np.float64)[:, None]).astype(np.float32)

    def _stored_as_queries(self, lo: int, hi: int) -> np.ndarray:
        from . import f32_to_bf16_bits
        if self.pool.key_format == "bf16":
            return self.pool.keys[lo:hi]               # stored (normalised) keys, as queries
        return f32_to_bf16_bits(self._stored_f32(lo, hi))

    def refresh(self) -> None:
        """Assign the rows appended since the last refresh."""
        n = len(self.pool)
        if n <= self.n_indexed:
            return
        keys = self._stored_as_queries(self.n_indexed, n)
        one = QueryParams(k=1, theta=-np.inf, depth_mode=DEPTH_FIXED, cont_len=1)
        new = np.empty(keys.shape[0], dtype=np.int64)
        step = 4096
        for r0 in range(0, keys.shape[0], step):
            new[r0:r0 + step] = self.cent.query(keys[r0:r0 + step], one).idx[:, 0]
        self.assign = np.concatenate([self.assign, new])

    def train(self, iterations: int) -> None:
        """Lloyd's iterations (see the header); afterwards every row of the pool is indexed."""
        from . import f32_to_bf16_bits
        for _ in range(int(iterations)):
            self.reset()
            self.refresh()
            x = self._stored_f32(0, len(self.pool)).astype(np.float64)    # stored elements, exact
            t = np.trunc(x * 2.0 ** 30).astype(np.int64)
            for l in range(self.n_lists):
                rows = np.nonzero(self.assign == l)[0]
                if rows.size == 0:
                    continue                                              # keeps its centroid
                total = t[rows].sum(axis=0, dtype=np.int64)               # exact, any order
                mean = total.astype(np.float64) / (float(rows.size) * 2.0 ** 30)
                self.cent_raw[l] = f32_to_bf16_bits(mean.astype(np.float32))
            self._build_centroids()
        self.reset()
        self.refresh()

    def lists(self) -> list[np.ndarray]:
        return [np.nonzero(self.assign == l)[0] for l in range(self.n_lists)]

    def probes(self, q_bits: np.ndarray, n_probe: int) -> np.ndarray:
        """[nq, n_probe] centroid ids, best first, -1 where fewer than n_probe exist."""
        pr = QueryParams(k=n_probe, theta=-np.inf, depth_mode=DEPTH_FIXED, cont_len=1)
        return self.cent.query(q_bits, pr).idx

    def candidates(self, probes_q: np.ndarray) -> np.ndarray:
        """Row mask [N]: rows of the probed lists, and the tail."""
        n = len(self.pool)
        mask = np.zeros(n, dtype=bool)
        good = probes_q[probes_q >= 0]
        mask[: self.n_indexed] = np.isin(self.assign, good)
        mask[self.n_indexed:] = True
        return mask

    def query(self, q_bits: np.ndarray, n_probe: int, params: QueryParams | None = None,
              want_all_scores: bool = False) -> QueryResult:
        pr = params or QueryParams()
        q = np.ascontiguousarray(q_bits, dtype=np.uint16).reshape(-1, self.pool.d)
        nq, k, L = q.shape[0], int(pr.k), int(pr.cont_len)
        full = self.pool.query(q, pr, want_all_scores=True)    # scores of EVERY row (exclusion applied)
        probes = self.probes(q, n_probe)
        idx = np.full((nq, k), -1, dtype=np.int64)
        score = np.full((nq, k), -np.inf, dtype=np.float32)
        fired = np.zeros(nq, dtype=np.int32)
        clen = np.zeros((nq, k), dtype=np.int32)
        ctok = np.full((nq, k, L), -1, dtype=np.int32)
        alls = np.full((nq, len(self.pool)), -np.inf, dtype=np.float32)
        for i in range(nq):
            s = full.all_scores[i].copy()
            s[~self.candidates(probes[i])] = -np.inf           # only candidates can be neighbours
            alls[i] = s
            rows = np.nonzero(np.isfinite(s))[0]
            order = rows[np.lexsort((rows, -s[rows].astype(np.float64)))]   # score desc, row asc
            top = order[:k]
            idx[i, : len(top)] = top
            score[i, : len(top)] = s[top]
            fired[i] = int(len(top) > 0 and np.float32(s[top[0]]) >= np.float32(pr.theta))
            for j, r in enumerate(top):
                dep = 0
                if fired[i]:
                    if pr.depth_mode == DEPTH_FIXED:
                        dep = L
                    elif pr.depth_mode == DEPTH_RANKED:
                        dep = depth_by_rank(j, pr.tier_depth)
                    else:
                        dep = oracle_depth(float(s[r]), pr.tier_thr, pr.tier_depth)
                tok, n = self.pool.gather_one(int(r), dep, pr.offset, L)
                ctok[i, j], clen[i, j] = tok, n
        return QueryResult(idx, score, fired, clen, ctok, alls if want_all_scores else None)
