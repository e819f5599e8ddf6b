"""CPU oracle for the Oilbird semantic-pool retrieval path (test infrastructure).

This package is NOT part of the product.  It wraps ``oilbird_oracle.c`` (plain C,
double precision, full sort) with ctypes and numpy so that tests, the smoke check
and the benchmark's CPU-baseline leg can compare the CUDA library against the
definition the paper gives (Section 4 "(i) Store" / "(ii) Retrieve", Eq. 1-3,
Algorithm 1).  It imports nothing from the CUDA package and the CUDA package
imports nothing from here.

bf16 data crosses this interface as ``numpy.uint16`` arrays holding the raw bit
patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oilbird_oracle.c")
_LIB = os.path.join(_HERE, "liboilbird_oracle.so")

DEPTH_FIXED = 0
DEPTH_TIERED = 1
DEPTH_RANKED = 2          # granularity ablation: depth by neighbour rank (tier_depth[j])

# Constants the paper prints (Algorithm 1's Require line; Eq. 3).
PAPER_K = 8
PAPER_THETA = 0.8
PAPER_OFFSET = 2
PAPER_TIER_THR = (0.90, 0.82)
PAPER_TIER_DEPTH = (48, 8)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over pool rows). Returns the .so path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
           "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    L = ctypes.CDLL(build())
    vp, i32, i64, u64, f32 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                              ctypes.c_uint64, ctypes.c_float)
    L.oracle_bf16_to_f32.restype = f32
    L.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
    L.oracle_f32_to_bf16.restype = ctypes.c_uint16
    L.oracle_f32_to_bf16.argtypes = [f32]
    L.oracle_pool_create.restype = vp
    L.oracle_pool_create.argtypes = [i32]
    L.oracle_pool_create_e4m3.restype = vp
    L.oracle_pool_create_e4m3.argtypes = [i32]
    L.oracle_e4m3_decode.restype = ctypes.c_double
    L.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
    L.oracle_e4m3_encode.restype = ctypes.c_uint8
    L.oracle_e4m3_encode.argtypes = [ctypes.c_double]
    L.oracle_quantize_e4m3.restype = ctypes.c_int
    L.oracle_quantize_e4m3.argtypes = [i32, vp, vp, vp]
    for name in ("codes", "scales"):
        fn = getattr(L, "oracle_pool_" + name)
        fn.restype = vp
        fn.argtypes = [vp]
    L.oracle_pool_evict_oldest.restype = i64
    L.oracle_pool_evict_oldest.argtypes = [vp, i32]
    L.oracle_pool_destroy.restype = None
    L.oracle_pool_destroy.argtypes = [vp]
    L.oracle_pool_reset.restype = None
    L.oracle_pool_reset.argtypes = [vp]
    L.oracle_pool_size.restype = i64
    L.oracle_pool_size.argtypes = [vp]
    L.oracle_pool_num_traces.restype = i32
    L.oracle_pool_num_traces.argtypes = [vp]
    L.oracle_pool_degenerate_rows.restype = i64
    L.oracle_pool_degenerate_rows.argtypes = [vp]
    for name in ("keys", "tokens", "trace_ids", "trace_starts", "trace_ends", "trace_tags"):
        fn = getattr(L, "oracle_pool_" + name)
        fn.restype = vp
        fn.argtypes = [vp]
    L.oracle_normalize_bf16.restype = ctypes.c_int
    L.oracle_normalize_bf16.argtypes = [i32, vp, vp]
    L.oracle_pool_append.restype = ctypes.c_int
    L.oracle_pool_append.argtypes = [vp, vp, vp, i64, u64, ctypes.c_int]
    L.oracle_scores.restype = ctypes.c_int
    L.oracle_scores.argtypes = [vp, vp, u64, vp]
    L.oracle_depth.restype = i32
    L.oracle_depth.argtypes = [f32, i32, vp, vp]
    L.oracle_depth_by_rank.restype = i32
    L.oracle_depth_by_rank.argtypes = [i32, i32, vp]
    L.oracle_gather_one.restype = i32
    L.oracle_gather_one.argtypes = [vp, i64, i32, i32, i32, vp]
    L.oracle_pool_query.restype = ctypes.c_int
    L.oracle_pool_query.argtypes = [vp, vp, i32, i32, f32, i32, i32, i32, i32, vp, vp, vp,
                                    vp, vp, vp, vp, vp, vp]
    L.oracle_ring_create.restype = vp
    L.oracle_ring_create.argtypes = [i32, i64, i32]
    L.oracle_ring_destroy.restype = None
    L.oracle_ring_destroy.argtypes = [vp]
    L.oracle_ring_reset.restype = None
    L.oracle_ring_reset.argtypes = [vp]
    L.oracle_ring_size.restype = i64
    L.oracle_ring_size.argtypes = [vp]
    L.oracle_ring_total.restype = i64
    L.oracle_ring_total.argtypes = [vp]
    for name in ("keys", "anchors", "rollouts"):
        fn = getattr(L, "oracle_ring_" + name)
        fn.restype = vp
        fn.argtypes = [vp]
    L.oracle_ring_append.restype = None
    L.oracle_ring_append.argtypes = [vp, vp, vp, vp, i64]
    L.oracle_ring_query.restype = ctypes.c_int
    L.oracle_ring_query.argtypes = [vp, vp, vp, i32, i32, f32, vp, vp, vp, vp, vp]
    L.oracle_num_threads.restype = i32
    L.oracle_num_threads.argtypes = []
    _lib = L
    return L


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 data must be passed as uint16 bit patterns")
    return a


def f32_to_bf16_bits(x) -> np.ndarray:
    """Round float32 values to bf16 bit patterns with the oracle's own helper."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    L = lib()
    out = np.empty(x.shape, dtype=np.uint16)
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = L.oracle_f32_to_bf16(float(flat_in[i]))
    return out


def bf16_bits_to_f32(b) -> np.ndarray:
    """Exact widening of bf16 bit patterns (plain shift; used by tests)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def normalize_bf16(x) -> tuple[np.ndarray, bool]:
    x = _u16(x).reshape(-1)
    out = np.empty_like(x)
    ok = lib().oracle_normalize_bf16(x.size, _ptr(x), _ptr(out))
    return out, bool(ok)


def e4m3_decode(code: int) -> float:
    return float(lib().oracle_e4m3_decode(int(code)))


def e4m3_encode(x: float) -> int:
    return int(lib().oracle_e4m3_encode(float(x)))


def quantize_e4m3(x) -> tuple[np.ndarray, float, bool]:
    """One raw bf16 row -> (E4M3 codes uint8 [d], fp32 scale, usable)."""
    x = _u16(x).reshape(-1)
    codes = np.empty(x.size, np.uint8)
    scale = np.zeros(1, np.float32)
    ok = lib().oracle_quantize_e4m3(x.size, _ptr(x), _ptr(codes), _ptr(scale))
    return codes, float(scale[0]), bool(ok)


@dataclass
class QueryParams:
    """Retrieval parameters; defaults are the values the paper deploys."""
    k: int = PAPER_K
    theta: float = PAPER_THETA
    offset: int = PAPER_OFFSET
    depth_mode: int = DEPTH_TIERED
    cont_len: int = 48
    tier_thr: tuple = PAPER_TIER_THR
    tier_depth: tuple = PAPER_TIER_DEPTH
    exclude_tag: np.ndarray | None = None  # [nq] uint64, 0 = no exclusion


@dataclass
class QueryResult:
    idx: np.ndarray        # [nq,k] int64
    score: np.ndarray      # [nq,k] float32
    fired: np.ndarray      # [nq]   int32
    cont_len: np.ndarray   # [nq,k] int32
    cont_tok: np.ndarray   # [nq,k,L] int32
    all_scores: np.ndarray | None = field(default=None)  # [nq,N] float32


class OraclePool:
    def __init__(self, d: int, key_format: str = "bf16"):
        self._L = lib()
        self.d = int(d)
        if key_format not in ("bf16", "e4m3"):
            raise ValueError("key_format must be 'bf16' or 'e4m3'")
        self.key_format = key_format
        self._h = (self._L.oracle_pool_create(self.d) if key_format == "bf16"
                   else self._L.oracle_pool_create_e4m3(self.d))
        if not self._h:
            raise MemoryError("oracle_pool_create failed")

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._L.oracle_pool_destroy(h)

    def __len__(self) -> int:
        return int(self._L.oracle_pool_size(self._h))

    def reset(self) -> None:
        self._L.oracle_pool_reset(self._h)

    def evict_oldest(self, n_traces: int) -> int:
        """Drop the n_traces oldest traces; rows and traces are renumbered. Returns rows dropped."""
        return int(self._L.oracle_pool_evict_oldest(self._h, int(n_traces)))

    def append(self, states, tokens, tag: int = 0, new_trace: bool = True) -> None:
        states = _u16(states).reshape(-1, self.d)
        tokens = np.ascontiguousarray(tokens, dtype=np.int32).reshape(-1)
        if states.shape[0] != tokens.shape[0]:
            raise ValueError("states and tokens disagree on the number of rows")
        rc = self._L.oracle_pool_append(self._h, _ptr(states), _ptr(tokens), states.shape[0],
                                        int(tag), int(bool(new_trace)))
        if rc != 0:
            raise MemoryError("oracle_pool_append failed")

    # -- views of the store (copies) ------------------------------------------
    def _copy(self, name, count, dtype):
        p = getattr(self._L, "oracle_pool_" + name)(self._h)
        if count == 0 or not p:
            return np.empty(0, dtype=dtype)
        buf = (ctypes.c_char * (count * np.dtype(dtype).itemsize)).from_address(p)
        return np.frombuffer(buf, dtype=dtype, count=count).copy()

    @property
    def keys(self) -> np.ndarray:
        return self._copy("keys", len(self) * self.d, np.uint16).reshape(len(self), self.d)

    @property
    def codes(self) -> np.ndarray:
        """E4M3 codes [N,d] uint8 (8-bit pools only)."""
        return self._copy("codes", len(self) * self.d, np.uint8).reshape(len(self), self.d)

    @property
    def scales(self) -> np.ndarray:
        """One fp32 scale per row (8-bit pools only)."""
        return self._copy("scales", len(self), np.float32)

    @property
    def tokens(self) -> np.ndarray:
        return self._copy("tokens", len(self), np.int32)

    @property
    def trace_ids(self) -> np.ndarray:
        return self._copy("trace_ids", len(self), np.int32)

    @property
    def num_traces(self) -> int:
        return int(self._L.oracle_pool_num_traces(self._h))

    @property
    def trace_starts(self) -> np.ndarray:
        return self._copy("trace_starts", self.num_traces, np.int64)

    @property
    def trace_ends(self) -> np.ndarray:
        return self._copy("trace_ends", self.num_traces, np.int64)

    @property
    def trace_tags(self) -> np.ndarray:
        return self._copy("trace_tags", self.num_traces, np.uint64)

    @property
    def degenerate_rows(self) -> int:
        return int(self._L.oracle_pool_degenerate_rows(self._h))

    # -- retrieval ------------------------------------------------------------
    def scores(self, q, exclude_tag: int = 0) -> np.ndarray:
        q = _u16(q).reshape(self.d)
        out = np.empty(len(self), dtype=np.float32)
        self._L.oracle_scores(self._h, _ptr(q), int(exclude_tag), _ptr(out))
        return out

    def query(self, q, params: QueryParams | None = None, want_all_scores: bool = False
              ) -> QueryResult:
        pr = params or QueryParams()
        q = _u16(q).reshape(-1, self.d)
        nq, k, L = q.shape[0], int(pr.k), int(pr.cont_len)
        thr = np.asarray(pr.tier_thr, dtype=np.float32)
        dep = np.asarray(pr.tier_depth, dtype=np.int32)
        if thr.shape != dep.shape:
            raise ValueError("tier_thr and tier_depth must have the same length")
        ex = None
        if pr.exclude_tag is not None:
            ex = np.ascontiguousarray(pr.exclude_tag, dtype=np.uint64).reshape(nq)
        idx = np.empty((nq, k), dtype=np.int64)
        score = np.empty((nq, k), dtype=np.float32)
        fired = np.empty(nq, dtype=np.int32)
        clen = np.empty((nq, k), dtype=np.int32)
        ctok = np.empty((nq, k, L), dtype=np.int32)
        alls = np.empty((nq, len(self)), dtype=np.float32) if want_all_scores else None
        rc = self._L.oracle_pool_query(self._h, _ptr(q), nq, k, float(pr.theta), int(pr.offset),
                                       int(pr.depth_mode), L, int(thr.size), _ptr(thr), _ptr(dep),
                                       _ptr(ex), _ptr(idx), _ptr(score), _ptr(fired), _ptr(clen),
                                       _ptr(ctok), _ptr(alls))
        if rc != 0:
            raise MemoryError("oracle_pool_query failed")
        return QueryResult(idx, score, fired, clen, ctok, alls)

    def gather_one(self, idx: int, dep: int, offset: int, L: int) -> tuple[np.ndarray, int]:
        out = np.empty(L, dtype=np.int32)
        n = self._L.oracle_gather_one(self._h, int(idx), int(dep), int(offset), int(L), _ptr(out))
        return out, int(n)


def depth_by_rank(j: int, tier_depth=PAPER_TIER_DEPTH) -> int:
    dep = np.asarray(tier_depth, dtype=np.int32)
    return int(lib().oracle_depth_by_rank(int(j), int(dep.size), _ptr(dep)))


def depth(s: float, tier_thr=PAPER_TIER_THR, tier_depth=PAPER_TIER_DEPTH) -> int:
    thr = np.asarray(tier_thr, dtype=np.float32)
    dep = np.asarray(tier_depth, dtype=np.int32)
    return int(lib().oracle_depth(float(s), int(thr.size), _ptr(thr), _ptr(dep)))


# ------------------------------------------------------------------ recycled pool ----
PAPER_RING_M = 4          # Algorithm 1: at most 4 rejected-branch rollouts
PAPER_RING_FLOOR = 0.8    # ... whose cosine reaches 0.8
PAPER_ROLLOUT = 6         # Section 4 (i b): continuations up to six deep


@dataclass
class RingResult:
    slot: np.ndarray         # [nq,m] int64, -1 padded
    score: np.ndarray        # [nq,m] float32, -inf padded
    count: np.ndarray        # [nq] int32
    rollout: np.ndarray      # [nq,m,R] int32, -1 padded
    rollout_len: np.ndarray  # [nq,m] int32


class OracleRing:
    """Rejected-branch ring buffer (Section 4 (i b); Algorithm 1's recycled-pool line)."""

    def __init__(self, d: int, capacity: int, max_rollout: int = PAPER_ROLLOUT):
        self._L = lib()
        self.d, self.capacity, self.max_rollout = int(d), int(capacity), int(max_rollout)
        self._h = self._L.oracle_ring_create(self.d, self.capacity, self.max_rollout)
        if not self._h:
            raise MemoryError("oracle_ring_create failed")

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._L.oracle_ring_destroy(h)

    def __len__(self) -> int:
        return int(self._L.oracle_ring_size(self._h))

    @property
    def total(self) -> int:
        return int(self._L.oracle_ring_total(self._h))

    def reset(self) -> None:
        self._L.oracle_ring_reset(self._h)

    def append(self, states, anchors, rollouts) -> None:
        states = _u16(states).reshape(-1, self.d)
        anchors = np.ascontiguousarray(anchors, dtype=np.int32).reshape(-1)
        rollouts = np.ascontiguousarray(rollouts, dtype=np.int32).reshape(-1, self.max_rollout)
        assert states.shape[0] == anchors.shape[0] == rollouts.shape[0]
        self._L.oracle_ring_append(self._h, _ptr(states), _ptr(anchors), _ptr(rollouts),
                                   states.shape[0])

    def _copy(self, name, count, dtype):
        p = getattr(self._L, "oracle_ring_" + name)(self._h)
        buf = (ctypes.c_char * (count * np.dtype(dtype).itemsize)).from_address(p)
        return np.frombuffer(buf, dtype=dtype, count=count).copy()

    @property
    def keys(self) -> np.ndarray:
        return self._copy("keys", self.capacity * self.d, np.uint16).reshape(self.capacity, self.d)

    @property
    def anchors(self) -> np.ndarray:
        return self._copy("anchors", self.capacity, np.int32)

    @property
    def rollouts(self) -> np.ndarray:
        return self._copy("rollouts", self.capacity * self.max_rollout, np.int32).reshape(
            self.capacity, self.max_rollout)

    def query(self, q, anchors, m: int = PAPER_RING_M, floor: float = PAPER_RING_FLOOR
              ) -> RingResult:
        q = _u16(q).reshape(-1, self.d)
        nq = q.shape[0]
        anchors = np.ascontiguousarray(anchors, dtype=np.int32).reshape(nq)
        slot = np.empty((nq, m), np.int64)
        score = np.empty((nq, m), np.float32)
        count = np.empty(nq, np.int32)
        roll = np.empty((nq, m, self.max_rollout), np.int32)
        rlen = np.empty((nq, m), np.int32)
        rc = self._L.oracle_ring_query(self._h, _ptr(q), _ptr(anchors), nq, int(m), float(floor),
                                       _ptr(slot), _ptr(score), _ptr(count), _ptr(roll), _ptr(rlen))
        if rc != 0:
            raise MemoryError("oracle_ring_query failed")
        return RingResult(slot, score, count, roll, rlen)
