"""Thin ctypes binding over the C-ABI of ``liboilbird.so`` (see ``include/oilbird.h``).

Argument marshalling only: every step of the retrieval path (normalise, score, top-k,
firing rule, depth, continuation gather) runs in the CUDA library.  torch is used for
device memory and streams.  There is no fallback: if the library cannot be loaded the
import of :func:`lib` raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

# The library chains the kernels of a step with programmatic launches only when the process
# loads CUDA modules eagerly (under lazy loading, the CUDA default, it launches plainly: the
# combination of lazy loading and chained launches was seen to dead-lock the first steps of a
# process now and then).  Asking for eager loading here buys those ~6 us per step on small
# pools; it takes effect if CUDA has not been initialised yet (importing torch does not do
# that), and the library is safe either way.
os.environ.setdefault("CUDA_MODULE_LOADING", "EAGER")

import numpy as np  # noqa: E402
import torch  # noqa: E402

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liboilbird.so")

OK, EINVAL, ECAPACITY, ENOMEM, ECUDA, ESTALL, EGUARD = 0, -1, -2, -3, -4, -5, -6
NEW_TRACE = 1
EVICT_TO_FIT = 2
EVICT_TO_FIT = 2
KEYS_E4M3 = 1          # pool flag: 8-bit keys
DEBUG_GUARDS = 2       # pool flag: sentinel bytes behind every array (see Pool.check_guards)
DEPTH_FIXED, DEPTH_TIERED, DEPTH_RANKED = 0, 1, 2
PATH_AUTO, PATH_GEMV, PATH_TENSOR, PATH_MMA = 0, 1, 2, 3
MAX_NQ, MAX_K, MAX_CONT_LEN, MAX_TIERS = 256, 128, 128, 4
HOST_SLOTS = 2


class PoolConfig(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("capacity_rows", ctypes.c_int64),
                ("max_traces", ctypes.c_int32), ("max_nq", ctypes.c_int32),
                ("max_k", ctypes.c_int32), ("max_append", ctypes.c_int32),
                ("device", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("arena", ctypes.c_void_p), ("arena_bytes", ctypes.c_size_t)]


class CQueryParams(ctypes.Structure):
    _fields_ = [("k", ctypes.c_int32), ("theta", ctypes.c_float), ("offset", ctypes.c_int32),
                ("depth_mode", ctypes.c_int32), ("cont_len", ctypes.c_int32),
                ("n_tiers", ctypes.c_int32), ("tier_thr", ctypes.c_float * MAX_TIERS),
                ("tier_depth", ctypes.c_int32 * MAX_TIERS), ("exclude_tag", ctypes.c_void_p),
                ("path", ctypes.c_int32)]


class CQueryOut(ctypes.Structure):
    _fields_ = [("idx", ctypes.c_void_p), ("score", ctypes.c_void_p), ("fired", ctypes.c_void_p),
                ("cont_len", ctypes.c_void_p), ("cont_tok", ctypes.c_void_p)]


class StaticPool(ctypes.Structure):
    _fields_ = [("keys", ctypes.c_void_p), ("tokens", ctypes.c_void_p),
                ("trace_id", ctypes.c_void_p), ("trace_end", ctypes.c_void_p),
                ("n_rows", ctypes.c_int64), ("d", ctypes.c_int32), ("device", ctypes.c_int32)]


class RingConfig(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("capacity", ctypes.c_int64),
                ("max_rollout", ctypes.c_int32), ("device", ctypes.c_int32)]


class CRingOut(ctypes.Structure):
    _fields_ = [("slot", ctypes.c_void_p), ("score", ctypes.c_void_p), ("count", ctypes.c_void_p),
                ("rollout", ctypes.c_void_p), ("rollout_len", ctypes.c_void_p)]


class MergeParams(ctypes.Structure):
    _fields_ = [("budget", ctypes.c_int32), ("max_nodes", ctypes.c_int32),
                ("min_len", ctypes.c_int32), ("root_attached", ctypes.c_int32)]


class PoolStats(ctypes.Structure):
    _fields_ = [("degenerate_rows", ctypes.c_int64), ("nonfinite_queries", ctypes.c_int64),
                ("stalled", ctypes.c_int32), ("reserved", ctypes.c_int32)]


# name -> (restype, argtypes): every symbol include/oilbird.h declares
_vp, _i32, _i64, _u64, _u32 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64,
                               ctypes.c_uint32)
SYMBOLS = {
    "oilbird_query_params_default": (None, [ctypes.POINTER(CQueryParams)]),
    "oilbird_pool_arena_bytes": (ctypes.c_size_t, [ctypes.POINTER(PoolConfig)]),
    "oilbird_pool_create": (ctypes.c_int, [ctypes.POINTER(_vp), ctypes.POINTER(PoolConfig)]),
    "oilbird_pool_reset": (ctypes.c_int, [_vp, _vp]),
    "oilbird_pool_destroy": (ctypes.c_int, [_vp]),
    "oilbird_pool_append": (ctypes.c_int, [_vp, _vp, _vp, _i64, _u64, _u32, _vp]),
    "oilbird_pool_query": (ctypes.c_int, [_vp, _vp, _i32, ctypes.POINTER(CQueryParams),
                                          ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_pool_gather": (ctypes.c_int, [_vp, _vp, _vp, _i32, ctypes.POINTER(CQueryParams),
                                           ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_pool_evict_oldest": (ctypes.c_int, [_vp, _i32, ctypes.POINTER(_i64), _vp]),
    "oilbird_pool_step": (ctypes.c_int, [_vp, _vp, _vp, _i64, _u64, _u32, _vp, _i32,
                                         ctypes.POINTER(CQueryParams),
                                         ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_pool_append_host": (ctypes.c_int, [_vp, _vp, _vp, _i64, _u64, _u32, _vp]),
    "oilbird_pool_query_host": (ctypes.c_int, [_vp, _vp, _i32, ctypes.POINTER(CQueryParams),
                                               ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_pool_step_host": (ctypes.c_int, [_vp, _vp, _vp, _i64, _u64, _u32, _vp, _i32,
                                              ctypes.POINTER(CQueryParams),
                                              ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_pool_step_host_begin": (ctypes.c_int, [_vp, _vp, _vp, _i64, _u64, _u32, _vp, _i32,
                                                    ctypes.POINTER(CQueryParams), _i32, _vp]),
    "oilbird_pool_step_host_end": (ctypes.c_int, [_vp, _i32, ctypes.POINTER(CQueryOut)]),
    "oilbird_pool_size": (_i64, [_vp]),
    "oilbird_pool_num_traces": (_i32, [_vp]),
    "oilbird_pool_status": (ctypes.c_int, [_vp, ctypes.POINTER(PoolStats), _vp]),
    "oilbird_pool_set_wait_limit": (ctypes.c_int, [_vp, _u64, _vp]),
    "oilbird_pool_stall_selftest": (ctypes.c_int, [_vp, _vp]),
    "oilbird_pool_check_guards": (ctypes.c_int, [_vp, _vp]),
    "oilbird_pool_read_rows": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "oilbird_pool_read_codes": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "oilbird_pool_read_traces": (_i32, [_vp, _vp, _vp, _vp, _i32]),
    "oilbird_pool_profile": (ctypes.c_int, [_vp, _i32]),
    "oilbird_pool_profile_read": (_i32, [_vp, _vp, _i32]),
    "oilbird_pool_launch_count": (_i64, [_vp]),
    "oilbird_ring_create": (ctypes.c_int, [ctypes.POINTER(_vp), ctypes.POINTER(RingConfig)]),
    "oilbird_ring_destroy": (ctypes.c_int, [_vp]),
    "oilbird_ring_reset": (ctypes.c_int, [_vp, _vp]),
    "oilbird_ring_size": (_i64, [_vp]),
    "oilbird_ring_total": (_i64, [_vp]),
    "oilbird_ring_append": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _vp]),
    "oilbird_ring_query": (ctypes.c_int, [_vp, _vp, _vp, _i32, _i32, ctypes.c_float,
                                          ctypes.POINTER(CRingOut), _vp]),
    "oilbird_ring_step": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _i32, _i32,
                                         ctypes.c_float, ctypes.POINTER(CRingOut), _vp]),
    "oilbird_ring_read": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "oilbird_ring_last_error": (ctypes.c_char_p, []),
    "oilbird_pool_append_global": (ctypes.c_int, [_vp, _vp, _vp, _i64, _u64, _u32, _i64, _vp]),
    "oilbird_pool_to_global": (ctypes.c_int, [_vp, _vp, _vp, _i64, _vp]),
    "oilbird_merge_shards": (ctypes.c_int, [_i32, _i32, _i32, _i32, ctypes.c_float, _vp,
                                            ctypes.c_size_t, ctypes.c_size_t, ctypes.c_size_t,
                                            ctypes.c_size_t, ctypes.c_size_t, _vp, _vp, _vp, _vp,
                                            _vp, _i32, _vp]),
    "oilbird_merge_params_default": (None, [ctypes.POINTER(MergeParams)]),
    "oilbird_merge_chains": (ctypes.c_int, [_i32, _vp, _vp, _i32, _i32, _vp, _vp, _i32, _i32, _vp,
                                            _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                            ctypes.POINTER(MergeParams), _i32, _vp]),
    "oilbird_index_create": (ctypes.c_int, [ctypes.POINTER(_vp), _vp, _vp, _i32, _vp]),
    "oilbird_index_refresh": (ctypes.c_int, [_vp, _vp]),
    "oilbird_index_reset": (ctypes.c_int, [_vp, _vp]),
    "oilbird_index_train": (ctypes.c_int, [_vp, _i32, _vp]),
    "oilbird_index_read_centroids": (ctypes.c_int, [_vp, _vp]),
    "oilbird_index_query": (ctypes.c_int, [_vp, _vp, _i32, _i32, ctypes.POINTER(CQueryParams),
                                           ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_index_destroy": (ctypes.c_int, [_vp]),
    "oilbird_index_rows": (_i64, [_vp]),
    "oilbird_index_read": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "oilbird_index_last_error": (ctypes.c_char_p, []),
    "oilbird_query_static": (ctypes.c_int, [ctypes.POINTER(StaticPool), _vp, _i32,
                                            ctypes.POINTER(CQueryParams),
                                            ctypes.POINTER(CQueryOut), _vp]),
    "oilbird_query_static_error": (ctypes.c_char_p, []),
    "oilbird_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "oilbird_last_cuda_error": (ctypes.c_char_p, []),
}

_lib = None
# Pools made without an explicit debug_guards argument take this (the GPU tests switch it on).
DEFAULT_DEBUG_GUARDS = False
GUARD_FAILURES: list = []      # pools whose guard check failed inside __del__


def _torch_empty(shape, dtype, device):
    return torch.empty(shape, dtype=dtype, device=device)


# Every result tensor this module creates comes from ALLOC(shape, dtype, device); the GPU
# tests replace it with an allocator that surrounds each tensor with sentinel bytes.
ALLOC = _torch_empty


def lib() -> ctypes.CDLL:
    """Load liboilbird.so (built by ``paper_2608_03839_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_03839_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(L, name)          # AttributeError if a declared symbol is missing
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class OilbirdError(RuntimeError):
    def __init__(self, code: int, where: str):
        L = lib()
        msg = L.oilbird_strerror(code).decode()
        if code in (ECUDA, ENOMEM, EGUARD) or (code == EINVAL and any(
                w in L.oilbird_last_cuda_error().decode() for w in ("aligned", "in flight"))):
            msg += " (" + L.oilbird_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [{code}]")
        self.code = code


def _flags(new_trace: bool, evict_to_fit: bool) -> int:
    return (NEW_TRACE if new_trace else 0) | (EVICT_TO_FIT if evict_to_fit else 0)


def _check(code: int, where: str) -> None:
    if code != OK:
        raise OilbirdError(code, where)


@dataclass
class QueryParams:
    """Defaults are the deployed values of the paper (k=8, theta=0.8, offset 2, D(s))."""
    k: int = 8
    theta: float = 0.8
    offset: int = 2
    depth_mode: int = DEPTH_TIERED
    cont_len: int = 48
    tier_thr: tuple = (0.90, 0.82)
    tier_depth: tuple = (48, 8)
    exclude_tag: torch.Tensor | np.ndarray | None = None   # [nq] uint64 (device: int64 tensor)
    path: int = PATH_AUTO

    def to_c(self, exclude_ptr=None) -> CQueryParams:
        key = (self.k, self.theta, self.offset, self.depth_mode, self.cont_len,
               tuple(self.tier_thr), tuple(self.tier_depth), self.path)
        c = _PARAM_CACHE.get(key)
        if c is None:
            c = CQueryParams()
            c.k, c.theta, c.offset = int(self.k), float(self.theta), int(self.offset)
            c.depth_mode, c.cont_len = int(self.depth_mode), int(self.cont_len)
            if len(self.tier_thr) != len(self.tier_depth) or len(self.tier_thr) > MAX_TIERS:
                raise ValueError("tier_thr / tier_depth: same length, at most 4")
            c.n_tiers = len(self.tier_thr)
            for i, (t, dd) in enumerate(zip(self.tier_thr, self.tier_depth)):
                c.tier_thr[i], c.tier_depth[i] = float(t), int(dd)
            c.path = int(self.path)
            if len(_PARAM_CACHE) < 256:
                _PARAM_CACHE[key] = c
        c.exclude_tag = exclude_ptr
        return c


_PARAM_CACHE: dict = {}


@dataclass
class QueryOut:
    idx: torch.Tensor        # [nq,k] int32
    score: torch.Tensor      # [nq,k] float32
    fired: torch.Tensor      # [nq] int32
    cont_len: torch.Tensor   # [nq,k] int32
    cont_tok: torch.Tensor   # [nq,k,L] int32
    _c: CQueryOut = field(default=None, repr=False)

    @staticmethod
    def empty(nq: int, k: int, L: int, device) -> "QueryOut":
        o = QueryOut(ALLOC((nq, k), torch.int32, device),
                     ALLOC((nq, k), torch.float32, device),
                     ALLOC((nq,), torch.int32, device),
                     ALLOC((nq, k), torch.int32, device),
                     ALLOC((nq, k, L), torch.int32, device))
        o._c = CQueryOut(o.idx.data_ptr(), o.score.data_ptr(), o.fired.data_ptr(),
                         o.cont_len.data_ptr(), o.cont_tok.data_ptr())
        return o

    def cpu(self) -> "QueryOut":
        return QueryOut(self.idx.cpu(), self.score.cpu(), self.fired.cpu(), self.cont_len.cpu(),
                        self.cont_tok.cpu())


def query_static(keys: torch.Tensor, tokens: torch.Tensor, trace_id: torch.Tensor,
                 trace_end: torch.Tensor, q: torch.Tensor, params: QueryParams,
                 out: QueryOut | None = None, stream=None) -> QueryOut:
    """oilbird_query_static: query caller-held pool arrays without any allocation.

    For hosts that own all device memory themselves and cannot let the library allocate;
    the library's only scratch is a fixed 1 MiB array in its image, so nq <= 2, k <= 128,
    no exclusion tags.  keys: CUDA bf16 [n,d], already L2-normalised (as append stores
    them); tokens / trace_id: CUDA int32 [n]; trace_end: CUDA int32 [n_traces].  Pass
    `out` to keep this wrapper itself from allocating result tensors.
    """
    for t, dt in ((keys, torch.bfloat16), (tokens, torch.int32), (trace_id, torch.int32),
                  (trace_end, torch.int32), (q, torch.bfloat16)):
        assert t.is_cuda and t.dtype == dt and t.is_contiguous()
    n, d = keys.shape
    q = q.reshape(-1, d)
    nq = q.shape[0]
    if out is None:
        out = QueryOut.empty(nq, params.k, params.cont_len, keys.device)
    sp = StaticPool(keys.data_ptr(), tokens.data_ptr(), trace_id.data_ptr(), trace_end.data_ptr(),
                    n, d, keys.device.index or 0)
    cp = params.to_c(None)
    if params.exclude_tag is not None:
        cp.exclude_tag = params.exclude_tag.data_ptr()
    L = lib()
    rc = L.oilbird_query_static(ctypes.byref(sp), q.data_ptr(), nq, ctypes.byref(cp),
                                ctypes.byref(out._c), _stream_ptr(stream))
    if rc != OK:
        err = OilbirdError(rc, "oilbird_query_static")
        err.args = (err.args[0] + ": " + L.oilbird_query_static_error().decode(),)
        raise err
    return out


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class Pool:
    """A semantic draft pool on one GPU (one per tenant)."""

    def __init__(self, d: int, capacity_rows: int, *, max_traces: int = 0, max_nq: int = 0,
                 max_k: int = 0, max_append: int = 0, device: int = 0, use_torch_arena=False,
                 key_format: str = "bf16", debug_guards: bool | None = None):
        """key_format: "bf16" (the paper's store) or "e4m3" (8-bit keys, one scale per row).
        debug_guards: sentinel bytes behind every array of the pool (check_guards() verifies
        them); None takes the module default DEFAULT_DEBUG_GUARDS."""
        self._L = lib()
        if key_format not in ("bf16", "e4m3"):
            raise ValueError("key_format must be 'bf16' or 'e4m3'")
        self.key_format = key_format
        self.debug_guards = DEFAULT_DEBUG_GUARDS if debug_guards is None else bool(debug_guards)
        if not torch.cuda.is_available():
            raise RuntimeError("oilbird pool needs a CUDA device; there is no CPU fallback")
        self.d, self.device = int(d), int(device)
        cfg = PoolConfig(d=d, capacity_rows=capacity_rows, max_traces=max_traces, max_nq=max_nq,
                         max_k=max_k, max_append=max_append, device=device,
                         flags=(KEYS_E4M3 if key_format == "e4m3" else 0) |
                               (DEBUG_GUARDS if self.debug_guards else 0),
                         arena=None, arena_bytes=0)
        self._arena = None
        if use_torch_arena:
            nbytes = self._L.oilbird_pool_arena_bytes(ctypes.byref(cfg))
            if nbytes == 0:
                raise OilbirdError(EINVAL, "oilbird_pool_arena_bytes")
            self._arena = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{device}")
            cfg.arena, cfg.arena_bytes = self._arena.data_ptr(), nbytes
        h = ctypes.c_void_p()
        _check(self._L.oilbird_pool_create(ctypes.byref(h), ctypes.byref(cfg)),
               "oilbird_pool_create")
        self._h = h
        self._dev = torch.device(f"cuda:{device}")

    def close(self) -> None:
        h, self._h = getattr(self, "_h", None), None
        if h:
            rc = OK
            if self.debug_guards:
                rc = self._L.oilbird_pool_check_guards(h, _stream_ptr(None))
            self._L.oilbird_pool_destroy(h)
            _check(rc, "oilbird_pool_check_guards (at close)")

    def __del__(self):
        try:
            self.close()
        except Exception as e:           # (module globals may be gone at interpreter exit)
            if type(e).__name__ == "OilbirdError":
                import traceback
                traceback.print_exc()
                GUARD_FAILURES.append(self)

    def check_guards(self, stream=None) -> None:
        """Raises OilbirdError(EGUARD) if a kernel wrote behind one of the pool's arrays."""
        _check(self._L.oilbird_pool_check_guards(self._h, _stream_ptr(stream)),
               "oilbird_pool_check_guards")

    def set_wait_limit(self, limit_ns: int, stream=None) -> None:
        _check(self._L.oilbird_pool_set_wait_limit(self._h, int(limit_ns), _stream_ptr(stream)),
               "oilbird_pool_set_wait_limit")

    def stall_selftest(self, stream=None) -> None:
        _check(self._L.oilbird_pool_stall_selftest(self._h, _stream_ptr(stream)),
               "oilbird_pool_stall_selftest")

    def status(self, stream=None) -> int:
        """The code of oilbird_pool_status: OK, or ESTALL after a device-side wait gave up."""
        return int(self._L.oilbird_pool_status(self._h, None, _stream_ptr(stream)))

    def __len__(self) -> int:
        return int(self._L.oilbird_pool_size(self._h))

    @property
    def num_traces(self) -> int:
        return int(self._L.oilbird_pool_num_traces(self._h))

    @property
    def launch_count(self) -> int:
        return int(self._L.oilbird_pool_launch_count(self._h))

    def reset(self, stream=None) -> None:
        _check(self._L.oilbird_pool_reset(self._h, _stream_ptr(stream)), "oilbird_pool_reset")

    # ---- device-buffer entry points -------------------------------------------------
    def append(self, states: torch.Tensor, tokens: torch.Tensor, tag: int = 0,
               new_trace: bool = True, evict_to_fit: bool = False, stream=None) -> None:
        n = int(tokens.shape[0])
        if n:
            assert states.is_cuda and tokens.is_cuda and states.dtype == torch.bfloat16
            assert tokens.dtype == torch.int32 and states.is_contiguous() and tokens.is_contiguous()
            assert states.shape == (n, self.d)
        _check(self._L.oilbird_pool_append(self._h, states.data_ptr() if n else None,
                                           tokens.data_ptr() if n else None, n, int(tag),
                                           _flags(new_trace, evict_to_fit), _stream_ptr(stream)),
               "oilbird_pool_append")

    def append_global(self, states: torch.Tensor, tokens: torch.Tensor, global_row: int,
                      tag: int = 0, new_trace: bool = True, evict_to_fit: bool = False, stream=None) -> None:
        """append() for a pool that is one shard of a larger one: global_row is the position
        of the first appended row in the logical pool."""
        n = int(tokens.shape[0])
        assert states.is_cuda and tokens.is_cuda and states.dtype == torch.bfloat16
        assert tokens.dtype == torch.int32 and states.is_contiguous() and tokens.is_contiguous()
        _check(self._L.oilbird_pool_append_global(
            self._h, states.data_ptr(), tokens.data_ptr(), n, int(tag),
            _flags(new_trace, evict_to_fit), int(global_row), _stream_ptr(stream)),
            "oilbird_pool_append_global")

    def to_global(self, idx: torch.Tensor, out: torch.Tensor | None = None, stream=None
                  ) -> torch.Tensor:
        """Local rows (int32) -> global positions (int64); -1 stays -1."""
        assert idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous()
        if out is None:
            out = ALLOC(tuple(idx.shape), torch.int64, idx.device)
        _check(self._L.oilbird_pool_to_global(self._h, idx.data_ptr(), out.data_ptr(),
                                              idx.numel(), _stream_ptr(stream)),
               "oilbird_pool_to_global")
        return out

    def query(self, q: torch.Tensor, params: QueryParams | None = None,
              out: QueryOut | None = None, stream=None) -> QueryOut:
        pr = params or QueryParams()
        assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
        q = q.reshape(-1, self.d)
        nq = q.shape[0]
        ex_ptr = None
        if pr.exclude_tag is not None:
            ex = pr.exclude_tag
            assert ex.is_cuda and ex.dtype in (torch.int64, torch.uint64) and ex.numel() == nq
            ex_ptr = ex.data_ptr()
        if out is None:
            out = QueryOut.empty(nq, pr.k, pr.cont_len, self._dev)
        cp = pr.to_c(ex_ptr)
        _check(self._L.oilbird_pool_query(self._h, q.data_ptr(), nq, ctypes.byref(cp),
                                          ctypes.byref(out._c), _stream_ptr(stream)),
               "oilbird_pool_query")
        return out

    def evict_oldest(self, n_traces: int, stream=None) -> int:
        """Drop the n_traces oldest traces and compact; rows and traces are renumbered.
        Returns the number of rows dropped."""
        dropped = ctypes.c_int64(0)
        _check(self._L.oilbird_pool_evict_oldest(self._h, int(n_traces), ctypes.byref(dropped),
                                                 _stream_ptr(stream)), "oilbird_pool_evict_oldest")
        return int(dropped.value)

    def step(self, states: torch.Tensor, tokens: torch.Tensor, q: torch.Tensor,
             params: QueryParams | None = None, out: QueryOut | None = None, tag: int = 0,
             new_trace: bool = True, evict_to_fit: bool = False, stream=None) -> QueryOut:
        """One serving step on device tensors: append(states, tokens) then query(q), in one
        call (same results as the two calls; the single-request scan overlaps the append)."""
        pr = params or QueryParams()
        assert states.is_cuda and states.dtype == torch.bfloat16 and states.is_contiguous()
        assert tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous()
        assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
        n = int(tokens.shape[0])
        assert states.numel() == n * self.d
        q = q.reshape(-1, self.d)
        nq = q.shape[0]
        ex_ptr = None
        if pr.exclude_tag is not None:
            ex = pr.exclude_tag
            assert ex.is_cuda and ex.dtype in (torch.int64, torch.uint64) and ex.numel() == nq
            ex_ptr = ex.data_ptr()
        if out is None:
            out = QueryOut.empty(nq, pr.k, pr.cont_len, self._dev)
        cp = pr.to_c(ex_ptr)
        _check(self._L.oilbird_pool_step(
            self._h, states.data_ptr(), tokens.data_ptr(), n, int(tag),
            _flags(new_trace, evict_to_fit), q.data_ptr(), nq, ctypes.byref(cp),
            ctypes.byref(out._c), _stream_ptr(stream)), "oilbird_pool_step")
        return out

    def gather(self, idx: torch.Tensor, score: torch.Tensor, params: QueryParams,
               stream=None) -> QueryOut:
        assert idx.is_cuda and idx.dtype == torch.int32 and score.dtype == torch.float32
        nq = idx.shape[0]
        out = QueryOut.empty(nq, params.k, params.cont_len, self._dev)
        out.idx, out.score = idx, score
        cp = params.to_c(None)
        co = CQueryOut(None, None, out.fired.data_ptr(), out.cont_len.data_ptr(),
                       out.cont_tok.data_ptr())
        _check(self._L.oilbird_pool_gather(self._h, idx.data_ptr(), score.data_ptr(), nq,
                                           ctypes.byref(cp), ctypes.byref(co),
                                           _stream_ptr(stream)), "oilbird_pool_gather")
        return out

    # ---- host-buffer entry points ---------------------------------------------------
    def append_host(self, states: torch.Tensor, tokens: torch.Tensor, tag: int = 0,
                    new_trace: bool = True, evict_to_fit: bool = False, stream=None) -> None:
        """states: CPU bf16 tensor [n,d] (ideally pinned); tokens: CPU int32 [n]."""
        n = int(tokens.shape[0])
        assert not states.is_cuda and not tokens.is_cuda and states.is_contiguous()
        _check(self._L.oilbird_pool_append_host(self._h, states.data_ptr(), tokens.data_ptr(), n,
                                                int(tag), _flags(new_trace, evict_to_fit),
                                                _stream_ptr(stream)), "oilbird_pool_append_host")

    def query_host(self, q: torch.Tensor, params: QueryParams | None = None,
                   out: QueryOut | None = None, stream=None) -> QueryOut:
        """q: CPU bf16 tensor [nq,d]; results land in CPU tensors."""
        pr = params or QueryParams()
        assert not q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
        q = q.reshape(-1, self.d)
        nq = q.shape[0]
        ex_ptr = None
        if pr.exclude_tag is not None:
            ex = pr.exclude_tag
            assert not ex.is_cuda and ex.numel() == nq
            ex_ptr = ex.data_ptr()
        if out is None:
            out = QueryOut.empty(nq, pr.k, pr.cont_len, "cpu")
        cp = pr.to_c(ex_ptr)
        _check(self._L.oilbird_pool_query_host(self._h, q.data_ptr(), nq, ctypes.byref(cp),
                                               ctypes.byref(out._c), _stream_ptr(stream)),
               "oilbird_pool_query_host")
        return out

    def step_host(self, states: torch.Tensor, tokens: torch.Tensor, q: torch.Tensor,
                  params: QueryParams, out: QueryOut, tag: int = 0, new_trace: bool = True, evict_to_fit: bool = False,
                  stream=None) -> QueryOut:
        """One serving step from host memory: append the committed rows, then query.
        All tensors are CPU tensors; `out` must have been made with QueryOut.empty(..., "cpu")."""
        cp = params.to_c(None)
        _check(self._L.oilbird_pool_step_host(
            self._h, states.data_ptr(), tokens.data_ptr(), int(tokens.shape[0]), int(tag),
            _flags(new_trace, evict_to_fit), q.data_ptr(), int(q.shape[0]), ctypes.byref(cp),
            ctypes.byref(out._c), _stream_ptr(stream)), "oilbird_pool_step_host")
        return out

    def step_host_begin(self, states: torch.Tensor, tokens: torch.Tensor, q: torch.Tensor,
                        params: QueryParams, slot: int, tag: int = 0, new_trace: bool = True, evict_to_fit: bool = False,
                        stream=None) -> None:
        """First half of step_host: returns once the step is enqueued (slot 0 or 1)."""
        ex_ptr = params.exclude_tag.data_ptr() if params.exclude_tag is not None else None
        cp = params.to_c(ex_ptr)
        _check(self._L.oilbird_pool_step_host_begin(
            self._h, states.data_ptr(), tokens.data_ptr(), int(tokens.shape[0]), int(tag),
            _flags(new_trace, evict_to_fit), q.data_ptr(), int(q.shape[0]), ctypes.byref(cp),
            int(slot), _stream_ptr(stream)), "oilbird_pool_step_host_begin")

    def step_host_end(self, slot: int, out: QueryOut) -> QueryOut:
        """Second half: waits for that slot's step, fills the CPU tensors of `out`."""
        _check(self._L.oilbird_pool_step_host_end(self._h, int(slot), ctypes.byref(out._c)),
               "oilbird_pool_step_host_end")
        return out

    # ---- introspection --------------------------------------------------------------
    def stats(self, stream=None) -> dict:
        s = PoolStats()
        rc = self._L.oilbird_pool_status(self._h, ctypes.byref(s), _stream_ptr(stream))
        if rc not in (OK, ESTALL):
            _check(rc, "oilbird_pool_status")
        return dict(degenerate_rows=int(s.degenerate_rows),
                    nonfinite_queries=int(s.nonfinite_queries), stalled=int(s.stalled))

    def read_rows(self, row0: int = 0, n: int | None = None):
        """(keys uint16 [n,d], tokens int32 [n], trace_ids int32 [n]) as numpy arrays."""
        n = len(self) - row0 if n is None else n
        keys = np.empty((n, self.d), dtype=np.uint16) if self.key_format == "bf16" else None
        tok = np.empty(n, dtype=np.int32)
        tid = np.empty(n, dtype=np.int32)
        _check(self._L.oilbird_pool_read_rows(self._h, row0, n,
                                              keys.ctypes.data if keys is not None else None,
                                              tok.ctypes.data, tid.ctypes.data),
               "oilbird_pool_read_rows")
        return keys, tok, tid

    def read_codes(self, row0: int = 0, n: int | None = None):
        """8-bit pools: (codes uint8 [n,d], scales float32 [n]) as numpy arrays."""
        n = len(self) - row0 if n is None else n
        codes = np.empty((n, self.d), dtype=np.uint8)
        scales = np.empty(n, dtype=np.float32)
        _check(self._L.oilbird_pool_read_codes(self._h, row0, n, codes.ctypes.data,
                                               scales.ctypes.data), "oilbird_pool_read_codes")
        return codes, scales

    def traces(self):
        """(start int64 [T], end int64 [T], tag uint64 [T]) as the host tracks them."""
        T = self.num_traces
        st, en, tg = (np.empty(T, np.int64), np.empty(T, np.int64), np.empty(T, np.uint64))
        self._L.oilbird_pool_read_traces(self._h, st.ctypes.data, en.ctypes.data, tg.ctypes.data, T)
        return st, en, tg

    def profile(self, enable: bool) -> None:
        _check(self._L.oilbird_pool_profile(self._h, int(enable)), "oilbird_pool_profile")

    def profile_read(self, max_n: int = 4096) -> np.ndarray:
        buf = np.empty(max_n, dtype=np.float32)
        n = self._L.oilbird_pool_profile_read(self._h, buf.ctypes.data, max_n)
        return buf[:n].copy()


# ------------------------------------------------------------------ coarse index ----
class Index:
    """Inverted-file index over a Pool (oilbird_index_* of the C-ABI): centroids the caller
    supplies, rows assigned by the library's own k = 1 lookup, queries answered from the
    n_probe best lists plus the rows appended since the last refresh."""

    def __init__(self, pool: Pool, centroids: torch.Tensor, stream=None):
        assert centroids.is_cuda and centroids.dtype == torch.bfloat16 and centroids.is_contiguous()
        assert centroids.dim() == 2 and centroids.shape[1] == pool.d
        self._L, self.pool, self.n_lists = lib(), pool, int(centroids.shape[0])
        h = ctypes.c_void_p()
        _check(self._L.oilbird_index_create(ctypes.byref(h), pool._h, centroids.data_ptr(),
                                            self.n_lists, _stream_ptr(stream)), "oilbird_index_create")
        self._h = h

    def close(self) -> None:
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._L.oilbird_index_destroy(h)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __len__(self) -> int:
        return int(self._L.oilbird_index_rows(self._h))

    def refresh(self, stream=None) -> None:
        _check(self._L.oilbird_index_refresh(self._h, _stream_ptr(stream)), "oilbird_index_refresh")

    def reset(self, stream=None) -> None:
        _check(self._L.oilbird_index_reset(self._h, _stream_ptr(stream)), "oilbird_index_reset")

    def train(self, iterations: int, stream=None) -> None:
        """Lloyd's iterations on the pool's rows; the lists are rebuilt afterwards."""
        _check(self._L.oilbird_index_train(self._h, int(iterations), _stream_ptr(stream)),
               "oilbird_index_train")

    def centroids(self) -> np.ndarray:
        """The raw centroid states, [n_lists, d] bf16 bit patterns (uint16)."""
        out = np.empty((self.n_lists, self.pool.d), dtype=np.uint16)
        _check(self._L.oilbird_index_read_centroids(self._h, out.ctypes.data),
               "oilbird_index_read_centroids")
        return out

    def query(self, q: torch.Tensor, n_probe: int, params: QueryParams | None = None,
              out: QueryOut | None = None, stream=None) -> QueryOut:
        pr = params or QueryParams()
        assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
        q = q.reshape(-1, self.pool.d)
        nq = q.shape[0]
        ex_ptr = None
        if pr.exclude_tag is not None:
            ex = pr.exclude_tag
            assert ex.is_cuda and ex.dtype in (torch.int64, torch.uint64) and ex.numel() == nq
            ex_ptr = ex.data_ptr()
        if out is None:
            out = QueryOut.empty(nq, pr.k, pr.cont_len, self.pool._dev)
        cp = pr.to_c(ex_ptr)
        _check(self._L.oilbird_index_query(self._h, q.data_ptr(), nq, int(n_probe), ctypes.byref(cp),
                                           ctypes.byref(out._c), _stream_ptr(stream)),
               "oilbird_index_query")
        return out

    def read(self):
        """(assign int32 [rows], list_off int32 [n_lists+1], list_rows int32 [rows])."""
        n = len(self)
        a, o, r = np.empty(n, np.int32), np.empty(self.n_lists + 1, np.int32), np.empty(n, np.int32)
        _check(self._L.oilbird_index_read(self._h, a.ctypes.data, o.ctypes.data, r.ctypes.data),
               "oilbird_index_read")
        return a, o, r


# ------------------------------------------------------------------ recycled pool ----
RING_MAX_M, RING_MAX_ROLLOUT, RING_MAX_NQ = 32, 16, 64


@dataclass
class RingOut:
    slot: torch.Tensor         # [nq,m] int32, -1 padded
    score: torch.Tensor        # [nq,m] float32, -inf padded
    count: torch.Tensor        # [nq] int32
    rollout: torch.Tensor      # [nq,m,R] int32, -1 padded
    rollout_len: torch.Tensor  # [nq,m] int32

    def cpu(self) -> "RingOut":
        return RingOut(self.slot.cpu(), self.score.cpu(), self.count.cpu(), self.rollout.cpu(),
                       self.rollout_len.cpu())


class Ring:
    """Rejected-branch ring buffer on one GPU (oilbird_ring_* of the C-ABI)."""

    def __init__(self, d: int, capacity: int, max_rollout: int = 6, device: int = 0):
        self._L = lib()
        if not torch.cuda.is_available():
            raise RuntimeError("oilbird ring needs a CUDA device; there is no CPU fallback")
        self.d, self.capacity, self.max_rollout = int(d), int(capacity), int(max_rollout)
        cfg = RingConfig(d=d, capacity=capacity, max_rollout=max_rollout, device=device)
        h = ctypes.c_void_p()
        _check(self._L.oilbird_ring_create(ctypes.byref(h), ctypes.byref(cfg)),
               "oilbird_ring_create")
        self._h = h
        self._dev = torch.device(f"cuda:{device}")

    def close(self) -> None:
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._L.oilbird_ring_destroy(h)

    __del__ = close

    def __len__(self) -> int:
        return int(self._L.oilbird_ring_size(self._h))

    @property
    def total(self) -> int:
        return int(self._L.oilbird_ring_total(self._h))

    def reset(self, stream=None) -> None:
        _check(self._L.oilbird_ring_reset(self._h, _stream_ptr(stream)), "oilbird_ring_reset")

    def append(self, states: torch.Tensor, anchors: torch.Tensor, rollouts: torch.Tensor,
               stream=None) -> None:
        n = int(anchors.shape[0])
        assert states.is_cuda and states.dtype == torch.bfloat16 and states.is_contiguous()
        assert anchors.is_cuda and anchors.dtype == torch.int32 and anchors.is_contiguous()
        assert rollouts.is_cuda and rollouts.dtype == torch.int32 and rollouts.is_contiguous()
        assert states.shape == (n, self.d) and rollouts.shape == (n, self.max_rollout)
        _check(self._L.oilbird_ring_append(self._h, states.data_ptr(), anchors.data_ptr(),
                                           rollouts.data_ptr(), n, _stream_ptr(stream)),
               "oilbird_ring_append")

    def query(self, q: torch.Tensor, anchors: torch.Tensor, m: int = 4, floor: float = 0.8,
              out: RingOut | None = None, stream=None) -> RingOut:
        assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
        q = q.reshape(-1, self.d)
        nq = q.shape[0]
        assert anchors.is_cuda and anchors.dtype == torch.int32 and anchors.numel() == nq
        if out is None:
            out = RingOut(ALLOC((nq, m), torch.int32, self._dev),
                          ALLOC((nq, m), torch.float32, self._dev),
                          ALLOC((nq,), torch.int32, self._dev),
                          ALLOC((nq, m, self.max_rollout), torch.int32, self._dev),
                          ALLOC((nq, m), torch.int32, self._dev))
        co = CRingOut(out.slot.data_ptr(), out.score.data_ptr(), out.count.data_ptr(),
                      out.rollout.data_ptr(), out.rollout_len.data_ptr())
        _check(self._L.oilbird_ring_query(self._h, q.data_ptr(), anchors.data_ptr(), nq, int(m),
                                          float(floor), ctypes.byref(co), _stream_ptr(stream)),
               "oilbird_ring_query")
        return out

    def step(self, states: torch.Tensor, anchors: torch.Tensor, rollouts: torch.Tensor,
             q: torch.Tensor, q_anchors: torch.Tensor, m: int = 4, floor: float = 0.8,
             out: RingOut | None = None, stream=None) -> RingOut:
        """One verification pass: append the records, then look up, in one call."""
        n = int(anchors.shape[0])
        assert states.is_cuda and states.dtype == torch.bfloat16 and states.is_contiguous()
        assert anchors.is_cuda and anchors.dtype == torch.int32 and anchors.is_contiguous()
        assert rollouts.is_cuda and rollouts.dtype == torch.int32 and rollouts.is_contiguous()
        assert states.shape == (n, self.d) and rollouts.shape == (n, self.max_rollout)
        assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
        q = q.reshape(-1, self.d)
        nq = q.shape[0]
        assert q_anchors.is_cuda and q_anchors.dtype == torch.int32 and q_anchors.numel() == nq
        if out is None:
            out = RingOut(ALLOC((nq, m), torch.int32, self._dev),
                          ALLOC((nq, m), torch.float32, self._dev),
                          ALLOC((nq,), torch.int32, self._dev),
                          ALLOC((nq, m, self.max_rollout), torch.int32, self._dev),
                          ALLOC((nq, m), torch.int32, self._dev))
        co = CRingOut(out.slot.data_ptr(), out.score.data_ptr(), out.count.data_ptr(),
                      out.rollout.data_ptr(), out.rollout_len.data_ptr())
        _check(self._L.oilbird_ring_step(self._h, states.data_ptr(), anchors.data_ptr(),
                                         rollouts.data_ptr(), n, q.data_ptr(), q_anchors.data_ptr(),
                                         nq, int(m), float(floor), ctypes.byref(co),
                                         _stream_ptr(stream)), "oilbird_ring_step")
        return out

    def read(self):
        """(keys uint16 [cap,d], anchors int32 [cap], rollouts int32 [cap,R]) as numpy arrays."""
        keys = np.empty((self.capacity, self.d), np.uint16)
        anc = np.empty(self.capacity, np.int32)
        roll = np.empty((self.capacity, self.max_rollout), np.int32)
        _check(self._L.oilbird_ring_read(self._h, keys.ctypes.data, anc.ctypes.data,
                                         roll.ctypes.data), "oilbird_ring_read")
        return keys, anc, roll


# ------------------------------------------------------------------ tree merge ----
TREE_MAX_NODES = 64
CHAIN_SHORT, CHAIN_DUPLICATE, CHAIN_MERGED, CHAIN_CUT, CHAIN_NOT_REACHED = range(5)


@dataclass
class MergeOut:
    tree_tok: torch.Tensor      # [nq,max_nodes] int32 (updated in place)
    tree_parent: torch.Tensor   # [nq,max_nodes] int32
    n_nodes: torch.Tensor       # [nq] int32
    depth: torch.Tensor         # [nq,max_nodes] int32
    mask: torch.Tensor          # [nq,max_nodes] int64 (bit j: node j is self or an ancestor)
    status: torch.Tensor        # [nq,k+ne] int32
    bought: torch.Tensor        # [nq,k+ne] int32
    walked: torch.Tensor        # [nq,k+ne] int32


def merge_chains(tree_tok: torch.Tensor, tree_parent: torch.Tensor, n_nodes: torch.Tensor,
                 sem_tok: torch.Tensor | None, sem_len: torch.Tensor | None,
                 extra_tok: torch.Tensor | None = None, extra_len: torch.Tensor | None = None,
                 budget: int = 16, min_len: int = 2, root_attached: bool = False,
                 stream=None, out: "MergeOut | None" = None) -> MergeOut:
    """oilbird_merge_chains: post-filter the chains and merge them into each request's tree.

    tree_tok / tree_parent: CUDA int32 [nq,max_nodes] (updated in place), n_nodes: [nq].
    sem_tok [nq,k,L] / sem_len [nq,k]: a query's cont_tok / cont_len.  extra_*: further chains.
    """
    nq, max_nodes = tree_tok.shape
    dev = tree_tok.device
    k, L = (sem_tok.shape[1], sem_tok.shape[2]) if sem_tok is not None else (0, 1)
    ne, Le = (extra_tok.shape[1], extra_tok.shape[2]) if extra_tok is not None else (0, 1)
    for t in (tree_tok, tree_parent, n_nodes, sem_tok, sem_len, extra_tok, extra_len):
        assert t is None or (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous())
    if out is not None:                      # result arrays of an earlier call, written again
        depth, mask, status, bought, walked = out.depth, out.mask, out.status, out.bought, out.walked
        assert depth.shape == (nq, max_nodes) and status.shape == (nq, k + ne)
    else:
        depth = ALLOC((nq, max_nodes), torch.int32, dev)
        mask = ALLOC((nq, max_nodes), torch.int64, dev)
        status = ALLOC((nq, k + ne), torch.int32, dev)
        bought = ALLOC((nq, k + ne), torch.int32, dev)
        walked = ALLOC((nq, k + ne), torch.int32, dev)
    mp = MergeParams(budget, max_nodes, min_len, int(bool(root_attached)))
    ptr = lambda t: None if t is None else t.data_ptr()
    _check(lib().oilbird_merge_chains(nq, ptr(sem_tok), ptr(sem_len), k, L, ptr(extra_tok),
                                      ptr(extra_len), ne, Le, tree_tok.data_ptr(),
                                      tree_parent.data_ptr(), n_nodes.data_ptr(), depth.data_ptr(),
                                      mask.data_ptr(), status.data_ptr(), bought.data_ptr(),
                                      walked.data_ptr(), ctypes.byref(mp), dev.index or 0,
                                      _stream_ptr(stream)), "oilbird_merge_chains")
    return MergeOut(tree_tok, tree_parent, n_nodes, depth, mask, status, bought, walked)
