"""ctypes binding of libdynakv.so: argument marshalling only, same names as the C ABI."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# DYNAKV_LIBRARY=checked selects the bounds-checked build of the same sources (libdynakv_checked.so), for test runs
_LIB_PATH = os.path.join(_HERE, "libdynakv_checked.so" if os.environ.get("DYNAKV_LIBRARY") == "checked" else "libdynakv.so")

F32, BF16, FP8 = 0, 1, 2
INIT_KMEANSPP, INIT_RANDOM = 0, 1
MODE_ADAPTIVE, MODE_STATIC, MODE_LOCAL, MODE_DELAYED = 0, 1, 2, 3
ST_BUDGET_EXCEEDED, ST_MAX_CLUSTERS, ST_MAX_TOKENS, ST_PAGE_POOL, ST_INTERNAL, ST_TIER_CACHE, ST_BOUNDS = 1, 2, 4, 8, 16, 32, 64

EXPORTED_SYMBOLS = [
    "dynakv_create", "dynakv_build_index", "dynakv_append", "dynakv_decode_step", "dynakv_split_check",
    "dynakv_decode_loop", "dynakv_step_host", "dynakv_get_status", "dynakv_export_state", "dynakv_get_selection",
    "dynakv_get_build_trace", "dynakv_set_timing", "dynakv_get_kernel_times", "dynakv_launch_count", "dynakv_last_error", "dynakv_destroy",
    "dynakv_attend_rows_noalloc", "dynakv_export_kv", "dynakv_import_state", "dynakv_decode_loop_host", "dynakv_selftest_wait_expiry", "dynakv_time_gather_attention",
    "dynakv_build_index_placed", "dynakv_get_work_list", "dynakv_work_list_capacity", "dynakv_get_tier_stats", "dynakv_checked_build",
]
ERR_TOO_LARGE = -5
NOALLOC_SCRATCH_BYTES = 4 * 1024 * 1024


class DynaKVError(RuntimeError):
    pass


class _Config(C.Structure):
    _fields_ = [("n_units", C.c_int32), ("gqa_group", C.c_int32), ("head_dim", C.c_int32), ("kv_dtype", C.c_int32),
                ("max_tokens", C.c_int32), ("max_clusters", C.c_int32), ("kmeans_iters", C.c_int32),
                ("init_mode", C.c_int32), ("split_size_factor", C.c_float), ("split_var_factor", C.c_float),
                ("split_min_size", C.c_int32), ("split_iters", C.c_int32), ("trace", C.c_int32),
                ("assign_mode", C.c_int32), ("attn_mode", C.c_int32), ("update_mode", C.c_int32), ("local_max", C.c_int32), ("det_sums", C.c_int32), ("buf_max", C.c_int32),
                ("tier", C.c_int32), ("cache_pages", C.c_int32)]


class _Status(C.Structure):
    _fields_ = [("error_bits", C.c_uint32), ("bounds_site", C.c_int32), ("n_appended", C.c_int64),
                ("n_splits", C.c_int64), ("tokens_selected", C.c_int64), ("clusters_selected", C.c_int64),
                ("pages_in_use", C.c_int64), ("assign_rechecked", C.c_int64), ("tokens_attended_total", C.c_int64),
                ("clusters_selected_total", C.c_int64)]

class _TierStats(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("pages_fetched", "clusters_hit", "clusters_fetched", "clusters_refreshed",
                                         "clusters_evicted", "copies_dropped_stale", "frames_in_use", "frames_total",
                                         "rows_fetched")]


KERNEL_CLASSES = ["init", "assign", "update", "finalize", "select", "attn", "combine", "append", "split", "front", "tier"]


@dataclass
class DynaKVConfig:
    n_units: int
    gqa_group: int
    head_dim: int
    kv_dtype: int
    max_tokens: int
    max_clusters: int
    kmeans_iters: int = 10
    init_mode: int = INIT_KMEANSPP
    split_size_factor: float = 2.0
    split_var_factor: float = 2.0
    split_min_size: int = 8
    split_iters: int = 8
    trace: int = 0
    assign_mode: int = 0
    attn_mode: int = 0
    update_mode: int = 0
    local_max: int = 64
    det_sums: int = 0
    buf_max: int = 64
    tier: int = 0
    cache_pages: int = 0


_lib = None


def load_library() -> C.CDLL:
    """Load libdynakv.so from the package directory; raise if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise DynaKVError(f"{_LIB_PATH} is missing: build it with `python -m paper_2511_07427_b200.build` "
                          "(there is no CPU fallback)")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    L.dynakv_create.restype = C.c_int
    L.dynakv_create.argtypes = [C.POINTER(_Config), vp, C.POINTER(vp)]
    L.dynakv_build_index.restype = C.c_int
    L.dynakv_build_index.argtypes = [vp, vp, vp, i64, i32, i32, u64]
    L.dynakv_build_index_placed.restype = C.c_int
    L.dynakv_build_index_placed.argtypes = [vp, vp, vp, i64, i32, i32, u64, vp, i64, i32]
    L.dynakv_get_work_list.restype = C.c_int
    L.dynakv_get_work_list.argtypes = [vp, vp, vp, i64]
    L.dynakv_work_list_capacity.restype = C.c_int
    L.dynakv_work_list_capacity.argtypes = [vp]
    L.dynakv_checked_build.restype = C.c_int
    L.dynakv_checked_build.argtypes = []
    L.dynakv_get_tier_stats.restype = C.c_int
    L.dynakv_get_tier_stats.argtypes = [vp, C.POINTER(_TierStats)]
    L.dynakv_append.restype = C.c_int
    L.dynakv_append.argtypes = [vp, vp, vp]
    L.dynakv_decode_step.restype = C.c_int
    L.dynakv_decode_step.argtypes = [vp, vp, i32, vp, vp]
    L.dynakv_split_check.restype = C.c_int
    L.dynakv_split_check.argtypes = [vp]
    L.dynakv_decode_loop.restype = C.c_int
    L.dynakv_decode_loop.argtypes = [vp, vp, vp, vp, i64, i32, vp]
    L.dynakv_step_host.restype = C.c_int
    L.dynakv_step_host.argtypes = [vp, vp, vp, vp, i32, vp]
    L.dynakv_get_status.restype = C.c_int
    L.dynakv_get_status.argtypes = [vp, C.POINTER(_Status)]
    L.dynakv_export_state.restype = C.c_int
    L.dynakv_export_state.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.dynakv_get_selection.restype = C.c_int
    L.dynakv_get_selection.argtypes = [vp, vp, vp]
    L.dynakv_decode_loop_host.restype = C.c_int
    L.dynakv_decode_loop_host.argtypes = [vp, vp, vp, vp, i64, i32, vp]
    L.dynakv_time_gather_attention.restype = C.c_int
    L.dynakv_time_gather_attention.argtypes = [vp, vp, vp, i32, vp]
    L.dynakv_selftest_wait_expiry.restype = C.c_int
    L.dynakv_selftest_wait_expiry.argtypes = [vp, vp]
    L.dynakv_export_kv.restype = C.c_int
    L.dynakv_export_kv.argtypes = [vp, vp, vp, i64]
    L.dynakv_import_state.restype = C.c_int
    L.dynakv_import_state.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32]
    L.dynakv_get_build_trace.restype = C.c_int
    L.dynakv_get_build_trace.argtypes = [vp, vp, vp]
    L.dynakv_set_timing.restype = C.c_int
    L.dynakv_set_timing.argtypes = [vp, i32]
    L.dynakv_get_kernel_times.restype = C.c_int
    L.dynakv_get_kernel_times.argtypes = [vp, vp, vp, i32]
    L.dynakv_launch_count.restype = C.c_int64
    L.dynakv_launch_count.argtypes = [vp]
    L.dynakv_last_error.restype = C.c_char_p
    L.dynakv_last_error.argtypes = []
    L.dynakv_destroy.restype = None
    L.dynakv_destroy.argtypes = [vp]
    L.dynakv_attend_rows_noalloc.restype = C.c_int
    L.dynakv_attend_rows_noalloc.argtypes = [vp, vp, vp, i32, i64, i32, i32, i32, vp, vp]
    _lib = L
    return L


def _np_ptr(a: Optional[np.ndarray]):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def attend_rows_noalloc(q, K, V, out=None, stream=None):
    """Softmax attention of q [U, G, d] (fp32) over all rows of K, V [U, n, d] (fp32 or bf16) through
    ``dynakv_attend_rows_noalloc``: the entry point for callers that must not allocate device memory
    (its split-K scratch is a fixed array inside the library).  ``out`` [U, G, d] fp32 should be passed
    by such callers; it is only created here as a convenience when omitted.  Calls share the library's
    scratch array, so keep them on one stream.  Raises DynaKVError with the size limit when the call
    needs more scratch than the library holds."""
    import torch
    L = load_library()
    if not (q.is_cuda and K.is_cuda and V.is_cuda):
        raise DynaKVError("attend_rows_noalloc takes CUDA tensors")
    U, G, d = q.shape
    n = K.shape[1]
    if K.dtype not in (torch.float32, torch.bfloat16) or V.dtype != K.dtype or q.dtype != torch.float32 or \
            tuple(K.shape) != (U, n, d) or tuple(V.shape) != (U, n, d) or \
            not (q.is_contiguous() and K.is_contiguous() and V.is_contiguous()):
        raise DynaKVError("expected contiguous q [U,G,d] fp32 and K, V [U,n,d] of one dtype (fp32 or bf16)")
    if out is None:
        out = torch.empty((U, G, d), dtype=torch.float32, device=q.device)
    elif out.dtype != torch.float32 or tuple(out.shape) != (U, G, d) or not out.is_contiguous() or not out.is_cuda:
        raise DynaKVError("expected contiguous CUDA out [U,G,d] fp32")
    st = stream if stream is not None else torch.cuda.current_stream()
    rc = L.dynakv_attend_rows_noalloc(C.c_void_p(q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                      U, n, G, d, F32 if K.dtype == torch.float32 else BF16,
                                      C.c_void_p(out.data_ptr()), C.c_void_p(st.cuda_stream))
    if rc == ERR_TOO_LARGE:
        raise DynaKVError(f"dynakv_attend_rows_noalloc: {U} units x 16 splits x {G} heads x ({d}+2) floats exceed the "
                          f"library's fixed scratch of {NOALLOC_SCRATCH_BYTES} bytes; pass fewer units per call")
    if rc != 0:
        raise DynaKVError(f"dynakv_attend_rows_noalloc returned {rc}")
    return out


class DynaKV:
    """One context: U independent KV heads with their cluster index and paged KV store in HBM.

    Methods mirror the C entry points (``build_index``, ``append``, ``decode_step``,
    ``split_check``, ``decode_loop``, ``step_host``) and take ``torch`` CUDA tensors (or
    pinned host tensors for ``step_host``).  Work is enqueued on the stream that was current
    when the context was created."""

    def __init__(self, cfg: DynaKVConfig, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise DynaKVError("no CUDA device: libdynakv has no CPU fallback")
        self._L = load_library()
        self.cfg = cfg
        self._torch = torch
        self._stream = stream if stream is not None else torch.cuda.current_stream()
        c = _Config(cfg.n_units, cfg.gqa_group, cfg.head_dim, cfg.kv_dtype, cfg.max_tokens, cfg.max_clusters,
                    cfg.kmeans_iters, cfg.init_mode, cfg.split_size_factor, cfg.split_var_factor,
                    cfg.split_min_size, cfg.split_iters, cfg.trace, cfg.assign_mode, cfg.attn_mode, cfg.update_mode, cfg.local_max, cfg.det_sums, cfg.buf_max,
                    cfg.tier, cfg.cache_pages)
        h = C.c_void_p()
        self._check(self._L.dynakv_create(C.byref(c), C.c_void_p(self._stream.cuda_stream), C.byref(h)), "dynakv_create")
        self._h = h
        self.n_prefill = 0
        self.n_clusters0 = 0
        self._keep = []

    # ---- helpers
    def _check(self, rc: int, what: str) -> None:
        if rc != 0:
            msg = self._L.dynakv_last_error().decode()
            raise DynaKVError(f"{what} returned {rc} {msg}")

    def _kv(self, t, shape):
        torch = self._torch
        want = torch.float32 if self.cfg.kv_dtype == F32 else torch.bfloat16
        if t.dtype != want or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
            raise DynaKVError(f"expected contiguous {want} tensor of shape {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")
        return C.c_void_p(t.data_ptr())

    def _f32(self, t, shape):
        torch = self._torch
        if t.dtype != torch.float32 or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
            raise DynaKVError(f"expected contiguous float32 tensor of shape {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")
        return C.c_void_p(t.data_ptr())

    # ---- the C ABI, one method per entry point
    def build_index(self, K, V, n_clusters: int, seed: int, placement_queries=None, placement_budget: int = 0) -> None:
        """placement_queries ([n_ref, U, G, d] fp32 on the device) selects the build with correlation-aware placement:
        the clusters' pages are ordered by how often the reference queries retrieve clusters together."""
        U, d = self.cfg.n_units, self.cfg.head_dim
        n = K.shape[1]
        assert K.is_cuda and V.is_cuda
        if placement_queries is None:
            self._check(self._L.dynakv_build_index(self._h, self._kv(K, (U, n, d)), self._kv(V, (U, n, d)), n, d,
                                                   n_clusters, seed), "dynakv_build_index")
        else:
            qr = placement_queries
            self._check(self._L.dynakv_build_index_placed(
                self._h, self._kv(K, (U, n, d)), self._kv(V, (U, n, d)), n, d, n_clusters, seed,
                self._f32(qr, (qr.shape[0], U, self.cfg.gqa_group, d)), qr.shape[0], placement_budget), "dynakv_build_index_placed")
        self.n_prefill, self.n_clusters0 = n, n_clusters

    def append(self, k, v) -> None:
        U, d = self.cfg.n_units, self.cfg.head_dim
        assert k.is_cuda and v.is_cuda
        self._check(self._L.dynakv_append(self._h, self._kv(k, (U, d)), self._kv(v, (U, d))), "dynakv_append")

    def decode_step(self, q, token_budget: int, out=None, selected_ids=None):
        torch = self._torch
        U, G, d = self.cfg.n_units, self.cfg.gqa_group, self.cfg.head_dim
        assert q.is_cuda
        if out is None:
            out = torch.empty((U, G, d), dtype=torch.float32, device=q.device)
        sp = None
        if selected_ids is not None:
            assert selected_ids.dtype == torch.int32 and selected_ids.is_contiguous() and \
                tuple(selected_ids.shape) == (U, self.cfg.max_clusters)
            sp = C.c_void_p(selected_ids.data_ptr())
        self._check(self._L.dynakv_decode_step(self._h, self._f32(q, (U, G, d)), token_budget,
                                               self._f32(out, (U, G, d)), sp), "dynakv_decode_step")
        return out

    def split_check(self) -> None:
        self._check(self._L.dynakv_split_check(self._h), "dynakv_split_check")

    def decode_loop(self, q_steps, k_steps, v_steps, token_budget: int, out_steps=None):
        torch = self._torch
        U, G, d = self.cfg.n_units, self.cfg.gqa_group, self.cfg.head_dim
        n = q_steps.shape[0]
        if out_steps is None:
            out_steps = torch.empty((n, U, G, d), dtype=torch.float32, device=q_steps.device)
        self._check(self._L.dynakv_decode_loop(self._h, self._f32(q_steps, (n, U, G, d)), self._kv(k_steps, (n, U, d)),
                                               self._kv(v_steps, (n, U, d)), n, token_budget,
                                               self._f32(out_steps, (n, U, G, d))), "dynakv_decode_loop")
        self._keep = [q_steps, k_steps, v_steps, out_steps]
        return out_steps

    def decode_loop_host(self, q_host, k_host, v_host, token_budget: int, out_host) -> None:
        """The captured loop on HOST tensors [n, U, ...] (pinned for the copies to overlap the loop)."""
        U, G, d = self.cfg.n_units, self.cfg.gqa_group, self.cfg.head_dim
        n = q_host.shape[0]
        assert not q_host.is_cuda and not out_host.is_cuda
        self._check(self._L.dynakv_decode_loop_host(self._h, self._f32(q_host, (n, U, G, d)), self._kv(k_host, (n, U, d)),
                                                    self._kv(v_host, (n, U, d)), n, token_budget, self._f32(out_host, (n, U, G, d))),
                    "dynakv_decode_loop_host")

    def step_host(self, q_host, k_host, v_host, token_budget: int, out_host) -> None:
        U, G, d = self.cfg.n_units, self.cfg.gqa_group, self.cfg.head_dim
        assert not q_host.is_cuda and not out_host.is_cuda
        self._check(self._L.dynakv_step_host(self._h, self._f32(q_host, (U, G, d)), self._kv(k_host, (U, d)),
                                             self._kv(v_host, (U, d)), token_budget, self._f32(out_host, (U, G, d))),
                    "dynakv_step_host")

    def get_status(self) -> dict:
        s = _Status()
        self._check(self._L.dynakv_get_status(self._h, C.byref(s)), "dynakv_get_status")
        return {k: getattr(s, k) for k, _ in _Status._fields_}

    def export_state(self) -> dict:
        U, Mx, d, nt = self.cfg.n_units, self.cfg.max_clusters, self.cfg.head_dim, self.cfg.max_tokens
        out = {
            "tok_cluster": np.empty((U, nt), np.int32), "centroids": np.empty((U, Mx, d), np.float32),
            "counts": np.empty((U, Mx), np.int32), "M2": np.empty((U, Mx), np.float32),
            "n_tokens": np.empty(U, np.int32), "n_ids": np.empty(U, np.int32), "tau": np.empty(U, np.float32),
        }
        self._check(self._L.dynakv_export_state(self._h, *[_np_ptr(out[k]) for k in
                    ("tok_cluster", "centroids", "counts", "M2", "n_tokens", "n_ids", "tau")]), "dynakv_export_state")
        return out

    def export_kv(self, n: int):
        """K, V rows of the first n tokens of every unit in token-id order: two device tensors [U, n, d]."""
        import torch
        U, d = self.cfg.n_units, self.cfg.head_dim
        dt = torch.float32 if self.cfg.kv_dtype == F32 else torch.bfloat16
        with torch.cuda.stream(self._stream):
            K = torch.empty((U, n, d), dtype=dt, device="cuda")
            V = torch.empty_like(K)
        self._check(self._L.dynakv_export_kv(self._h, C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()), n), "dynakv_export_kv")
        return K, V

    def import_state(self, K, V, tok_cluster, n_ids, tau, n_build_clusters: int) -> None:
        """Resume from a checkpoint (export_state + export_kv) instead of building: K, V [U, n, d] device tensors,
        tok_cluster [U, n] (device tensor or array), n_ids [U] and tau [U] arrays."""
        import torch
        U, d = self.cfg.n_units, self.cfg.head_dim
        n = K.shape[1]
        tc = torch.as_tensor(np.ascontiguousarray(tok_cluster), dtype=torch.int32) if not torch.is_tensor(tok_cluster) else tok_cluster
        with torch.cuda.stream(self._stream):
            tc = tc.to(device="cuda", dtype=torch.int32).contiguous()
        self._stream.synchronize()
        if tuple(tc.shape) != (U, n):
            raise DynaKVError(f"expected tok_cluster of shape {(U, n)}, got {tuple(tc.shape)}")
        ids = np.ascontiguousarray(n_ids, dtype=np.int32); ta = np.ascontiguousarray(tau, dtype=np.float32)
        self._check(self._L.dynakv_import_state(self._h, self._kv(K, (U, n, d)), self._kv(V, (U, n, d)), n, C.c_void_p(tc.data_ptr()),
                                                _np_ptr(ids), _np_ptr(ta), n_build_clusters), "dynakv_import_state")

    def time_gather_attention(self, q, out, reps: int) -> float:
        """Milliseconds per launch of the gather-attention kernel over `reps` back-to-back launches on the last selection."""
        U, G, d = self.cfg.n_units, self.cfg.gqa_group, self.cfg.head_dim
        ms = np.zeros(1, np.float32)
        self._check(self._L.dynakv_time_gather_attention(self._h, self._f32(q, (U, G, d)), self._f32(out, (U, G, d)), reps,
                                                         _np_ptr(ms)), "dynakv_time_gather_attention")
        return float(ms[0])

    def selftest_wait_expiry(self) -> int:
        """Runs the bounded-wait self-test; returns 1 when the wait gave up as it must."""
        flag = np.zeros(1, np.int32)
        self._check(self._L.dynakv_selftest_wait_expiry(self._h, _np_ptr(flag)), "dynakv_selftest_wait_expiry")
        return int(flag[0])

    def get_selection(self):
        U = self.cfg.n_units
        a, b = np.empty(U, np.int32), np.empty(U, np.int32)
        self._check(self._L.dynakv_get_selection(self._h, _np_ptr(a), _np_ptr(b)), "dynakv_get_selection")
        return a, b

    def get_work_list(self):
        """The last decode step's gather list: (n_entries [U], entries [U, W, 2] = first row in the unit's page pool and
        row count of every run the attention kernel copied)."""
        U = self.cfg.n_units
        W = self._L.dynakv_work_list_capacity(self._h)
        n = np.empty(U, np.int32); e = np.empty((U, W, 2), np.int32)
        self._check(self._L.dynakv_get_work_list(self._h, _np_ptr(n), _np_ptr(e), W), "dynakv_get_work_list")
        return n, e

    def get_tier_stats(self) -> dict:
        """Two-tier mode: the cache counters since the context was created, summed over units."""
        st = _TierStats()
        self._check(self._L.dynakv_get_tier_stats(self._h, C.byref(st)), "dynakv_get_tier_stats")
        return {k: int(getattr(st, k)) for k, _ in _TierStats._fields_}

    def get_build_trace(self):
        U, T = self.cfg.n_units, self.cfg.kmeans_iters
        picks = np.empty((U, self.n_clusters0), np.int32)
        assign = np.empty((T, U, self.n_prefill), np.int32)
        self._check(self._L.dynakv_get_build_trace(self._h, _np_ptr(picks), _np_ptr(assign)), "dynakv_get_build_trace")
        return picks, assign

    def set_timing(self, on: bool) -> None:
        self._check(self._L.dynakv_set_timing(self._h, 1 if on else 0), "dynakv_set_timing")

    def get_kernel_times(self, reset: bool = True) -> dict:
        ms = np.zeros(len(KERNEL_CLASSES), np.float64); n = np.zeros(len(KERNEL_CLASSES), np.int64)
        self._check(self._L.dynakv_get_kernel_times(self._h, _np_ptr(ms), _np_ptr(n), 1 if reset else 0),
                    "dynakv_get_kernel_times")
        return {k: {"ms": float(ms[i]), "launches": int(n[i])} for i, k in enumerate(KERNEL_CLASSES)}

    def launch_count(self) -> int:
        return int(self._L.dynakv_launch_count(self._h))

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            self._L.dynakv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
