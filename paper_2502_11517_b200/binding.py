"""ctypes binding of the C ABI in include/pasta.h — argument marshalling only.

Function names match the C entry points (`pasta_` prefix dropped on the `Pool` methods).  Device
tensors are torch CUDA tensors whose data pointers are handed to the library; the current torch
stream is used unless a stream is given.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from .build import LIB

OK, INVALID_ARG, OUT_OF_PAGES, BAD_STATE, CAPACITY, CUDA, DEVICE_CHECK, TIMEOUT = range(8)
FLAG_HOST_ONLY, FLAG_NO_TENSOR_PATH, FLAG_OUT_BF16 = 1, 2, 4
_NAMES = ["OK", "INVALID_ARG", "OUT_OF_PAGES", "BAD_STATE", "CAPACITY", "CUDA", "DEVICE_CHECK", "TIMEOUT"]

EXPORTS = [
    "pasta_kv_bytes", "pasta_workspace_bytes", "pasta_pool_create", "pasta_pool_destroy",
    "pasta_request_begin", "pasta_request_end", "pasta_thread_spawn", "pasta_thread_finish",
    "pasta_sync_merge", "pasta_step_begin", "pasta_step_slots", "pasta_kv_append", "pasta_decode_attn",
    "pasta_kv_append_run", "pasta_step_host_bytes", "pasta_step_host", "pasta_kv_read",
    "pasta_pool_dump", "pasta_plan_dump", "pasta_pool_status", "pasta_launch_count",
    "pasta_profile_enable", "pasta_profile_read", "pasta_decode_attn_noalloc",
    "pasta_thread_spawn_predicted", "pasta_step_positions", "pasta_kv_append_rope", "pasta_rope_queries",
    "pasta_kv_append_run_rope", "pasta_step_device",
    "pasta_last_cuda_error", "pasta_debug_set_wait_limit", "pasta_debug_wait_expiry", "pasta_debug_hold_roles",
    "pasta_debug_stream_read", "pasta_step_host_begin", "pasta_step_host_wait",
    "pasta_dense_mask_scratch_bytes", "pasta_dense_append", "pasta_dense_mask_attn", "pasta_debug_set_tail",
    "pasta_debug_set_launch_overlap",
]


class PastaError(RuntimeError):
    def __init__(self, code: int, where: str):
        extra = f" (cudaError {lib().pasta_last_cuda_error()})" if code == CUDA else ""
        super().__init__(f"{where}: {_NAMES[code] if 0 <= code < len(_NAMES) else code}{extra}")
        self.code = code


class Config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("page_size", C.c_int32), ("n_pages", C.c_int32),
        ("max_requests", C.c_int32), ("max_threads_per_request", C.c_int32),
        ("max_segments_per_thread", C.c_int32), ("max_step_queries", C.c_int32),
        ("max_partial_rows", C.c_int32), ("max_layers_per_launch", C.c_int32),
        ("flags", C.c_int32), ("device", C.c_int32),
        ("kv_base", C.c_void_p), ("kv_bytes", C.c_size_t),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("free_order", C.POINTER(C.c_int32)),
    ]


_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built: there is no other implementation."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise RuntimeError(f"{LIB} is missing: run paper_2502_11517_b200.build.build() (needs nvcc); "
                               "this package has no CPU fallback")
        _lib = C.CDLL(LIB)
        for name in EXPORTS:
            getattr(_lib, name).restype = C.c_int32
        _lib.pasta_debug_set_launch_overlap.restype = None
    return _lib


def _check(code: int, where: str) -> None:
    if code != OK:
        raise PastaError(code, where)


def _i32(a) -> np.ndarray:
    if isinstance(a, np.ndarray) and a.dtype == np.int32 and a.flags.c_contiguous:
        return a                                  # callers that step in a loop convert once and pass arrays
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _dev(t) -> C.c_void_p:
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream if isinstance(stream, int) else stream.cuda_stream)


class Pool:
    """One KV pool on one GPU (or a host-only pool for bookkeeping tests)."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_pages: int,
                 max_requests: int, max_threads_per_request: int, max_segments_per_thread: int,
                 free_order=None, page_size: int = 16, max_step_queries: int = 0, max_partial_rows: int = 0,
                 max_layers_per_launch: int = 0, flags: int = 0, device: int = 0):
        self._h = C.c_void_p()
        self.cfg = cfg = Config()
        cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
        cfg.page_size, cfg.n_pages = page_size, n_pages
        cfg.max_requests, cfg.max_threads_per_request = max_requests, max_threads_per_request
        cfg.max_segments_per_thread = max_segments_per_thread
        cfg.max_step_queries, cfg.max_partial_rows = max_step_queries, max_partial_rows
        cfg.max_layers_per_launch, cfg.flags, cfg.device = max_layers_per_launch, flags, device
        self.host_only = bool(flags & FLAG_HOST_ONLY)
        L = lib()
        order = None if free_order is None else _i32(free_order)
        cfg.free_order = order.ctypes.data_as(C.POINTER(C.c_int32)) if order is not None else C.POINTER(C.c_int32)()
        self.kv = self.workspace = None
        if not self.host_only:
            import torch
            if not torch.cuda.is_available():
                raise RuntimeError("a CUDA device is required: this package has no CPU fallback")
            kvb, wsb = C.c_size_t(), C.c_size_t()
            _check(L.pasta_kv_bytes(C.byref(cfg), C.byref(kvb)), "pasta_kv_bytes")
            _check(L.pasta_workspace_bytes(C.byref(cfg), C.byref(wsb)), "pasta_workspace_bytes")
            dev = torch.device("cuda", device)
            # torch's caching allocator returns 512-byte aligned blocks; over-allocate to align to 1024
            self._kv_raw = torch.empty(kvb.value + 1024, dtype=torch.uint8, device=dev)
            off = (-self._kv_raw.data_ptr()) % 1024
            self.kv = self._kv_raw[off:off + kvb.value]
            self.workspace = torch.empty(wsb.value, dtype=torch.uint8, device=dev)
            cfg.kv_base, cfg.kv_bytes = self.kv.data_ptr(), kvb.value
            cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), wsb.value
            torch.cuda.synchronize(dev)
        _check(L.pasta_pool_create(C.byref(cfg), C.byref(self._h)), "pasta_pool_create")
        self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
        self._last_entries = (0, None)

    @property
    def _last_n(self) -> int:
        """Queries of the last planned step: one per entry, or one per new token of an entry that appends several."""
        n, nn = self._last_entries
        return n if nn is None else int(np.maximum(nn, 1).sum())

    def close(self) -> None:
        if self._h:
            lib().pasta_pool_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- lifecycle
    def request_begin(self) -> int:
        out = C.c_int32()
        _check(lib().pasta_request_begin(self._h, C.byref(out)), "pasta_request_begin")
        return out.value

    def request_end(self, req: int) -> None:
        _check(lib().pasta_request_end(self._h, req), "pasta_request_end")

    def thread_spawn(self, req: int) -> int:
        out = C.c_int32()
        _check(lib().pasta_thread_spawn(self._h, req, C.byref(out)), "pasta_thread_spawn")
        return out.value

    def thread_spawn_predicted(self, req: int, predicted_tokens: int, pending: int = 0) -> int:
        out = C.c_int32()
        _check(lib().pasta_thread_spawn_predicted(self._h, req, predicted_tokens, pending, C.byref(out)),
               "pasta_thread_spawn_predicted")
        return out.value

    def thread_finish(self, req: int, thread: int) -> None:
        _check(lib().pasta_thread_finish(self._h, req, thread), "pasta_thread_finish")

    def sync_merge(self, req: int, threads: Optional[Sequence[int]] = None) -> None:
        if threads is None:
            _check(lib().pasta_sync_merge(self._h, req, -1, None), "pasta_sync_merge")
        else:
            ids = _i32(threads)
            _check(lib().pasta_sync_merge(self._h, req, len(ids), _ptr(ids)), "pasta_sync_merge")

    # ---- one step
    def step_begin(self, req_ids, thread_ids, n_new=None, stream=None) -> None:
        r, t = _i32(req_ids), _i32(thread_ids)
        nn = None if n_new is None else _i32(n_new)
        st = C.c_void_p(0) if self.host_only else _stream(stream)
        _check(lib().pasta_step_begin(self._h, len(r), _ptr(r), _ptr(t), _ptr(nn), st), "pasta_step_begin")
        self._last_entries = (len(r), nn)             # the step's number of queries is worked out when asked for

    def step_slots(self) -> np.ndarray:
        out = np.empty((self._last_n, 2), dtype=np.int32)
        _check(lib().pasta_step_slots(self._h, _ptr(out), self._last_n), "pasta_step_slots")
        return out

    def step_positions(self) -> np.ndarray:
        out = np.empty(self._last_n, dtype=np.int32)
        _check(lib().pasta_step_positions(self._h, _ptr(out), self._last_n), "pasta_step_positions")
        return out

    def kv_append_rope(self, k_new, v_new, theta: float = 10000.0, layer_begin: int = 0,
                       layer_count: Optional[int] = None, stream=None) -> None:
        cnt = self.n_layers - layer_begin if layer_count is None else layer_count
        _check(lib().pasta_kv_append_rope(self._h, layer_begin, cnt, _dev(k_new), _dev(v_new), C.c_float(theta),
                                          _stream(stream)), "pasta_kv_append_rope")

    def rope_queries(self, q, theta: float = 10000.0, layer_count: Optional[int] = None, stream=None) -> None:
        cnt = self.n_layers if layer_count is None else layer_count
        _check(lib().pasta_rope_queries(self._h, cnt, _dev(q), C.c_float(theta), _stream(stream)), "pasta_rope_queries")

    def kv_append_run_rope(self, req: int, thread: int, m: int, k, v, theta: float = 10000.0, layer_begin: int = 0,
                           layer_count: Optional[int] = None, stream=None) -> None:
        cnt = self.n_layers - layer_begin if layer_count is None else layer_count
        _check(lib().pasta_kv_append_run_rope(self._h, req, thread, m, layer_begin, cnt, _dev(k), _dev(v),
                                              C.c_float(theta), _stream(stream)), "pasta_kv_append_run_rope")

    def kv_append(self, k_new, v_new, layer_begin: int = 0, layer_count: Optional[int] = None, stream=None) -> None:
        cnt = self.n_layers - layer_begin if layer_count is None else layer_count
        _check(lib().pasta_kv_append(self._h, layer_begin, cnt, _dev(k_new), _dev(v_new), _stream(stream)),
               "pasta_kv_append")

    def decode_attn(self, q, out, lse=None, scale: float = 0.0, layer_begin: int = 0,
                    layer_count: Optional[int] = None, stream=None) -> None:
        cnt = self.n_layers - layer_begin if layer_count is None else layer_count
        _check(lib().pasta_decode_attn(self._h, layer_begin, cnt, _dev(q), _dev(out), _dev(lse), C.c_float(scale),
                                       _stream(stream)), "pasta_decode_attn")

    def decode_attn_noalloc(self, q, out, lse=None, scale: float = 0.0, layer: int = 0, stream=None) -> None:
        """One layer of the planned step, partial results in the library's built-in device array: the call
        allocates nothing (see include/pasta.h for the size limit and the sharing rule)."""
        _check(lib().pasta_decode_attn_noalloc(self._h, layer, _dev(q), _dev(out), _dev(lse), C.c_float(scale),
                                               _stream(stream)), "pasta_decode_attn_noalloc")

    def kv_append_run(self, req: int, thread: int, m: int, k=None, v=None, layer_begin: int = 0,
                      layer_count: Optional[int] = None, stream=None) -> None:
        cnt = (0 if k is None else self.n_layers - layer_begin) if layer_count is None else layer_count
        st = C.c_void_p(0) if (self.host_only or cnt == 0) else _stream(stream)
        _check(lib().pasta_kv_append_run(self._h, req, thread, m, layer_begin, cnt, _dev(k), _dev(v), st),
               "pasta_kv_append_run")

    def step_device(self, req_ids, thread_ids, n_new, k_new, v_new, q, out, lse=None, scale: float = 0.0,
                    stream=None) -> None:
        """step_begin + kv_append + decode_attn for all layers in one library call (device tensors)."""
        r, t = _i32(req_ids), _i32(thread_ids)
        nn = None if n_new is None else _i32(n_new)
        _check(lib().pasta_step_device(self._h, len(r), _ptr(r), _ptr(t), _ptr(nn), _dev(k_new), _dev(v_new), _dev(q),
                                       _dev(out), _dev(lse), C.c_float(scale), _stream(stream)), "pasta_step_device")
        self._last_entries = (len(r), nn)

    def step_host_bytes(self, n: int) -> int:
        out = C.c_size_t()
        _check(lib().pasta_step_host_bytes(self._h, n, C.byref(out)), "pasta_step_host_bytes")
        return out.value

    def step_host(self, req_ids, thread_ids, n_new, k_new, v_new, q, out, staging, scale: float = 0.0,
                  stream=None) -> None:
        """k_new, v_new, q, out: host (CPU) torch tensors, ideally pinned; staging: device scratch tensor."""
        r, t = _i32(req_ids), _i32(thread_ids)
        nn = None if n_new is None else _i32(n_new)
        _check(lib().pasta_step_host(self._h, len(r), _ptr(r), _ptr(t), _ptr(nn), _dev(k_new), _dev(v_new), _dev(q),
                                     _dev(out), _dev(staging), C.c_size_t(staging.numel() * staging.element_size()),
                                     C.c_float(scale), _stream(stream)), "pasta_step_host")
        self._last_entries = (len(r), None)

    def step_host_begin(self, req_ids, thread_ids, n_new, k_new, v_new, q, out, staging, scale: float = 0.0,
                        stream=None) -> None:
        """First half of step_host: everything is enqueued, nothing is waited for (at most two steps in flight)."""
        r, t = _i32(req_ids), _i32(thread_ids)
        nn = None if n_new is None else _i32(n_new)
        _check(lib().pasta_step_host_begin(self._h, len(r), _ptr(r), _ptr(t), _ptr(nn), _dev(k_new), _dev(v_new), _dev(q),
                                           _dev(out), _dev(staging), C.c_size_t(staging.numel() * staging.element_size()),
                                           C.c_float(scale), _stream(stream)), "pasta_step_host_begin")
        self._last_entries = (len(r), None)

    def step_host_wait(self) -> None:
        _check(lib().pasta_step_host_wait(self._h), "pasta_step_host_wait")

    def debug_stream_read(self, src=None, mode: int = 0, stream=None) -> int:
        """Enqueues the read-only measurement kernel over `src` (a torch CUDA tensor; None = the pool's KV memory);
        returns the number of bytes it reads."""
        nbytes = self.kv.numel() if src is None else src.numel() * src.element_size()
        _check(lib().pasta_debug_stream_read(self._h, _dev(src), C.c_size_t(nbytes), mode, _stream(stream)),
               "pasta_debug_stream_read")
        return nbytes // 65536 * 65536 if mode else nbytes // 16 * 16

    # ---- introspection
    def kv_read(self, layer: int, req: int, stream_id: int, start: int, m: int, stream=None):
        import torch
        dev = self.kv.device
        k = torch.empty((m, self.n_kv_heads, self.head_dim), dtype=torch.bfloat16, device=dev)
        v = torch.empty_like(k)
        _check(lib().pasta_kv_read(self._h, layer, req, stream_id, start, m, _dev(k), _dev(v), _stream(stream)),
               "pasta_kv_read")
        return k, v

    def _words(self, fn, where: str) -> np.ndarray:
        need = C.c_size_t()
        _check(fn(self._h, None, C.c_size_t(0), C.byref(need)), where)
        buf = np.empty(need.value, dtype=np.int32)
        _check(fn(self._h, _ptr(buf), C.c_size_t(need.value), C.byref(need)), where)
        return buf

    def dump(self) -> dict:
        """The bookkeeping state, parsed into the same structure the tests build from their own model."""
        w = self._words(lib().pasta_pool_dump, "pasta_pool_dump").tolist()
        pos = 0

        def take(k=1):
            nonlocal pos
            out = w[pos:pos + k]
            pos += k
            return out

        reqs = {}
        for _ in range(take()[0]):
            req, n_streams = take(2)
            streams = {}
            for _s in range(n_streams):
                sid, ln, npg = take(3)
                streams[sid] = {"len": ln, "pages": take(npg)}
            threads = {}
            for _t in range(take()[0]):
                tid, state, cutoff, pos_next, nseg = take(5)
                threads[tid] = {"state": state, "cutoff": cutoff, "pos_next": pos_next,
                                "view": [tuple(take(3)) for _k in range(nseg)]}
            reqs[req] = {"streams": streams, "threads": threads}
        free = take(take()[0])
        assert pos == len(w)
        return {"requests": reqs, "free": free}

    def plan_words(self) -> np.ndarray:
        return self._words(lib().pasta_plan_dump, "pasta_plan_dump")

    def status(self, stream=None) -> int:
        st = C.c_void_p(0) if self.host_only else _stream(stream)
        return lib().pasta_pool_status(self._h, st)

    def profile_enable(self, on=True) -> None:
        """False / 0: off; True / 1: time every launch group; k > 1: time every k-th one."""
        _check(lib().pasta_profile_enable(self._h, int(on)), "pasta_profile_enable")

    def profile_read(self):
        """(ms, launches): device time and number of timed launches of the tensor, warp and merge kernels."""
        ms = (C.c_double * 3)()
        cnt = (C.c_int64 * 3)()
        _check(lib().pasta_profile_read(self._h, ms, cnt), "pasta_profile_read")
        return list(ms), list(cnt)

    def debug_set_wait_limit(self, cycles: int) -> None:
        _check(lib().pasta_debug_set_wait_limit(self._h, C.c_int64(cycles)), "pasta_debug_set_wait_limit")

    def debug_set_tail(self, percent: int, tiles: int) -> None:
        _check(lib().pasta_debug_set_tail(self._h, percent, tiles), "pasta_debug_set_tail")

    @staticmethod
    def debug_set_launch_overlap(on: bool) -> None:
        lib().pasta_debug_set_launch_overlap(1 if on else 0)

    def debug_hold_roles(self, role_mask: int) -> None:
        _check(lib().pasta_debug_hold_roles(self._h, role_mask), "pasta_debug_hold_roles")

    def debug_wait_expiry(self, stream=None) -> None:
        _check(lib().pasta_debug_wait_expiry(self._h, _stream(stream)), "pasta_debug_wait_expiry")

    def launch_count(self) -> int:
        out = C.c_int64()
        _check(lib().pasta_launch_count(self._h, C.byref(out)), "pasta_launch_count")
        return out.value


# ---- the stateless calls of the dense-pool comparison layout (tensors are held by dense_mask.DensePool)
def dense_mask_scratch_bytes(n_queries: int, n_slots: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> int:
    out = C.c_size_t()
    _check(lib().pasta_dense_mask_scratch_bytes(n_queries, n_slots, n_q_heads, n_kv_heads, head_dim, C.byref(out)),
           "pasta_dense_mask_scratch_bytes")
    return out.value


def dense_append(k_pool, v_pool, mask, own, slot0: int, rows, k_new, v_new, stream=None) -> None:
    r = _i32(rows)
    _check(lib().pasta_dense_append(_dev(k_pool), _dev(v_pool), _dev(mask), _dev(own), C.c_int64(mask.shape[1]), slot0,
                                    len(r), _ptr(r), _dev(k_new), _dev(v_new), k_pool.shape[1], k_pool.shape[2],
                                    _stream(stream)), "pasta_dense_append")


def dense_mask_attn(k_pool, v_pool, mask, mask_row, q, out, lse, scratch, n_slots: int, scale: float = 0.0,
                    stream=None) -> None:
    _check(lib().pasta_dense_mask_attn(_dev(k_pool), _dev(v_pool), _dev(mask), C.c_int64(mask.shape[1]), _dev(mask_row),
                                       _dev(q), _dev(out), _dev(lse), _dev(scratch), C.c_size_t(scratch.numel()),
                                       q.shape[0], n_slots, q.shape[1], k_pool.shape[1], k_pool.shape[2], C.c_float(scale),
                                       _stream(stream)), "pasta_dense_mask_attn")
