"""ctypes binding of ``include/hpl.h``: the same calls, argument marshalling only.

Every step of the hot path runs inside the library; nothing here computes.  Device pointers
are plain integers (e.g. ``tensor.data_ptr()``), host buffers anything exposing the buffer
protocol or an integer address.
"""
from __future__ import annotations

import ctypes as C
import os

HPL_OK = 0
HPL_ERR_INVALID, HPL_ERR_NOT_FOUND, HPL_ERR_EXISTS, HPL_ERR_TIMEOUT = -1, -2, -3, -4
HPL_ERR_INSUFFICIENT, HPL_ERR_FAILED_WORKER, HPL_ERR_CUDA, HPL_ERR_NOMEM = -5, -6, -7, -8
HPL_F32, HPL_BF16 = 0, 1
HPL_SUM, HPL_MIN, HPL_MAX = 0, 1, 2
(HPL_EV_CREATE, HPL_EV_PUT, HPL_EV_PUT_HOST, HPL_EV_REDUCE, HPL_EV_BROADCAST, HPL_EV_JOIN, HPL_EV_FAIL, HPL_EV_REJOIN,
 HPL_EV_PROGRESS, HPL_EV_GET, HPL_EV_DELETE, HPL_EV_SYNC, HPL_EV_MARK) = range(1, 14)

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


def lib_path() -> str:
    """The library this process uses: ``libhpl.so``, or with ``HPL_DEBUG_BOUNDS=1`` in the environment the
    bounds-checking build ``libhpl_debug.so`` (same code, kernels check every tile against the directory)."""
    return os.path.join(_HERE, "libhpl_debug.so" if os.environ.get("HPL_DEBUG_BOUNDS") == "1" else "libhpl.so")


class Config(C.Structure):
    """Mirror of ``hpl_config``."""
    _fields_ = [("chunk_bytes", C.c_uint64), ("reduce_degree", C.c_int32), ("bcast_degree", C.c_int32),
                ("virt_chunk_ns", C.c_uint64), ("poll_budget_ns", C.c_uint64), ("eager", C.c_int32),
                ("plan_ahead", C.c_int32), ("fuse", C.c_int32), ("time_kernels", C.c_int32),
                ("arena", C.c_void_p), ("arena_bytes", C.c_uint64),
                ("model_latency_ns", C.c_uint64), ("model_bandwidth_bps", C.c_uint64),
                ("fuse_fanout", C.c_int32), ("pipeline_chunks", C.c_int32), ("debug_guard_bytes", C.c_uint64),
                ("rank", C.c_int32), ("world_size", C.c_int32)]


class Stats(C.Structure):
    """Mirror of ``hpl_stats_t``."""
    _fields_ = [(n, C.c_uint64) for n in ("kernel_launches", "reduce_tasks", "fanout_tasks", "tiles",
                                          "bytes_read_planned", "bytes_written_planned", "device_timeouts",
                                          "arena_used", "h2d_bytes", "d2h_bytes", "last_kernel_grid",
                                          "reduce_launches", "fanout_launches", "reduce_kernel_ns",
                                          "fanout_kernel_ns", "device_waits", "fused_fanout_tasks", "evictions", "bounds_errors")]


class Event(C.Structure):
    """Mirror of ``hpl_event``."""
    _fields_ = [("t_ns", C.c_uint64), ("kind", C.c_int32), ("worker", C.c_int32), ("object_id", C.c_int64),
                ("ptr", C.c_void_p), ("bytes", C.c_uint64), ("ids", C.POINTER(C.c_int64)), ("n_ids", C.c_int32),
                ("k", C.c_int32), ("op", C.c_int32), ("dtype", C.c_int32)]


class EventList:
    """A timeline prepared once for ``Context.submit``: a ctypes array of ``hpl_event`` plus the id arrays its
    Reduce / broadcast requests point to (kept alive here).  ``add`` takes the fields by name."""

    def __init__(self, capacity: int):
        self.array = (Event * capacity)()
        self.n = 0
        self._keep = []

    def add(self, kind: int, t_ns: int = 0, object_id: int = 0, worker: int = 0, ptr: int = 0, nbytes: int = 0, ids=None,
            k: int = 0, op: int = HPL_SUM, dtype: int = HPL_F32):
        e = self.array[self.n]
        self.n += 1
        e.t_ns, e.kind, e.worker, e.object_id, e.ptr, e.bytes = t_ns, kind, worker, object_id, ptr or None, nbytes
        e.k, e.op, e.dtype = k, op, dtype
        if ids is not None:
            arr = (C.c_int64 * len(ids))(*ids)
            self._keep.append(arr)
            e.ids, e.n_ids = arr, len(ids)
        return self

    def __len__(self):
        return self.n


class HplError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {code} ({_strerror(code)})")


def _strerror(code: int) -> str:
    try:
        return load_library().hpl_strerror(code).decode()
    except Exception:  # pragma: no cover
        return "?"


def load_library():
    """Loads ``libhpl.so``.  There is no fallback: a missing library is an error."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2002_05814_b200.build`")
    lib = C.CDLL(path)
    P, I32, I64, U64, VP = C.POINTER, C.c_int32, C.c_int64, C.c_uint64, C.c_void_p
    sig = {
        "hpl_init": [P(Config), VP, P(VP)],
        "hpl_shutdown": [VP],
        "hpl_advance": [VP, U64],
        "hpl_create": [VP, I64, I32, U64, I32],
        "hpl_put": [VP, I64, VP, U64],
        "hpl_put_host": [VP, I64, VP, U64],
        "hpl_create_batch": [VP, I32, P(I64), P(I32), U64, I32, P(I32)],
        "hpl_put_batch": [VP, I32, P(I64), P(VP), P(U64), P(I32)],
        "hpl_join_batch": [VP, I32, P(I64), P(VP), P(I32)],
        "hpl_get_batch": [VP, I32, P(I64), P(VP), P(I32)],
        "hpl_submit": [VP, P(Event), I32, P(I32)],
        "hpl_reduce": [VP, I64, P(I64), I32, I32, I32, I32],
        "hpl_broadcast": [VP, I64, P(I64), I32],
        "hpl_join": [VP, I64, VP],
        "hpl_get": [VP, I64, P(VP), P(U64)],
        "hpl_get_host": [VP, I64, VP, U64],
        "hpl_fail": [VP, I32],
        "hpl_rejoin": [VP, I32],
        "hpl_delete": [VP, I64],
        "hpl_progress": [VP],
        "hpl_sync": [VP],
        "hpl_schedule_dump": [VP, I64, P(I64), U64, P(U64)],
        "hpl_stats": [VP, P(Stats)],
        "hpl_check_guards": [VP, P(U64)],
        "hpl_set_peer_arena": [VP, I32, VP],
        "hpl_pending_levels": [VP, P(I32)],
        "hpl_run_level": [VP],
        "hpl_fail_rank": [VP, I32],
        "hpl_ipc_export": [VP, P(C.c_uint8), P(U64)],
        "hpl_ipc_import": [P(C.c_uint8), U64, P(VP)],
        "hpl_ipc_close": [VP],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.hpl_reduce_noalloc.argtypes = [P(VP), I32, I32, I32, I32, U64, VP, VP]
    lib.hpl_reduce_noalloc.restype = C.c_int
    lib.hpl_choose_degree.argtypes = [I32, U64, C.c_double, C.c_double]
    lib.hpl_choose_degree.restype = I32
    lib.hpl_strerror.argtypes = [C.c_int]
    lib.hpl_strerror.restype = C.c_char_p
    _LIB = lib
    return lib


def _addr(buf) -> int:
    if isinstance(buf, int):
        return buf
    if hasattr(buf, "data_ptr"):        # torch tensor (host or device)
        return buf.data_ptr()
    if hasattr(buf, "ctypes"):          # numpy array
        return buf.ctypes.data
    return C.addressof(C.c_char.from_buffer(buf))


class Context:
    """One ``hpl_ctx``.  Methods are the C calls of the same name; errors raise :class:`HplError`
    unless the method is documented to return the code."""

    def __init__(self, chunk_bytes: int, reduce_degree: int = 2, bcast_degree: int = 2, *, arena=0,
                 arena_bytes: int = 0, stream=0, virt_chunk_ns: int = 0, poll_budget_ns: int = 0,
                 eager: bool = False, plan_ahead: bool = False, fuse: bool = True, time_kernels: bool = False,
                 model_latency_ns: int = 0, model_bandwidth_bps: int = 0, fuse_fanout: bool = True,
                 debug_guard_bytes: int = 0, rank: int = 0, world_size: int = 1, pipeline_chunks: int = 0):
        self._lib = load_library()
        cfg = Config(chunk_bytes, reduce_degree, bcast_degree, virt_chunk_ns, poll_budget_ns, int(eager),
                     int(plan_ahead), int(fuse), int(time_kernels), _addr(arena) if arena else None, arena_bytes,
                     model_latency_ns, model_bandwidth_bps, int(fuse_fanout), pipeline_chunks, debug_guard_bytes, rank, world_size)
        self._h = C.c_void_p()
        self._p, self._n = C.c_void_p(), C.c_uint64()
        self._pref, self._nref = C.byref(self._p), C.byref(self._n)
        self._check(self._lib.hpl_init(C.byref(cfg), C.c_void_p(stream or None), C.byref(self._h)), "hpl_init")

    def _check(self, rc: int, what: str) -> int:
        if rc != HPL_OK:
            raise HplError(rc, what)
        return rc

    def shutdown(self):
        if self._h:
            self._lib.hpl_shutdown(self._h)
            self._h = C.c_void_p()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.shutdown()

    # the per-object calls below are on every step's path: they pass plain integers straight to ctypes
    def advance(self, t_ns: int):
        rc = self._lib.hpl_advance(self._h, t_ns)
        if rc:
            raise HplError(rc, "hpl_advance")

    def create(self, object_id: int, worker: int, total_bytes: int, dtype: int = HPL_F32):
        rc = self._lib.hpl_create(self._h, object_id, worker, total_bytes, dtype)
        if rc:
            raise HplError(rc, "hpl_create")

    def put(self, object_id: int, dev_buf, nbytes: int):
        rc = self._lib.hpl_put(self._h, object_id, dev_buf if type(dev_buf) is int else _addr(dev_buf), nbytes)
        if rc:
            raise HplError(rc, "hpl_put")

    # batch forms: the arrays may be prepared once (``ids_array`` etc.) and reused
    @staticmethod
    def ids_array(ids):
        return (C.c_int64 * len(ids))(*ids)

    @staticmethod
    def ptr_array(ptrs):
        return (C.c_void_p * len(ptrs))(*ptrs)

    def create_batch(self, ids, workers, total_bytes: int, dtype: int = HPL_F32):
        ids = ids if isinstance(ids, C.Array) else self.ids_array(ids)
        wk = workers if isinstance(workers, C.Array) else (C.c_int32 * len(workers))(*workers)
        self._check(self._lib.hpl_create_batch(self._h, len(ids), ids, wk, total_bytes, dtype, None), "hpl_create_batch")

    def put_batch(self, ids, dev_ptrs, nbytes):
        ids = ids if isinstance(ids, C.Array) else self.ids_array(ids)
        ptrs = dev_ptrs if isinstance(dev_ptrs, C.Array) else self.ptr_array(dev_ptrs)
        nb = nbytes if isinstance(nbytes, C.Array) else (C.c_uint64 * len(ids))(*([nbytes] * len(ids) if isinstance(nbytes, int) else nbytes))
        self._check(self._lib.hpl_put_batch(self._h, len(ids), ids, ptrs, nb, None), "hpl_put_batch")

    def join_batch(self, ids, dev_ptrs):
        ids = ids if isinstance(ids, C.Array) else self.ids_array(ids)
        ptrs = dev_ptrs if isinstance(dev_ptrs, C.Array) else self.ptr_array(dev_ptrs)
        self._check(self._lib.hpl_join_batch(self._h, len(ids), ids, ptrs, None), "hpl_join_batch")

    def get_batch(self, ids, out_ptrs=None):
        """``hpl_get`` for every id; returns the device pointers (or fills the ctypes array ``out_ptrs``)."""
        ids = ids if isinstance(ids, C.Array) else self.ids_array(ids)
        out = out_ptrs if out_ptrs is not None else (C.c_void_p * len(ids))()
        self._check(self._lib.hpl_get_batch(self._h, len(ids), ids, out, None), "hpl_get_batch")
        return out if out_ptrs is not None else list(out)

    def submit(self, events: EventList):
        """``hpl_submit``: the whole prepared timeline in one call.  Results of Get events are in ``events.array``."""
        done = C.c_int32()
        rc = self._lib.hpl_submit(self._h, events.array, events.n, C.byref(done))
        if rc:
            raise HplError(rc, f"hpl_submit (event {done.value} of {events.n})")

    def put_host(self, object_id: int, host_buf, nbytes: int):
        self._check(self._lib.hpl_put_host(self._h, object_id, C.c_void_p(_addr(host_buf)), nbytes), "hpl_put_host")

    def reduce(self, target_id: int, src_ids, k_first_ready: int, op: int = HPL_SUM, dtype: int = HPL_F32):
        arr = (C.c_int64 * len(src_ids))(*src_ids)
        self._check(self._lib.hpl_reduce(self._h, target_id, arr, len(src_ids), k_first_ready, op, dtype), "hpl_reduce")

    def broadcast(self, src_id: int, dst_ids):
        arr = (C.c_int64 * len(dst_ids))(*dst_ids)
        self._check(self._lib.hpl_broadcast(self._h, src_id, arr, len(dst_ids)), "hpl_broadcast")

    def join(self, dst_id: int, dev_buf=0):
        if dev_buf is None:
            ptr = None
        else:
            ptr = dev_buf if type(dev_buf) is int else _addr(dev_buf)
        rc = self._lib.hpl_join(self._h, dst_id, ptr)
        if rc:
            raise HplError(rc, "hpl_join")

    def get(self, object_id: int):
        """Returns ``(device_pointer, nbytes)``."""
        p, n = self._p, self._n
        rc = self._lib.hpl_get(self._h, object_id, self._pref, self._nref)
        if rc:
            raise HplError(rc, "hpl_get")
        return p.value, n.value

    def try_get(self, object_id: int):
        """As :meth:`get` but returns ``(code, device_pointer, nbytes)`` instead of raising."""
        p, n = C.c_void_p(), C.c_uint64()
        rc = self._lib.hpl_get(self._h, object_id, C.byref(p), C.byref(n))
        return rc, p.value, n.value

    def get_host(self, object_id: int, host_buf, cap: int):
        self._check(self._lib.hpl_get_host(self._h, object_id, C.c_void_p(_addr(host_buf)), cap), "hpl_get_host")

    def fail(self, worker: int):
        self._check(self._lib.hpl_fail(self._h, worker), "hpl_fail")

    def rejoin(self, worker: int):
        self._check(self._lib.hpl_rejoin(self._h, worker), "hpl_rejoin")

    def delete(self, object_id: int):
        self._check(self._lib.hpl_delete(self._h, object_id), "hpl_delete")

    def progress(self):
        self._check(self._lib.hpl_progress(self._h), "hpl_progress")

    def sync(self) -> int:
        """Returns the code (HPL_OK or HPL_ERR_TIMEOUT) instead of raising on a timeout."""
        rc = self._lib.hpl_sync(self._h)
        if rc not in (HPL_OK, HPL_ERR_TIMEOUT):
            raise HplError(rc, "hpl_sync")
        return rc

    def schedule_dump(self, op_id: int) -> list[int]:
        n = C.c_uint64()
        rc = self._lib.hpl_schedule_dump(self._h, op_id, None, 0, C.byref(n))
        if rc == HPL_ERR_NOT_FOUND:
            raise HplError(rc, "hpl_schedule_dump")
        buf = (C.c_int64 * n.value)()
        self._check(self._lib.hpl_schedule_dump(self._h, op_id, buf, n.value, C.byref(n)), "hpl_schedule_dump")
        return list(buf)

    # ---- worker-per-GPU mode (world_size > 1): every rank makes the same calls; see include/hpl.h
    def set_peer_arena(self, rank: int, arena_base: int):
        self._check(self._lib.hpl_set_peer_arena(self._h, rank, C.c_void_p(arena_base)), "hpl_set_peer_arena")

    def pending_levels(self) -> int:
        n = C.c_int32()
        self._check(self._lib.hpl_pending_levels(self._h, C.byref(n)), "hpl_pending_levels")
        return n.value

    def run_level(self):
        self._check(self._lib.hpl_run_level(self._h), "hpl_run_level")

    def fail_rank(self, rank: int):
        self._check(self._lib.hpl_fail_rank(self._h, rank), "hpl_fail_rank")

    def drive(self, barrier):
        """Called by every live rank together: plans, then releases the plan level by level -- own tasks of the level,
        wait for the own stream, ``barrier()`` over the live ranks -- and plans again until nothing is left to do."""
        while True:
            self.progress()
            n = self.pending_levels()
            if n == 0:
                return
            for _ in range(n):
                self.run_level()
                self.sync()
                barrier()

    def check_guards(self) -> int:
        """``hpl_check_guards``: canary bytes behind arena blocks found changed so far (0 without debug_guard_bytes)."""
        n = C.c_uint64()
        self._check(self._lib.hpl_check_guards(self._h, C.byref(n)), "hpl_check_guards")
        return n.value

    def stats(self) -> dict:
        st = Stats()
        self._check(self._lib.hpl_stats(self._h, C.byref(st)), "hpl_stats")
        return {name: getattr(st, name) for name, _ in Stats._fields_}


def reduce_noalloc(src_ptrs, degree: int, op: int, dtype: int, elems: int, out_ptr: int, stream: int = 0) -> int:
    """``hpl_reduce_noalloc``: the tree reduce for callers that cannot allocate device memory (no context,
    no arena; its small scratch is a fixed array inside the library).  ``src_ptrs``: device addresses of the
    complete objects in arrival order; ``out_ptr``: device fp32 buffer.  Returns the library's code."""
    lib = load_library()
    arr = (C.c_void_p * len(src_ptrs))(*src_ptrs)
    return lib.hpl_reduce_noalloc(arr, len(src_ptrs), degree, op, dtype, elems, C.c_void_p(out_ptr), C.c_void_p(stream or None))


def ipc_export(dev_ptr: int):
    """``hpl_ipc_export``: ``(handle, offset)`` -- the 64-byte CUDA IPC handle of the allocation that holds ``dev_ptr``
    and the pointer's offset inside it."""
    h = (C.c_uint8 * 64)()
    off = C.c_uint64()
    rc = load_library().hpl_ipc_export(C.c_void_p(dev_ptr), h, C.byref(off))
    if rc:
        raise HplError(rc, "hpl_ipc_export")
    return bytes(h), off.value


def ipc_import(handle: bytes, offset: int = 0) -> int:
    """``hpl_ipc_import``: maps another process' allocation; returns the address of the exported byte in this process."""
    h = (C.c_uint8 * 64)(*handle)
    p = C.c_void_p()
    rc = load_library().hpl_ipc_import(h, offset, C.byref(p))
    if rc:
        raise HplError(rc, "hpl_ipc_import")
    return p.value


def ipc_close(dev_ptr: int):
    rc = load_library().hpl_ipc_close(C.c_void_p(dev_ptr))
    if rc:
        raise HplError(rc, "hpl_ipc_close")


def choose_degree(n: int, object_bytes: int, latency_s: float, bandwidth_bytes_per_s: float) -> int:
    """``hpl_choose_degree``: Eq. 1's best degree among 1, 2 and n."""
    return load_library().hpl_choose_degree(n, object_bytes, latency_s, bandwidth_bytes_per_s)
