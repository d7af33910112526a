"""ctypes binding of libsparbit_b200.so: argument marshalling only, same names as the C ABI.

Every step of a collective runs in the library's CUDA kernels.  There is no fallback: if the
shared library is missing or cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

_LIB_PATH = Path(__file__).resolve().parent / "libsparbit_b200.so"

OK = 0
(ERR_ARG, ERR_OVERFLOW, ERR_ALIAS, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NOMEM, ERR_LIMIT,
 ERR_BARRIER) = range(1, 11)
MULTI_MAX_DEVICES = 16
IPC_HANDLE_BYTES = 64
ALGO_SPARBIT, ALGO_RING, ALGO_RECURSIVE_DOUBLING, ALGO_BRUCK, ALGO_NEIGHBOR_EXCHANGE = range(5)
EXEC_AUTO, EXEC_PERSISTENT, EXEC_GRAPH, EXEC_STREAM, EXEC_FLOW, EXEC_MIRROR = range(6)
COPY_AUTO, COPY_VECTOR, COPY_BULK = range(3)
SPACE_SEND, SPACE_RECV, SPACE_WORKSPACE = range(3)
MAP_SEQUENTIAL, MAP_CYCLIC = range(2)
(TUNE_BULK_MIN_BLOCK_BYTES, TUNE_BULK_MIN_MOVED_BYTES, TUNE_FLOW_UNITS_PER_WARP, TUNE_FLOW_MAX_UNIT_SPANS,
 TUNE_FLOW_MIN_MOVED_BYTES, TUNE_FLOW_MAX_MOVED_BYTES, TUNE_MIRROR_MAX_BYTES,
 TUNE_FLOW_MIN_PASS_SPANS, TUNE_MIRROR_MAX_VECTORS, TUNE_MIRROR_CLUSTER_MAX_BLOCK,
 TUNE_MIRROR_CTA_VECTORS, TUNE_MIRROR_THREAD_VECTORS, TUNE_FLOW_COOPERATIVE, TUNE_FLOW_SKIP_WAITS,
 TUNE_GROUPED_FRONT, TUNE_FLOW_WIDE_MAX_MOVED_BYTES, TUNE_VEC_DENSE_MAX_RECV_BYTES,
 TUNE_STREAM_MAX_LAUNCHES) = range(18)

ALGO_NAMES = {ALGO_SPARBIT: "sparbit", ALGO_RING: "ring", ALGO_RECURSIVE_DOUBLING: "recursive_doubling",
              ALGO_BRUCK: "bruck", ALGO_NEIGHBOR_EXCHANGE: "neighbor_exchange"}
EXEC_NAMES = {EXEC_AUTO: "auto", EXEC_PERSISTENT: "persistent", EXEC_GRAPH: "graph", EXEC_STREAM: "stream",
              EXEC_FLOW: "flow", EXEC_MIRROR: "mirror"}
COPY_NAMES = {COPY_AUTO: "auto", COPY_VECTOR: "vector", COPY_BULK: "bulk"}

MSG_DTYPE = np.dtype([("phase", "<i4"), ("src_rank", "<i4"), ("dst_rank", "<i4"), ("src_space", "<i4"),
                      ("src_slot", "<i4"), ("dst_space", "<i4"), ("dst_slot", "<i4")])

#: every symbol include/sparbit.h declares, with (restype, argtypes)
_vp, _sz, _i, _u64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64
_pi = ctypes.POINTER(ctypes.c_int)
SYMBOLS = {
    "sparbit_plan": (_vp, [_i, _sz]),
    "sparbit_plan_create": (_i, [_i, _sz, _i, _i, ctypes.POINTER(_vp)]),
    "sparbit_plan_create_v": (_i, [_i, ctypes.POINTER(_sz), _i, _i, ctypes.POINTER(_vp)]),
    "sparbit_plan_destroy": (_i, [_vp]),
    "sparbit_allgather": (_i, [_vp, _vp, _vp, _vp]),
    "sparbit_allgather_steps": (_i, [_vp, _vp, _vp, _vp, _i, _i]),
    "sparbit_allgather_host": (_i, [_vp, _vp, _vp]),
    "sparbit_plan_num_steps": (_i, [_vp]),
    "sparbit_plan_last_phase": (_i, [_vp]),
    "sparbit_plan_step_info": (_i, [_vp, _i, _pi, _pi, _pi]),
    "sparbit_plan_messages": (_i, [_vp, _i, _vp, _sz, ctypes.POINTER(_sz)]),
    "sparbit_plan_validate": (_i, [_vp, _pi]),
    "sparbit_plan_validate_flow": (_i, [_vp, _i, _i, _pi, _pi]),
    "sparbit_rank_device": (_i, [_i, _i, _i, _i]),
    "sparbit_plan_partition": (_i, [_vp, _i, _i, _i, ctypes.POINTER(_u64)]),
    "sparbit_plan_partition_messages": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _sz, ctypes.POINTER(_sz)]),
    "sparbit_multi_rank_count": (_i, [_i, _i, _i, _i]),
    "sparbit_multi_local_index": (_i, [_i, _i, _i, _i]),
    "sparbit_allgather_multi_phases": (_i, [_vp, _i, _i, _i, _vp, ctypes.POINTER(_vp), _vp, _i, _i]),
    "sparbit_allgather_multi": (_i, [_vp, _i, _i, _i, _vp, ctypes.POINTER(_vp), _vp, _vp, _vp]),
    "sparbit_ipc_export": (_i, [_vp, _vp, ctypes.POINTER(_u64)]),
    "sparbit_ipc_open": (_i, [_vp, _u64, ctypes.POINTER(_vp), ctypes.POINTER(_vp)]),
    "sparbit_ipc_close": (_i, [_vp]),
    "sparbit_plan_workspace_bytes": (_sz, [_vp]),
    "sparbit_plan_set_workspace": (_i, [_vp, _vp, _sz]),
    "sparbit_plan_set_copy_path": (_i, [_vp, _i]),
    "sparbit_plan_set_tunable": (_i, [_vp, _i, _u64]),
    "sparbit_plan_get_tunable": (_i, [_vp, _i, ctypes.POINTER(_u64)]),
    "sparbit_plan_exec_mode": (_i, [_vp]),
    "sparbit_plan_copy_path": (_i, [_vp]),
    "sparbit_plan_launch_counts": (_i, [_vp, ctypes.POINTER(_u64), ctypes.POINTER(_u64)]),
    "sparbit_plan_status": (_i, [_vp, _pi]),
    "sparbit_plan_set_trace": (_i, [_vp, _i]),
    "sparbit_plan_get_trace": (_i, [_vp, ctypes.POINTER(_u64), _sz, ctypes.POINTER(_sz)]),
    "sparbit_plan_set_barrier_test": (_i, [_vp, _i, _u64]),
    "sparbit_plan_set_mbarrier_test": (_i, [_vp, ctypes.c_uint32, _u64]),
    "sparbit_allgather_noalloc": (_i, [_i, _sz, _i, _vp, _vp, _vp]),
    "sparbit_strerror": (ctypes.c_char_p, [_i]),
    "sparbit_last_cuda_error": (ctypes.c_char_p, []),
}

if not _LIB_PATH.exists():
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2109_08751_b200.build` "
        "(there is no fallback path)")
lib = ctypes.CDLL(str(_LIB_PATH))
for _name, (_res, _args) in SYMBOLS.items():
    _fn = getattr(lib, _name)  # AttributeError here means the library does not match the header
    _fn.restype = _res
    _fn.argtypes = _args


#: sparbit_device_barrier_fn
BARRIER_FN = ctypes.CFUNCTYPE(_i, _vp, _vp)


class SparbitError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib.sparbit_strerror(code).decode()
        if code == ERR_CUDA:
            msg += ": " + lib.sparbit_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (code {code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise SparbitError(code, where)


def _ptr(x) -> int | None:
    """Device or host address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()  # torch.Tensor


def _stream_handle(stream) -> int | None:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream  # torch.cuda.Stream


class Plan:
    """A plan of the C library (sparbit_plan_create ... sparbit_plan_destroy)."""

    def __init__(self, P: int, block_bytes: int, algo: int = ALGO_SPARBIT, exec_mode: int = EXEC_AUTO):
        h = _vp()
        _check(lib.sparbit_plan_create(P, block_bytes, algo, exec_mode, ctypes.byref(h)), "sparbit_plan_create")
        self._h = h
        self.P, self.block_bytes, self.algo = P, block_bytes, algo
        self._workspace = None

    @classmethod
    def create_v(cls, block_bytes, algo: int = ALGO_SPARBIT, exec_mode: int = EXEC_AUTO) -> "Plan":
        """A plan for blocks of different sizes (sparbit_plan_create_v): block_bytes[j] is the
        byte count rank j contributes."""
        counts = [int(x) for x in block_bytes]
        arr = (_sz * len(counts))(*counts)
        h = _vp()
        _check(lib.sparbit_plan_create_v(len(counts), arr, algo, exec_mode, ctypes.byref(h)),
               "sparbit_plan_create_v")
        self = cls.__new__(cls)
        self._h = h
        self.P, self.block_bytes, self.algo = len(counts), counts, algo
        self._workspace = None
        return self

    # -- the collective
    def allgather(self, sendbuf, recvbuf, stream=None) -> None:
        _check(lib.sparbit_allgather(self._h, _ptr(sendbuf), _ptr(recvbuf), _stream_handle(stream)),
               "sparbit_allgather")

    def allgather_steps(self, sendbuf, recvbuf, first: int, last: int, stream=None) -> None:
        _check(lib.sparbit_allgather_steps(self._h, _ptr(sendbuf), _ptr(recvbuf), _stream_handle(stream),
                                           first, last), "sparbit_allgather_steps")

    def allgather_host(self, host_send, host_recv) -> None:
        _check(lib.sparbit_allgather_host(self._h, _ptr(host_send), _ptr(host_recv)), "sparbit_allgather_host")

    # -- introspection
    @property
    def num_steps(self) -> int:
        return lib.sparbit_plan_num_steps(self._h)

    @property
    def last_phase(self) -> int:
        return lib.sparbit_plan_last_phase(self._h)

    def step_info(self, step: int):
        d, n, ig = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        _check(lib.sparbit_plan_step_info(self._h, step, ctypes.byref(d), ctypes.byref(n), ctypes.byref(ig)),
               "sparbit_plan_step_info")
        return d.value, n.value, ig.value

    def messages(self, phase: int) -> np.ndarray:
        n = _sz()
        _check(lib.sparbit_plan_messages(self._h, phase, None, 0, ctypes.byref(n)), "sparbit_plan_messages")
        out = np.zeros(n.value, dtype=MSG_DTYPE)
        if n.value:
            _check(lib.sparbit_plan_messages(self._h, phase, out.ctypes.data, n.value, ctypes.byref(n)),
                   "sparbit_plan_messages")
        return out

    def partition(self, G: int, mapping: int, phase: int) -> np.ndarray:
        """blocks[s, d] = blocks ranks on device s send to ranks on device d in `phase`."""
        out = np.zeros((G, G), dtype=np.uint64)
        _check(lib.sparbit_plan_partition(self._h, G, mapping, phase,
                                          out.ctypes.data_as(ctypes.POINTER(_u64))), "sparbit_plan_partition")
        return out

    def partition_messages(self, G: int, mapping: int, phase: int, src_device: int, dst_device: int) -> np.ndarray:
        n = _sz()
        _check(lib.sparbit_plan_partition_messages(self._h, G, mapping, phase, src_device, dst_device, None, 0,
                                                   ctypes.byref(n)), "sparbit_plan_partition_messages")
        out = np.zeros(n.value, dtype=MSG_DTYPE)
        if n.value:
            _check(lib.sparbit_plan_partition_messages(self._h, G, mapping, phase, src_device, dst_device,
                                                       out.ctypes.data, n.value, ctypes.byref(n)),
                   "sparbit_plan_partition_messages")
        return out

    # -- one communicator on G devices
    def allgather_multi_phases(self, G: int, mapping: int, device: int, send_local, recv_bases, first: int,
                               last: int, stream=None) -> None:
        """This device's share of phases first..last (no cross-device barrier is issued)."""
        bases = (_vp * G)(*[_ptr(b) for b in recv_bases])
        _check(lib.sparbit_allgather_multi_phases(self._h, G, mapping, device, _ptr(send_local), bases,
                                                  _stream_handle(stream), first, last),
               "sparbit_allgather_multi_phases")

    def allgather_multi(self, G: int, mapping: int, device: int, send_local, recv_bases, barrier,
                        stream=None) -> None:
        """The whole collective for this device; `barrier(stream_handle)` is the cross-device
        barrier (returns None/0 on success), called K + 1 times by the library."""
        bases = (_vp * G)(*[_ptr(b) for b in recv_bases])
        failure = []

        def _cb(_ctx, stream_handle):
            try:
                return int(barrier(stream_handle) or 0)
            except BaseException as e:  # an exception must not unwind through the C frames
                failure.append(e)
                return 1

        cb = BARRIER_FN(_cb) if barrier is not None else None
        code = lib.sparbit_allgather_multi(self._h, G, mapping, device, _ptr(send_local), bases,
                                           _stream_handle(stream), ctypes.cast(cb, _vp) if cb else None, None)
        if failure:
            raise failure[0]
        _check(code, "sparbit_allgather_multi")

    def validate(self) -> None:
        """Host-side race and bounds check of the descriptors (raises with the offending phase)."""
        bad = ctypes.c_int()
        code = lib.sparbit_plan_validate(self._h, ctypes.byref(bad))
        if code != OK:
            raise SparbitError(code, f"sparbit_plan_validate (phase {bad.value})")

    def validate_flow(self, vector_bytes: int = 16, resident_warps: int = 4736) -> int:
        """Host-side check of the flow executor's units and counters; returns the library's code
        (OK, or ERR_UNSUPPORTED when the plan cannot run on that executor) and raises on a fault."""
        bad, first = ctypes.c_int(), ctypes.c_int()
        code = lib.sparbit_plan_validate_flow(self._h, vector_bytes, resident_warps, ctypes.byref(first),
                                              ctypes.byref(bad))
        if code not in (OK, ERR_UNSUPPORTED):
            raise SparbitError(code, f"sparbit_plan_validate_flow (pass {bad.value})")
        self.first_flow_pass = first.value
        return code

    @property
    def workspace_bytes(self) -> int:
        return lib.sparbit_plan_workspace_bytes(self._h)

    def set_workspace(self, dev, nbytes: int) -> None:
        _check(lib.sparbit_plan_set_workspace(self._h, _ptr(dev), nbytes), "sparbit_plan_set_workspace")
        self._workspace = dev  # keep the owner alive

    def set_tunable(self, key: int, value: int) -> None:
        _check(lib.sparbit_plan_set_tunable(self._h, key, value), "sparbit_plan_set_tunable")

    def get_tunable(self, key: int) -> int:
        v = _u64()
        _check(lib.sparbit_plan_get_tunable(self._h, key, ctypes.byref(v)), "sparbit_plan_get_tunable")
        return int(v.value)

    def set_copy_path(self, path: int) -> None:
        _check(lib.sparbit_plan_set_copy_path(self._h, path), "sparbit_plan_set_copy_path")

    @property
    def exec_mode(self) -> int:
        return lib.sparbit_plan_exec_mode(self._h)

    @property
    def copy_path(self) -> int:
        return lib.sparbit_plan_copy_path(self._h)

    def launch_counts(self):
        k, g = _u64(), _u64()
        _check(lib.sparbit_plan_launch_counts(self._h, ctypes.byref(k), ctypes.byref(g)),
               "sparbit_plan_launch_counts")
        return k.value, g.value

    def status(self) -> int:
        """Synchronises; returns OK or ERR_TIMEOUT (raises on CUDA errors)."""
        raw = ctypes.c_int()
        code = lib.sparbit_plan_status(self._h, ctypes.byref(raw))
        if code not in (OK, ERR_TIMEOUT):
            raise SparbitError(code, "sparbit_plan_status")
        return code

    def set_trace(self, on: bool) -> None:
        _check(lib.sparbit_plan_set_trace(self._h, int(bool(on))), "sparbit_plan_set_trace")

    def get_trace(self) -> np.ndarray:
        """Time stamps (ns) of the last persistent launch: kernel start, then the end of every pass."""
        n = _sz()
        _check(lib.sparbit_plan_get_trace(self._h, None, 0, ctypes.byref(n)), "sparbit_plan_get_trace")
        out = np.zeros(n.value, dtype=np.uint64)
        if n.value:
            _check(lib.sparbit_plan_get_trace(self._h, out.ctypes.data_as(ctypes.POINTER(_u64)), n.value,
                                              ctypes.byref(n)), "sparbit_plan_get_trace")
        return out

    def set_mbarrier_test(self, extra_tx_bytes: int, timeout_ns: int) -> None:
        _check(lib.sparbit_plan_set_mbarrier_test(self._h, extra_tx_bytes, timeout_ns),
               "sparbit_plan_set_mbarrier_test")

    def set_barrier_test(self, extra_arrivals: int, timeout_ns: int) -> None:
        _check(lib.sparbit_plan_set_barrier_test(self._h, extra_arrivals, timeout_ns),
               "sparbit_plan_set_barrier_test")

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            _check(lib.sparbit_plan_destroy(h), "sparbit_plan_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def multi_rank_count(P: int, G: int, mapping: int, device: int) -> int:
    return lib.sparbit_multi_rank_count(P, G, mapping, device)


def multi_local_index(P: int, G: int, mapping: int, rank: int) -> int:
    return lib.sparbit_multi_local_index(P, G, mapping, rank)


def ipc_export(dev_ptr) -> tuple[bytes, int]:
    """(64-byte handle, offset) of the device allocation that contains dev_ptr."""
    h = ctypes.create_string_buffer(IPC_HANDLE_BYTES)
    off = _u64()
    _check(lib.sparbit_ipc_export(_ptr(dev_ptr), h, ctypes.byref(off)), "sparbit_ipc_export")
    return h.raw, int(off.value)


def ipc_open(handle: bytes, offset: int) -> tuple[int, int]:
    """(device address of the exported location, mapping base for ipc_close)."""
    ptr, base = _vp(), _vp()
    _check(lib.sparbit_ipc_open(handle, offset, ctypes.byref(ptr), ctypes.byref(base)), "sparbit_ipc_open")
    return int(ptr.value), int(base.value)


def ipc_close(mapping_base: int) -> None:
    _check(lib.sparbit_ipc_close(mapping_base), "sparbit_ipc_close")


def sparbit_plan(P: int, block_bytes: int) -> Plan:
    """The short form of the C ABI: a Sparbit plan with automatic executor choice."""
    return Plan(P, block_bytes, ALGO_SPARBIT, EXEC_AUTO)


def sparbit_allgather(plan: Plan, sendbuf, recvbuf, stream=None) -> None:
    plan.allgather(sendbuf, recvbuf, stream)


def sparbit_allgather_noalloc(P: int, block_bytes: int, sendbuf, recvbuf, stream=None,
                              algo: int = ALGO_SPARBIT) -> None:
    """The collective without any device allocation by the library (fixed 2 KiB scratch that is
    part of the library image).  For callers whose device memory is managed elsewhere and who
    must not trigger cudaMalloc.  Waits for completion.  Calls on one device must not overlap."""
    _check(lib.sparbit_allgather_noalloc(P, block_bytes, algo, _ptr(sendbuf), _ptr(recvbuf),
                                         _stream_handle(stream)), "sparbit_allgather_noalloc")
