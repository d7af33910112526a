"""Python face of the CPU oracle (allgather_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may import this
package.  The CUDA library and its Python binding never do, and this package never imports them.

The C file is compiled with gcc on first use (or by `build()`), into this folder.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "allgather_oracle.c"
_LIB = _HERE / "liballgather_oracle.so"

SPARBIT, RING, RECURSIVE_DOUBLING, BRUCK, NEIGHBOR_EXCHANGE = 0, 1, 2, 3, 4
ALGO_NAMES = {SPARBIT: "sparbit", RING: "ring", RECURSIVE_DOUBLING: "recursive_doubling", BRUCK: "bruck",
              NEIGHBOR_EXCHANGE: "neighbor_exchange"}
SPACE_SEND, SPACE_RECV, SPACE_SCRATCH = 0, 1, 2

MSG_DTYPE = np.dtype(
    [
        ("phase", "<i4"),
        ("src_rank", "<i4"),
        ("dst_rank", "<i4"),
        ("src_space", "<i4"),
        ("src_slot", "<i4"),
        ("dst_space", "<i4"),
        ("dst_slot", "<i4"),
    ]
)


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc if the shared object is missing or older than the source."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["gcc", "-O2", "-std=c11", "-D_GNU_SOURCE", "-Wall", "-Wextra", "-fPIC", "-shared",
               "-pthread", str(_SRC), "-o", str(tmp)]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        lib.oracle_last_error.restype = ctypes.c_char_p
        lib.oracle_plan_create.restype = ctypes.c_void_p
        lib.oracle_plan_create.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.oracle_plan_destroy.argtypes = [ctypes.c_void_p]
        lib.oracle_plan_num_steps.argtypes = [ctypes.c_void_p]
        lib.oracle_plan_has_rotation.argtypes = [ctypes.c_void_p]
        lib.oracle_plan_num_messages.restype = ctypes.c_size_t
        lib.oracle_plan_num_messages.argtypes = [ctypes.c_void_p]
        lib.oracle_plan_messages.restype = ctypes.c_void_p
        lib.oracle_plan_messages.argtypes = [ctypes.c_void_p]
        lib.oracle_run.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        lib.oracle_run_v.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_int, ctypes.c_int, ctypes.c_int]
        _lib = lib
    return _lib


class OracleError(RuntimeError):
    pass


class Plan:
    """Explicit message lists of one algorithm for P ranks, matched and checked."""

    def __init__(self, algo: int, P: int):
        lib = _load()
        self._h = lib.oracle_plan_create(int(algo), int(P))
        if not self._h:
            raise OracleError(lib.oracle_last_error().decode())
        self.algo, self.P = int(algo), int(P)
        self.num_steps = lib.oracle_plan_num_steps(self._h)
        self.has_rotation = bool(lib.oracle_plan_has_rotation(self._h))
        n = lib.oracle_plan_num_messages(self._h)
        ptr = lib.oracle_plan_messages(self._h)
        raw = (ctypes.c_char * (n * MSG_DTYPE.itemsize)).from_address(ptr)
        #: structured array of every message, ordered by phase (a copy; safe after destroy)
        self.messages = np.frombuffer(raw, dtype=MSG_DTYPE, count=n).copy()

    @property
    def last_phase(self) -> int:
        return self.num_steps if self.has_rotation else self.num_steps - 1

    def phase_messages(self, phase: int) -> np.ndarray:
        return self.messages[self.messages["phase"] == phase]

    def run(self, m: int, send: np.ndarray, recv: np.ndarray, scratch: np.ndarray | None = None,
            first: int = -1, last: int | None = None, threads: int = 1) -> None:
        """Apply phases first..last (inclusive) in place on host buffers (uint8, C-contiguous)."""
        P = self.P
        if last is None:
            last = self.last_phase
        for name, buf, need in (("send", send, P * m), ("recv", recv, P * P * m)):
            if buf.dtype != np.uint8 or not buf.flags.c_contiguous or buf.size != need:
                raise ValueError(f"{name} must be contiguous uint8 of {need} bytes")
        if not recv.flags.writeable:
            raise ValueError("recv must be writeable")
        sp = None
        if self.algo == BRUCK:
            if scratch is None or scratch.dtype != np.uint8 or scratch.size != P * P * m \
                    or not scratch.flags.c_contiguous or not scratch.flags.writeable:
                raise ValueError("Bruck needs a contiguous writeable uint8 scratch of P*P*m bytes")
            sp = scratch.ctypes.data
        lib = _load()
        rc = lib.oracle_run(self._h, m, send.ctypes.data, recv.ctypes.data, sp, first, last, threads)
        if rc:
            raise OracleError(lib.oracle_last_error().decode())

    def run_v(self, counts, send: np.ndarray, recv: np.ndarray, first: int = -1, last: int | None = None,
              threads: int = 1) -> None:
        """Allgatherv: blocks of counts[j] bytes, contiguous displacements (see oracle_run_v)."""
        P = self.P
        off = np.zeros(P + 1, dtype=np.uint64)
        off[1:] = np.cumsum(np.asarray(counts, dtype=np.uint64))
        T = int(off[P])
        if last is None:
            last = self.last_phase
        for name, buf, need in (("send", send, T), ("recv", recv, P * T)):
            if buf.dtype != np.uint8 or not buf.flags.c_contiguous or buf.size != need:
                raise ValueError(f"{name} must be contiguous uint8 of {need} bytes")
        lib = _load()
        rc = lib.oracle_run_v(self._h, off.ctypes.data, send.ctypes.data, recv.ctypes.data, first, last, threads)
        if rc:
            raise OracleError(lib.oracle_last_error().decode())

    def trace(self, rank: int, slot: int):
        """Follow the messages that fill receive slot `slot` of `rank` back to a send buffer.

        Returns the list of messages on the way, first hop first.  The first hop reads the send
        block of the rank whose data ends up in the slot, so a sampled output of a run too large
        to simulate in full is `send[trace(...)[0]["src_rank"]]`.
        """
        if not hasattr(self, "_by_dst"):
            m = self.messages
            key = (m["dst_space"].astype(np.int64) * self.P + m["dst_rank"]) * self.P + m["dst_slot"]
            self._by_dst = dict(zip(key.tolist(), range(len(m))))
        path = []
        space, r, s = SPACE_RECV, int(rank), int(slot)
        while space != SPACE_SEND:
            k = self._by_dst[(space * self.P + r) * self.P + s]
            msg = self.messages[k]
            path.append(msg)
            space, r, s = int(msg["src_space"]), int(msg["src_rank"]), int(msg["src_slot"])
        return path[::-1]

    def close(self) -> None:
        if getattr(self, "_h", None):
            _load().oracle_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def allgather(algo: int, P: int, m: int, send: np.ndarray, sentinel: int = 0xA5,
              first: int = -1, last: int | None = None, threads: int = 1):
    """Run the collective from sentinel-filled buffers; returns (recv, scratch-or-None).

    recv has shape (P, P*m): row r is rank r's receive buffer.
    """
    plan = Plan(algo, P)
    send = np.ascontiguousarray(send, dtype=np.uint8).reshape(-1)
    recv = np.full(P * P * m, sentinel, dtype=np.uint8)
    scratch = np.full(P * P * m, sentinel, dtype=np.uint8) if algo == BRUCK else None
    plan.run(m, send, recv, scratch, first, last, threads)
    plan.close()
    return recv.reshape(P, P * m), (None if scratch is None else scratch.reshape(P, P * m))
