"""One communicator on G devices (Section III-C): the executing half of the partitioner.

CPU tests: the placement helpers and the argument checks (nothing is launched).
GPU tests: G devices emulated on ONE GPU - each "device" is a separate allocation, its kernels
store into the others' allocations through the pointer table exactly as they would through peer
pointers.  The kernels never wait on one another, so the emulation is a faithful run of the same
code: stream order (one stream) or a host barrier between steps (one stream per device, one
thread per device) stands in for the cross-device barrier.  Every device's receive buffers are
compared with the CPU oracle, whole state, sentinel bytes included.
"""
import ctypes
import subprocess
import sys
import threading
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
import paper_2109_08751_b200 as sp
import seeded_inputs as si

ROOT = Path(__file__).resolve().parent.parent
MAPPINGS = (sp.MAP_SEQUENTIAL, sp.MAP_CYCLIC)


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    return torch.device("cuda:0")


def ranks_of(P, G, mapping, g):
    return [r for r in range(P) if sp.binding.lib.sparbit_rank_device(P, G, mapping, r) == g]


# ------------------------------------------------------------------------------------------ CPU
def test_placement_helpers_agree_with_rank_device():
    for P in list(range(1, 40)) + [61, 64, 100, 256, 1000]:
        for G in (1, 2, 3, 4, 5, 7, 8, 16):
            for mapping in MAPPINGS:
                seen = [0] * G
                for r in range(P):
                    g = sp.binding.lib.sparbit_rank_device(P, G, mapping, r)
                    assert sp.multi_local_index(P, G, mapping, r) == seen[g]
                    seen[g] += 1
                assert seen == [sp.multi_rank_count(P, G, mapping, g) for g in range(G)]
                assert sum(seen) == P
    assert sp.multi_rank_count(8, 4, 2, 0) == -1 and sp.multi_rank_count(8, 4, 0, 4) == -1
    assert sp.multi_local_index(8, 4, 0, 8) == -1


def test_argument_errors_are_found_before_any_launch():
    plan = sp.Plan(8, 64)
    bases = [4096 * (g + 1) for g in range(4)]
    lib, h = sp.binding.lib, plan._h
    arr = (ctypes.c_void_p * 4)(*bases)

    def phases(G, mapping, device, send, first, last, plan_h=h):
        return lib.sparbit_allgather_multi_phases(plan_h, G, mapping, device, send, arr, None, first, last)

    assert phases(0, 0, 0, 4096, -1, 2) == sp.ERR_ARG
    assert phases(17, 0, 0, 4096, -1, 2) == sp.ERR_ARG
    assert phases(4, 2, 0, 4096, -1, 2) == sp.ERR_ARG
    assert phases(4, 0, 4, 4096, -1, 2) == sp.ERR_ARG
    assert phases(4, 0, 0, None, -1, 2) == sp.ERR_ARG
    assert phases(4, 0, 0, 4096, -2, 2) == sp.ERR_ARG
    assert phases(4, 0, 0, 4096, 0, 3) == sp.ERR_ARG
    assert phases(4, 0, 0, 4096, 2, 1) == sp.ERR_ARG
    assert phases(4, 0, 0, 4096, -1, 2, plan_h=None) == sp.ERR_ARG
    arr[2] = None
    assert phases(4, 0, 0, 4096, -1, 2) == sp.ERR_ARG
    arr[2] = bases[2]
    # a missing barrier is an error as soon as there is a second device
    assert lib.sparbit_allgather_multi(h, 2, 0, 0, 4096, arr, None, None, None) == sp.ERR_ARG
    bruck = sp.Plan(8, 64, sp.ALGO_BRUCK)
    assert phases(4, 0, 0, 4096, -1, 2, plan_h=bruck._h) == sp.ERR_UNSUPPORTED
    var = sp.Plan.create_v([16, 0, 32, 48])
    assert phases(2, 0, 0, 4096, -1, 1, plan_h=var._h) == sp.ERR_UNSUPPORTED
    # blocks of zero bytes: valid, nothing to do, nothing launched (no GPU needed)
    empty = sp.Plan(8, 0)
    assert phases(4, 0, 0, None, -1, 2, plan_h=empty._h) == sp.OK
    assert b"barrier" in lib.sparbit_strerror(sp.ERR_BARRIER)


# ------------------------------------------------------------------------------------------ GPU
class Emulated:
    """G devices as G pairs of allocations on one GPU, with guard bands around the receive buffers."""

    GUARD = 4096

    def __init__(self, dev, P, m, G, mapping, seed, misalign=0):
        self.P, self.m, self.G, self.mapping = P, m, G, mapping
        self.host_send = si.send_blocks(P, m, seed)  # [P][m]
        self.ranks = [ranks_of(P, G, mapping, g) for g in range(G)]
        self.send, self.raw, self.recv = [], [], []
        for g in range(G):
            n = len(self.ranks[g])
            s = torch.empty(n * m + misalign, dtype=torch.uint8, device=dev)[misalign:]
            if n:
                s.copy_(torch.from_numpy(np.ascontiguousarray(self.host_send[self.ranks[g]]).reshape(-1)))
            raw = torch.full((n * P * m + 2 * self.GUARD + misalign,), si.SENTINEL, dtype=torch.uint8, device=dev)
            self.send.append(s)
            self.raw.append(raw)
            self.recv.append(raw[self.GUARD + misalign: self.GUARD + misalign + n * P * m])
        self.bases = [r.data_ptr() for r in self.recv]

    def check(self, want, what=""):
        """want: the oracle's receive space, flat [P][P][m]; guard bands must be untouched."""
        want = want.reshape(self.P, self.P * self.m)
        for g in range(self.G):
            got = self.recv[g].cpu().numpy().reshape(len(self.ranks[g]), self.P * self.m)
            for li, r in enumerate(self.ranks[g]):
                assert np.array_equal(got[li], want[r]), (what, "device", g, "rank", r)
            raw = self.raw[g].cpu().numpy()
            n = self.recv[g].numel()
            lo = self.recv[g].data_ptr() - self.raw[g].data_ptr()
            assert (raw[:lo] == si.SENTINEL).all() and (raw[lo + n:] == si.SENTINEL).all(), (what, "guard", g)


CASES = [
    (sp.ALGO_SPARBIT, 8, 64), (sp.ALGO_SPARBIT, 13, 272), (sp.ALGO_SPARBIT, 6, 4096), (sp.ALGO_SPARBIT, 21, 24),
    (sp.ALGO_SPARBIT, 61, 1040), (sp.ALGO_SPARBIT, 5, 3), (sp.ALGO_RING, 6, 272), (sp.ALGO_RECURSIVE_DOUBLING, 16, 272),
    (sp.ALGO_NEIGHBOR_EXCHANGE, 10, 272),
]


@pytest.mark.gpu
@pytest.mark.parametrize("mapping", MAPPINGS)
@pytest.mark.parametrize("G", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("algo,P,m", CASES)
def test_state_after_every_phase_on_emulated_devices(dev, algo, P, m, G, mapping):
    plan = sp.Plan(P, m, algo)
    ref = oracle.Plan(algo, P)
    em = Emulated(dev, P, m, G, mapping, seed=90 + P)
    want = si.sentinel_buffer(P * P * m)
    for ph in range(-1, ref.last_phase + 1):
        for g in range(G):  # one stream: every device's phase ph is complete before phase ph + 1 starts
            plan.allgather_multi_phases(G, mapping, g, em.send[g], em.bases, ph, ph)
        torch.cuda.synchronize()
        ref.run(m, em.host_send.reshape(-1), want, None, first=ph, last=ph)
        em.check(want, f"phase {ph}")


@pytest.mark.gpu
@pytest.mark.parametrize("mapping", MAPPINGS)
@pytest.mark.parametrize("misalign", [0, 1, 2, 4, 8])
def test_fused_first_pass_and_misaligned_buffers(dev, mapping, misalign):
    """Phases -1 and 0 in one call run as one pass; odd addresses pick narrower vectors."""
    P, m, G = 13, 1040 + (misalign % 8), 3
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT)
    em = Emulated(dev, P, m, G, mapping, seed=7, misalign=misalign)
    for g in range(G):
        plan.allgather_multi_phases(G, mapping, g, em.send[g], em.bases, -1, 0)
    torch.cuda.synchronize()
    want, _ = oracle.allgather(sp.ALGO_SPARBIT, P, m, em.host_send, last=0)
    em.check(want.reshape(-1), "after the fused pass")
    for ph in range(1, plan.last_phase + 1):
        for g in range(G):
            plan.allgather_multi_phases(G, mapping, g, em.send[g], em.bases, ph, ph)
    torch.cuda.synchronize()
    want, _ = oracle.allgather(sp.ALGO_SPARBIT, P, m, em.host_send)
    em.check(want.reshape(-1), "final")


@pytest.mark.gpu
@pytest.mark.parametrize("mapping", MAPPINGS)
@pytest.mark.parametrize("algo,P,m,G", [(sp.ALGO_SPARBIT, 256, 4096, 4), (sp.ALGO_SPARBIT, 1000, 64, 8),
                                        (sp.ALGO_SPARBIT, 100, 16384, 3), (sp.ALGO_RECURSIVE_DOUBLING, 64, 8192, 2)])
def test_larger_collectives_several_tiles_and_a_ragged_tail(dev, algo, P, m, G, mapping):
    plan = sp.Plan(P, m, algo)
    em = Emulated(dev, P, m, G, mapping, seed=11)
    for ph in range(-1, plan.last_phase + 1):
        for g in range(G):
            plan.allgather_multi_phases(G, mapping, g, em.send[g], em.bases, ph, ph)
    torch.cuda.synchronize()
    want, _ = oracle.allgather(algo, P, m, em.host_send, threads=8)
    em.check(want.reshape(-1))


def random_cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        algo = int(rng.choice([sp.ALGO_SPARBIT] * 3 + [sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING,
                                                       sp.ALGO_NEIGHBOR_EXCHANGE]))
        P = int(rng.integers(1, 97))
        if algo == sp.ALGO_RECURSIVE_DOUBLING:
            P = 1 << int(rng.integers(0, 7))
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE:
            P += P & 1
        if algo == sp.ALGO_RING and P > 24:
            P = int(rng.integers(1, 25))
        m = int(rng.choice([1, 3, 8, 24, 64, 100, 272, 1040, 4096, 5000, 16400]))
        G = int(rng.integers(1, 17))  # more devices than ranks happens: some devices hold nothing
        out.append((algo, P, m, G, int(rng.integers(0, 2)), int(rng.choice([0, 0, 1, 2, 4, 8]))))
    return out


@pytest.mark.gpu
@pytest.mark.parametrize("case", random_cases(80, 20211), ids=lambda c: "-".join(map(str, c)))
def test_random_cases_on_emulated_devices(dev, case):
    algo, P, m, G, mapping, misalign = case
    plan = sp.Plan(P, m, algo)
    em = Emulated(dev, P, m, G, mapping, seed=P + m, misalign=misalign)
    assert [len(r) for r in em.ranks] == [sp.multi_rank_count(P, G, mapping, g) for g in range(G)]
    for g in range(G):
        plan.allgather_multi_phases(G, mapping, g, em.send[g], em.bases, -1, min(0, plan.last_phase))
    for ph in range(1, plan.last_phase + 1):
        for g in range(G):
            plan.allgather_multi_phases(G, mapping, g, em.send[g], em.bases, ph, ph)
    torch.cuda.synchronize()
    want, _ = oracle.allgather(algo, P, m, em.host_send)
    em.check(want.reshape(-1))


@pytest.mark.gpu
@pytest.mark.parametrize("mapping", MAPPINGS)
@pytest.mark.parametrize("P,m,G", [(13, 272, 3), (32, 4096, 4), (8, 64, 8)])
def test_whole_collective_with_the_callers_barrier(dev, P, m, G, mapping):
    """sparbit_allgather_multi, one host thread and one stream per device; the barrier is a stream
    synchronise followed by a host barrier.  It is called once on entry and once after every step."""
    plan = sp.Plan(P, m)
    em = Emulated(dev, P, m, G, mapping, seed=5)
    gate = threading.Barrier(G)
    calls, errors = [0] * G, []

    def device(g):
        try:
            torch.cuda.set_device(dev)
            stream = torch.cuda.Stream(device=dev)

            def barrier(_handle):
                calls[g] += 1
                stream.synchronize()
                gate.wait(timeout=60)

            plan.allgather_multi(G, mapping, g, em.send[g], em.bases, barrier, stream)
            stream.synchronize()
        except BaseException as e:  # noqa: BLE001
            errors.append(e)
            gate.abort()

    torch.cuda.synchronize()
    threads = [threading.Thread(target=device, args=(g,)) for g in range(G)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(120)
    assert not errors, errors
    assert calls == [plan.num_steps + 1] * G
    want, _ = oracle.allgather(sp.ALGO_SPARBIT, P, m, em.host_send)
    em.check(want.reshape(-1))


@pytest.mark.gpu
def test_a_failing_barrier_is_reported(dev):
    plan = sp.Plan(8, 64)
    em = Emulated(dev, 8, 64, 2, sp.MAP_SEQUENTIAL, seed=3)
    with pytest.raises(sp.SparbitError) as e:
        plan.allgather_multi(2, sp.MAP_SEQUENTIAL, 0, em.send[0], em.bases, lambda _h: 1)
    assert e.value.code == sp.ERR_BARRIER
    with pytest.raises(ZeroDivisionError):
        plan.allgather_multi(2, sp.MAP_SEQUENTIAL, 0, em.send[0], em.bases, lambda _h: 1 // 0)
    torch.cuda.synchronize()


@pytest.mark.gpu
@pytest.mark.parametrize("mapping", ["sequential", "cyclic"])
def test_two_processes_share_their_buffers_through_ipc_handles(mapping):
    """One process per device, as on a multi-GPU node, here both on GPU 0: each exports its receive
    buffers (sparbit_ipc_export), opens the other's (sparbit_ipc_open) and runs
    sparbit_allgather_multi with a gloo barrier.  Each checks its ranks against the oracle."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(__import__("os").environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(ROOT / "tests" / "multi_device_worker.py"), mapping],
                                      env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        outs.append(out)
    for p, out in zip(procs, outs):
        assert p.returncode == 0, out
        assert "multi-device worker ok" in out, out
