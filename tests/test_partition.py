"""Placement of the ranks on several devices (Section III-C: sequential and cyclic mappings).

The library only describes the split of every phase into device-local copies and blocks that
cross to another device; these tests check that description on CPU: against the oracle's message
sets, against the counts that follow from the mapping by hand, and by executing it as a
world_size-2 gloo job on host buffers, which must reproduce the oracle's final state.
"""
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

import oracle
import paper_2109_08751_b200 as sp

ROOT = Path(__file__).resolve().parent.parent
KEYS = ("src_rank", "dst_rank", "src_space", "src_slot", "dst_space", "dst_slot")


def as_set(msgs):
    return set(zip(*(msgs[k].tolist() for k in KEYS)))


def device_of(P, G, mapping, r):
    """The mappings restated: contiguous ranges whose sizes differ by at most one, or round robin."""
    if mapping == sp.MAP_CYCLIC:
        return r % G
    bounds = [g * P // G for g in range(G + 1)]
    return next(g for g in range(G) if bounds[g] <= r < bounds[g + 1])


@pytest.mark.parametrize("mapping", [sp.MAP_SEQUENTIAL, sp.MAP_CYCLIC])
def test_rank_device_is_the_stated_mapping(mapping):
    for P in (1, 2, 5, 8, 13, 64, 100):
        for G in (1, 2, 3, 4, 8):
            got = [sp.binding.lib.sparbit_rank_device(P, G, mapping, r) for r in range(P)]
            assert got == [device_of(P, G, mapping, r) for r in range(P)], (P, G)
            sizes = np.bincount(got, minlength=G)
            assert sizes.max() - sizes.min() <= 1
    assert sp.binding.lib.sparbit_rank_device(8, 2, mapping, 8) == -1
    assert sp.binding.lib.sparbit_rank_device(8, 0, mapping, 0) == -1


@pytest.mark.parametrize("algo", [sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK,
                                  sp.ALGO_NEIGHBOR_EXCHANGE])
@pytest.mark.parametrize("mapping", [sp.MAP_SEQUENTIAL, sp.MAP_CYCLIC])
def test_partition_covers_the_oracle_message_set_exactly_once(algo, mapping):
    for P in (4, 6, 8, 13, 16, 21, 32):
        if algo == sp.ALGO_RECURSIVE_DOUBLING and P & (P - 1):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        ref = oracle.Plan(algo, P)
        plan = sp.Plan(P, 16, algo)
        for G in (1, 2, 3, 4):
            for ph in range(-1, plan.last_phase + 1):
                want = as_set(ref.phase_messages(ph))
                counts = plan.partition(G, mapping, ph)
                seen = set()
                for s in range(G):
                    for d in range(G):
                        part = plan.partition_messages(G, mapping, ph, s, d)
                        assert len(part) == counts[s, d]
                        assert all(device_of(P, G, mapping, int(x)) == s for x in part["src_rank"])
                        assert all(device_of(P, G, mapping, int(x)) == d for x in part["dst_rank"])
                        ps = as_set(part)
                        assert len(ps) == len(part) and not (ps & seen)
                        seen |= ps
                assert seen == want, (algo, P, G, ph)
        plan.destroy()


def test_sparbit_cross_device_blocks_follow_from_the_distance():
    """P = 256 on 8 devices.  Sequential (32 consecutive ranks per device): a step at distance
    d sends min(d, 32) of every 32 senders' traffic off the device.  Cyclic: a step stays local
    exactly when its distance is a multiple of 8.  Section III-C's argument in numbers: the
    late, heavy steps of Sparbit are local under the sequential mapping."""
    P, G = 256, 8
    plan = sp.Plan(P, 1)
    for step in range(plan.num_steps):
        d, n, _ = plan.step_info(step)
        seq = plan.partition(G, sp.MAP_SEQUENTIAL, step)
        cyc = plan.partition(G, sp.MAP_CYCLIC, step)
        assert int(seq.sum()) == int(cyc.sum()) == P * n
        assert int(seq.sum() - np.trace(seq)) == G * min(d, 32) * n
        assert int(cyc.sum() - np.trace(cyc)) == (0 if d % G == 0 else P * n)
        if d < 32:   # only the next device is ever reached
            for s in range(G):
                assert seq[s, (s + 1) % G] == d * n and seq[s, s] == (32 - d) * n
    total = P * (P - 1)
    cross_seq = sum(int(plan.partition(G, sp.MAP_SEQUENTIAL, s).sum() - np.trace(plan.partition(G, sp.MAP_SEQUENTIAL, s)))
                    for s in range(plan.num_steps))
    cross_cyc = sum(int(plan.partition(G, sp.MAP_CYCLIC, s).sum() - np.trace(plan.partition(G, sp.MAP_CYCLIC, s)))
                    for s in range(plan.num_steps))
    assert (cross_seq, cross_cyc) == (6912, 57344) and total == 65280
    plan.destroy()


def test_partition_argument_errors():
    plan = sp.Plan(8, 16)
    lib = sp.binding.lib
    buf = np.zeros(4, dtype=np.uint64)
    assert lib.sparbit_plan_partition(plan._h, 2, 7, 0, buf.ctypes.data_as(
        __import__("ctypes").POINTER(__import__("ctypes").c_uint64))) == sp.ERR_ARG
    with pytest.raises(sp.binding.SparbitError):
        plan.partition(2, sp.MAP_CYCLIC, 5)
    with pytest.raises(sp.binding.SparbitError):
        plan.partition_messages(2, sp.MAP_CYCLIC, 0, 2, 0)
    plan.destroy()


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("mapping", ["sequential", "cyclic"])
def test_two_devices_execute_the_partition_over_gloo(mapping):
    """Two processes stand in for two devices: each holds its ranks' receive buffers in host
    memory, runs its local copy lists and exchanges the crossing blocks through gloo, phase by
    phase; rank 0 compares the gathered result with the oracle's final state."""
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(ROOT / "tests" / "partition_worker.py"), mapping],
                                      env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    assert outs[0][0].startswith("ok ")
