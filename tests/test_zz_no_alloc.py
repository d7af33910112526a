"""The entry point that allocates no device memory, against the regular one.

`sparbit_allgather_noalloc` serves callers that cannot call cudaMalloc (device memory owned by
their own pool or framework, plug-ins that only get buffers and a stream): its scratch is a fixed
2 KiB array inside the library image instead of a per-plan allocation.  It must produce exactly
what `sparbit_allgather` produces.  Because every call shares that one array and it keeps the
previous call's contents, the check is made on two calls in a row with different sizes and data.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.  It passes alone in a fresh process as well as after the others.
"""
import ctypes

import numpy as np
import pytest

import oracle
import seeded_inputs as si
import paper_2109_08751_b200 as sp
from paper_2109_08751_b200 import binding

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def regular(P, m, algo, send, dev):
    """Result of the existing entry point with the same executor and copy engine."""
    plan = sp.Plan(P, m, algo, sp.EXEC_PERSISTENT)
    plan.set_copy_path(sp.COPY_VECTOR)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    plan.destroy()
    return recv


def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    # two different collectives back to back: the second finds the first one's descriptors and
    # barrier words in the shared scratch and must not be disturbed by them
    cases = [(13, 4096, sp.ALGO_SPARBIT, 11), (64, 1040, sp.ALGO_SPARBIT, 12),
             (16, 272, sp.ALGO_RECURSIVE_DOUBLING, 13), (9, 100, sp.ALGO_RING, 14),
             (10, 48, sp.ALGO_NEIGHBOR_EXCHANGE, 15)]
    stream = torch.cuda.Stream(device=dev)
    for P, m, algo, seed in cases:
        for call in range(2):
            host_send = si.send_blocks(P, m, seed + 100 * call)
            send = torch.from_numpy(host_send.reshape(-1)).to(dev)
            got = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
            torch.cuda.synchronize(dev)
            binding.sparbit_allgather_noalloc(P, m, send, got, stream, algo=algo)
            want = regular(P, m, algo, send, dev)
            assert torch.equal(got, want), (P, m, algo, call)          # bit-exact, as everywhere
            # and both are what the CPU oracle computes, over the whole receive space
            ref, _ = oracle.allgather(algo, P, m, host_send)
            assert np.array_equal(got.cpu().numpy(), ref.reshape(-1)), (P, m, algo, call)


def test_noalloc_leaves_the_amount_of_free_device_memory_alone():
    """The point of the entry point: after the first call on the device (module load, address
    look-up) later calls of any size, algorithm and alignment must not change what the driver
    reports as free device memory, i.e. nothing is allocated behind the caller's back."""
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    # all buffers first, so that torch's own allocator is quiet during the measured calls
    cases = [(8, 64, sp.ALGO_SPARBIT), (21, 5000, sp.ALGO_SPARBIT), (32, 16384, sp.ALGO_RECURSIVE_DOUBLING),
             (12, 3, sp.ALGO_RING), (30, 2048, sp.ALGO_NEIGHBOR_EXCHANGE), (200, 1024, sp.ALGO_SPARBIT)]
    bufs = []
    for P, m, algo in cases:
        host_send = si.send_blocks(P, m, 3 + P)
        bufs.append((host_send, torch.from_numpy(host_send.reshape(-1)).to(dev),
                     torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)))
    stream = torch.cuda.Stream(device=dev)
    binding.sparbit_allgather_noalloc(cases[0][0], cases[0][1], bufs[0][1], bufs[0][2], stream, algo=cases[0][2])
    torch.cuda.synchronize(dev)
    for attempt in range(2):   # the figure is device-wide: one repeat, should anything else have moved it
        free_before = torch.cuda.mem_get_info(dev)[0]
        changed = []
        for (P, m, algo), (host_send, send, recv) in zip(cases, bufs):
            binding.sparbit_allgather_noalloc(P, m, send, recv, stream, algo=algo)
            if torch.cuda.mem_get_info(dev)[0] != free_before:
                changed.append((P, m, algo))
        if not changed:
            break
    assert not changed, changed
    for (P, m, algo), (host_send, send, recv) in zip(cases, bufs):
        ref, _ = oracle.allgather(algo, P, m, host_send)
        assert np.array_equal(recv.cpu().numpy(), ref.reshape(-1)), (P, m, algo)


def test_noalloc_refuses_what_does_not_fit_its_scratch():
    lib = binding.lib
    # host-side checks: nothing is enqueued, the pointers are never touched
    assert lib.sparbit_allgather_noalloc(64, 16, sp.ALGO_RING, 4096, 1 << 20, None) == sp.ERR_LIMIT
    assert lib.sparbit_allgather_noalloc(8, 16, sp.ALGO_BRUCK, 4096, 1 << 20, None) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_allgather_noalloc(58, 16, sp.ALGO_NEIGHBOR_EXCHANGE, 4096, 1 << 20, None) == sp.ERR_LIMIT
    assert lib.sparbit_allgather_noalloc(7, 16, sp.ALGO_NEIGHBOR_EXCHANGE, 4096, 1 << 20, None) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_allgather_noalloc(8, 16, 5, 4096, 1 << 20, None) == sp.ERR_ARG
    assert lib.sparbit_allgather_noalloc(6, 16, sp.ALGO_RECURSIVE_DOUBLING, 4096, 1 << 20, None) \
        == sp.ERR_UNSUPPORTED
    assert lib.sparbit_allgather_noalloc(0, 16, sp.ALGO_SPARBIT, 4096, 1 << 20, None) == sp.ERR_ARG
    assert lib.sparbit_allgather_noalloc(8, 16, sp.ALGO_SPARBIT, 4096, 4100, None) == sp.ERR_ALIAS
    assert lib.sparbit_allgather_noalloc(8, 0, sp.ALGO_SPARBIT, None, None, None) == sp.OK
    assert "limit" in lib.sparbit_strerror(sp.ERR_LIMIT).decode()


def test_noalloc_refuses_a_capturing_stream_and_leaves_the_capture_intact():
    """The entry point waits for its stream, which a stream under capture does not allow: the call
    must say so before it enqueues anything, and the caller's capture must go on undisturbed."""
    dev = torch.device("cuda", 0)
    P, m = 8, 256
    send = torch.from_numpy(si.send_blocks(P, m, 9).reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    other = torch.zeros(1024, device=dev)
    stream = torch.cuda.Stream(device=dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        torch.cuda.synchronize()
        graph.capture_begin()
        other.add_(1.0)
        rc = binding.lib.sparbit_allgather_noalloc(P, m, sp.ALGO_SPARBIT, send.data_ptr(), recv.data_ptr(),
                                                   ctypes.c_void_p(stream.cuda_stream))
        other.add_(1.0)
        graph.capture_end()
    assert rc == sp.ERR_UNSUPPORTED
    graph.replay()
    torch.cuda.synchronize()
    assert float(other[0]) == 2.0                                   # the capture held both additions
    assert bool((recv == si.SENTINEL).all())                        # and nothing of the collective
    rc = binding.lib.sparbit_allgather_noalloc(P, m, sp.ALGO_SPARBIT, send.data_ptr(), recv.data_ptr(),
                                               ctypes.c_void_p(stream.cuda_stream))
    assert rc == sp.OK
    assert all(torch.equal(recv.view(P, P * m)[r], send) for r in range(P))
