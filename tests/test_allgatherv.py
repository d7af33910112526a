"""Blocks of different sizes (MPI_Allgatherv with contiguous displacements) on the same schedules.

CPU part: the oracle's variable-size run against the plain definition of the result (every
receive buffer is the concatenation of all send blocks, whatever their sizes), against the
fixed-size run when all sizes are equal, and the library's host-side checks.  GPU part: the CUDA
path against the oracle, bit for bit, including the state after every phase.
"""
import ctypes

import numpy as np
import pytest

import oracle
import seeded_inputs as si
import paper_2109_08751_b200 as sp
from paper_2109_08751_b200 import binding

V_ALGOS = [sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_NEIGHBOR_EXCHANGE]


def defined_for(algo, P):
    if algo == sp.ALGO_RECURSIVE_DOUBLING:
        return P & (P - 1) == 0
    if algo == sp.ALGO_NEIGHBOR_EXCHANGE:
        return P % 2 == 0
    return True


# ------------------------------------------------------------------------------------ CPU: oracle
@pytest.mark.parametrize("algo", V_ALGOS)
def test_oracle_v_final_state_is_the_concatenation(algo):
    for P in list(range(1, 34)) + [64]:
        if not defined_for(algo, P):
            continue
        for unit, scale in ((1, 9), (16, 4)):
            counts = si.block_counts(P, 100 + P, unit=unit, scale=scale)
            send = si.send_blocks_v(counts, 5)
            T = len(send)
            recv = si.sentinel_buffer(P * T)
            oracle.Plan(algo, P).run_v(counts, send, recv)
            assert np.array_equal(recv.reshape(P, T), np.broadcast_to(send, (P, T))), (algo, P)


def test_oracle_v_with_equal_sizes_is_the_fixed_size_run():
    P, m = 13, 24
    send = si.send_blocks(P, m, 5).reshape(-1)
    assert np.array_equal(si.send_blocks_v([m] * P, 5), send)
    for last in range(-1, 4):
        a = si.sentinel_buffer(P * P * m)
        oracle.Plan(oracle.SPARBIT, P).run_v([m] * P, send, a, last=last)
        b, _ = oracle.allgather(oracle.SPARBIT, P, m, send, last=last)
        assert np.array_equal(a, b.reshape(-1)), last


def test_oracle_v_partial_state_only_touches_delivered_blocks():
    """After phase k exactly the blocks the fixed-size schedule has delivered are filled."""
    P = 11
    counts = [3 + 2 * r for r in range(P)]
    off = np.concatenate([[0], np.cumsum(counts)])
    T = int(off[-1])
    send = si.send_blocks_v(counts, 9)
    ref = oracle.Plan(oracle.SPARBIT, P)
    for last in range(-1, ref.num_steps):
        recv = si.sentinel_buffer(P * T)
        ref.run_v(counts, send, recv, last=last)
        fixed, _ = oracle.allgather(oracle.SPARBIT, P, 4, si.send_blocks(P, 4, 1), last=last)
        for r in range(P):
            for b in range(P):
                got = recv[r * T + off[b]:r * T + off[b + 1]]
                delivered = not (fixed[r].reshape(P, 4)[b] == si.SENTINEL).all()
                if delivered:
                    assert np.array_equal(got, send[off[b]:off[b + 1]])
                else:
                    assert (got == si.SENTINEL).all()


def test_oracle_v_refuses_bruck():
    with pytest.raises(oracle.OracleError):
        oracle.Plan(oracle.BRUCK, 4).run_v([1, 2, 3, 4], si.send_blocks_v([1, 2, 3, 4], 1), si.sentinel_buffer(40))


# ------------------------------------------------------------------------------------ CPU: library host side
def test_create_v_errors_and_introspection():
    lib = binding.lib
    out = ctypes.c_void_p()
    counts = (ctypes.c_size_t * 4)(16, 0, 32, 48)
    assert lib.sparbit_plan_create_v(4, None, 0, 0, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create_v(0, counts, 0, 0, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create_v(4, counts, 0, 0, None) == sp.ERR_ARG
    assert lib.sparbit_plan_create_v(4, counts, sp.ALGO_BRUCK, 0, ctypes.byref(out)) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_plan_create_v(4, counts, 0, sp.EXEC_FLOW, ctypes.byref(out)) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_plan_create_v(4, counts, 0, sp.EXEC_MIRROR, ctypes.byref(out)) == sp.OK
    assert lib.sparbit_plan_destroy(out) == sp.OK
    assert lib.sparbit_plan_create_v(4, counts, 0, 9, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create_v(3, counts, sp.ALGO_RECURSIVE_DOUBLING, 0, ctypes.byref(out)) == sp.ERR_UNSUPPORTED
    many = (ctypes.c_size_t * 8193)(*([16] * 8193))
    assert lib.sparbit_plan_create_v(8193, many, 0, 0, ctypes.byref(out)) == sp.ERR_LIMIT
    big = (ctypes.c_size_t * 2)(1 << 61, 1 << 61)
    assert lib.sparbit_plan_create_v(2, big, 0, 0, ctypes.byref(out)) == sp.ERR_OVERFLOW
    plan = sp.Plan.create_v([16, 0, 32, 48, 8])
    ref = oracle.Plan(oracle.SPARBIT, 5)
    assert plan.num_steps == 3 and plan.workspace_bytes == 0
    for ph in range(-1, 3):   # the schedule is the fixed-size one, block for block
        got = {tuple(int(x) for x in m) for m in plan.messages(ph)}
        want = {tuple(int(x) for x in m) for m in ref.phase_messages(ph)}
        assert got == want
    # argument checks before any launch: send is 104 bytes, recv 5 * 104
    assert lib.sparbit_allgather(plan._h, 4096, 4096 + 100, None) == sp.ERR_ALIAS
    assert lib.sparbit_allgather(plan._h, None, 1 << 20, None) == sp.ERR_ARG
    empty = sp.Plan.create_v([0, 0, 0])
    assert lib.sparbit_allgather(empty._h, None, None, None) == sp.OK


# ------------------------------------------------------------------------------------ GPU
def _gpu():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    return torch, torch.device("cuda:0")


def run_v_case(P, counts, algo, exec_mode, seed, shift=0, iters=2, copy=sp.COPY_AUTO):
    torch, dev = _gpu()
    plan = sp.Plan.create_v(counts, algo, exec_mode)
    plan.set_copy_path(copy)
    ref = oracle.Plan(algo, P)
    T = sum(counts)
    G = si.GUARD_BYTES
    send_raw = torch.full((T + 2 * G + 64,), 0x3C, dtype=torch.uint8, device=dev)
    recv_raw = torch.full((P * T + 2 * G + 64,), si.SENTINEL, dtype=torch.uint8, device=dev)
    s0 = (-send_raw.data_ptr()) % 256 + G + shift
    r0 = (-recv_raw.data_ptr()) % 256 + G + shift
    send, recv = send_raw[s0:s0 + T], recv_raw[r0:r0 + P * T]
    for it in range(iters):
        host_send = si.send_blocks_v(counts, seed + it)
        send.copy_(torch.from_numpy(host_send))
        recv_raw.fill_(si.SENTINEL)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK
        want = si.sentinel_buffer(P * T)
        ref.run_v(counts, host_send, want)
        assert np.array_equal(recv.cpu().numpy(), want), (P, algo, exec_mode, it)
        assert bool((recv_raw[:r0] == si.SENTINEL).all()) and bool((recv_raw[r0 + P * T:] == si.SENTINEL).all())
    plan.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("algo", V_ALGOS)
@pytest.mark.parametrize("exec_mode", [sp.EXEC_AUTO, sp.EXEC_STREAM, sp.EXEC_PERSISTENT, sp.EXEC_MIRROR])
@pytest.mark.parametrize("copy", [sp.COPY_VECTOR, sp.COPY_BULK])
def test_gpu_v_parity_mixed_sizes(algo, exec_mode, copy):
    """Both copy engines and all four executors (the mirror executor where the receive buffers
    fit one SM's shared memory, the graph chain in its place where not).  Byte counts that are not multiples of 16 send
    a bulk request to the vector engine (the bulk engine moves 16-byte units), which is part of
    what is checked."""
    for P in (1, 2, 5, 6, 8, 13, 16, 32, 50, 64):
        if not defined_for(algo, P):
            continue
        for unit, scale in ((16, 40), (1, 30), (4, 300), (16, 1200)):
            run_v_case(P, si.block_counts(P, 40 + P + unit, unit=unit, scale=scale), algo, exec_mode, 77, iters=1,
                       copy=copy)


@pytest.mark.gpu
def test_gpu_v_mirror_is_used_where_it_fits():
    torch, dev = _gpu()
    for counts, want in (([64, 0, 200, 16, 48, 1000, 8, 24], sp.EXEC_MIRROR),         # 10.6 KiB in all
                         ([3000] * 8, sp.EXEC_MIRROR),                                 # 187.5 KiB: on request only
                         ([4000] * 8, sp.EXEC_GRAPH)):                                 # 250 KiB: fits no SM
        P, T = len(counts), sum(counts)
        plan = sp.Plan.create_v(counts, sp.ALGO_SPARBIT, sp.EXEC_MIRROR)
        host_send = si.send_blocks_v(counts, 5)
        send = torch.from_numpy(host_send).to(dev)
        recv = torch.full((P * T,), si.SENTINEL, dtype=torch.uint8, device=dev)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK and plan.exec_mode == want, counts
        assert all(torch.equal(recv.view(P, T)[r], send) for r in range(P))
        assert plan.launch_counts() == ((1, 0) if want == sp.EXEC_MIRROR else (3, 1))   # the mirror kernel is launched as itself
        plan.destroy()
    small = sp.Plan.create_v([64, 0, 200, 16, 48, 1000, 8, 24])
    assert small.exec_mode == sp.EXEC_MIRROR                  # what AUTO picks below 64 KiB
    big = sp.Plan.create_v([3000] * 8)
    assert big.exec_mode == sp.EXEC_STREAM                    # three passes: launched kernel by kernel


@pytest.mark.gpu
def test_gpu_v_all_empty_but_one_and_misaligned():
    run_v_case(9, [0, 0, 0, 4096, 0, 0, 0, 0, 0], sp.ALGO_SPARBIT, sp.EXEC_AUTO, 1)
    run_v_case(9, [16 * (r + 1) for r in range(9)], sp.ALGO_SPARBIT, sp.EXEC_AUTO, 2, shift=4)
    run_v_case(12, [1000 + 7 * r for r in range(12)], sp.ALGO_NEIGHBOR_EXCHANGE, sp.EXEC_AUTO, 3, shift=1)
    run_v_case(9, [0, 0, 0, 4096, 0, 0, 0, 0, 0], sp.ALGO_SPARBIT, sp.EXEC_MIRROR, 1)
    run_v_case(9, [16 * (r + 1) for r in range(9)], sp.ALGO_SPARBIT, sp.EXEC_MIRROR, 2, shift=4)
    run_v_case(12, [1000 + 7 * r for r in range(12)], sp.ALGO_NEIGHBOR_EXCHANGE, sp.EXEC_MIRROR, 3, shift=1)
    run_v_case(16, [5000] + [0] * 15, sp.ALGO_RING, sp.EXEC_MIRROR, 4, shift=2)


@pytest.mark.gpu
def test_gpu_v_equal_sizes_match_the_fixed_size_plan():
    torch, dev = _gpu()
    P, m = 24, 2048
    host_send = si.send_blocks(P, m, 8).reshape(-1)
    send = torch.from_numpy(host_send).to(dev)
    a = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    b = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    pv = sp.Plan.create_v([m] * P)
    pf = sp.Plan(P, m)
    pv.allgather(send, a)
    pf.allgather(send, b)
    assert pv.status() == sp.OK and pf.status() == sp.OK
    assert torch.equal(a, b)


@pytest.mark.gpu
@pytest.mark.parametrize("exec_mode,copy", [(sp.EXEC_STREAM, sp.COPY_VECTOR), (sp.EXEC_STREAM, sp.COPY_BULK),
                                            (sp.EXEC_PERSISTENT, sp.COPY_VECTOR), (sp.EXEC_PERSISTENT, sp.COPY_BULK)])
def test_gpu_v_state_after_every_phase(exec_mode, copy):
    torch, dev = _gpu()
    P = 21
    counts = si.block_counts(P, 5, unit=16, scale=400)   # up to 13 KiB: several segments per block
    T = sum(counts)
    plan = sp.Plan.create_v(counts, sp.ALGO_SPARBIT, exec_mode)
    plan.set_copy_path(copy)
    ref = oracle.Plan(oracle.SPARBIT, P)
    host_send = si.send_blocks_v(counts, 3)
    send = torch.from_numpy(host_send).to(dev)
    recv = torch.full((P * T,), si.SENTINEL, dtype=torch.uint8, device=dev)
    want = si.sentinel_buffer(P * T)
    for ph in range(-1, ref.num_steps):
        plan.allgather_steps(send, recv, ph, ph)
        assert plan.status() == sp.OK
        ref.run_v(counts, host_send, want, first=ph, last=ph)
        assert np.array_equal(recv.cpu().numpy(), want), ph
    assert plan.copy_path == copy
    # and two phases in one launch (the persistent kernel's grid barrier between them)
    recv.fill_(si.SENTINEL)
    want.fill(si.SENTINEL)
    plan.allgather_steps(send, recv, -1, 1)
    plan.allgather_steps(send, recv, 2, ref.num_steps - 1)
    assert plan.status() == sp.OK
    ref.run_v(counts, host_send, want)
    assert np.array_equal(recv.cpu().numpy(), want)


@pytest.mark.gpu
def test_gpu_v_large_blocks_and_host_entry_point():
    P = 64
    counts = si.block_counts(P, 11, unit=16, scale=2048)   # about 32 KiB on average, up to ~390 KiB
    run_v_case(P, counts, sp.ALGO_SPARBIT, sp.EXEC_AUTO, 5, iters=1)
    run_v_case(P, counts, sp.ALGO_SPARBIT, sp.EXEC_PERSISTENT, 5, iters=2, copy=sp.COPY_BULK)
    run_v_case(P, counts, sp.ALGO_SPARBIT, sp.EXEC_GRAPH, 5, iters=2, copy=sp.COPY_BULK)
    plan = sp.Plan.create_v(counts)
    T = sum(counts)
    host_send = si.send_blocks_v(counts, 6)
    host_recv = si.sentinel_buffer(P * T)
    plan.allgather_host(host_send, host_recv)
    assert np.array_equal(host_recv.reshape(P, T), np.broadcast_to(host_send, (P, T)))
