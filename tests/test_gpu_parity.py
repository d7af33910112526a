"""GPU parity: the CUDA step executor against the CPU oracle, bit for bit, through the C ABI.

Receive buffers (and Bruck workspaces) are pre-filled with a sentinel and sit between guard bands
that are checked after every run; the data changes on every iteration, because an allgather
repeated on unchanged inputs would hide stale reads (the previous run already left the right
answer in place).
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

ALGOS = [sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK, sp.ALGO_NEIGHBOR_EXCHANGE]
EXECS = [sp.EXEC_PERSISTENT, sp.EXEC_GRAPH, sp.EXEC_STREAM, sp.EXEC_FLOW, sp.EXEC_MIRROR]
COPIES = [sp.COPY_VECTOR, sp.COPY_BULK]
G = si.GUARD_BYTES


def is_pow2(p):
    return p & (p - 1) == 0


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    return torch.device("cuda:0")


class Guarded:
    """A device byte buffer of `n` bytes at byte offset `shift` inside a sentinel-filled
    allocation with guard bands on both sides."""

    def __init__(self, n, dev, shift=0, fill=si.SENTINEL):
        self.n, self.shift, self.fill = n, shift, fill
        self.raw = torch.full((n + 2 * G + 64,), fill, dtype=torch.uint8, device=dev)
        base = self.raw.data_ptr()
        align = (-base) % 256  # torch allocations are 512-aligned, but do not rely on it
        self.off = align + G + shift
        self.view = self.raw[self.off:self.off + n]

    @property
    def ptr(self):
        return self.view.data_ptr()

    def guards_intact(self):
        lo = self.raw[: self.off]
        hi = self.raw[self.off + self.n:]
        return bool((lo == self.fill).all()) and bool((hi == self.fill).all())

    def refill(self):
        self.raw.fill_(self.fill)


def run_case(dev, P, m, algo, exec_mode, copy, seed, iters=2, shift_send=0, shift_recv=0, shift_work=0, tune=None,
             ran=None):
    plan = sp.Plan(P, m, algo, exec_mode)
    plan.set_copy_path(copy)
    for key, value in (tune or {}).items():
        plan.set_tunable(key, value)
    send = Guarded(P * m, dev, shift_send, fill=0x3C)
    recv = Guarded(P * P * m, dev, shift_recv)
    work = None
    if algo == sp.ALGO_BRUCK:
        work = Guarded(P * P * m, dev, shift_work)
        plan.set_workspace(work.ptr, P * P * m)
    ref_plan = oracle.Plan(algo, P)
    for it in range(iters):
        host_send = si.send_blocks(P, m, seed + it)
        send.view.copy_(torch.from_numpy(host_send.reshape(-1)))
        recv.refill()
        if work:
            work.refill()
        plan.allgather(send.ptr, recv.ptr)
        assert plan.status() == sp.OK
        want = si.sentinel_buffer(P * P * m)
        scratch = si.sentinel_buffer(P * P * m) if algo == sp.ALGO_BRUCK else None
        ref_plan.run(m, host_send.reshape(-1), want, scratch)
        got = recv.view.cpu().numpy()
        assert np.array_equal(got, want), (P, m, algo, exec_mode, copy, it)
        assert recv.guards_intact() and send.guards_intact()
        assert np.array_equal(send.view.cpu().numpy(), host_send.reshape(-1))  # send is read-only
        if work:
            assert work.guards_intact()
            assert np.array_equal(work.view.cpu().numpy(), scratch)
    if ran is not None:
        assert plan.exec_mode == ran, (P, m, algo, plan.exec_mode)
    plan.destroy()


# ---------------------------------------------------------------- config 1: P=8, m=64 B
@pytest.mark.parametrize("exec_mode", EXECS)
@pytest.mark.parametrize("copy", COPIES)
def test_config1_p8_m64(dev, exec_mode, copy):
    run_case(dev, 8, 64, sp.ALGO_SPARBIT, exec_mode, copy, si.BASE_SEED + 1, iters=3)


# ---------------------------------------------------------------- config 2: non powers of two, all algorithms
@pytest.mark.parametrize("P", [6, 13])
@pytest.mark.parametrize("algo", [sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_BRUCK])
@pytest.mark.parametrize("exec_mode", EXECS)
@pytest.mark.parametrize("copy", COPIES)
def test_config2_non_power_of_two(dev, P, algo, exec_mode, copy):
    run_case(dev, P, 4096, algo, exec_mode, copy, si.BASE_SEED + 2)


@pytest.mark.parametrize("P", [4, 8, 16])
@pytest.mark.parametrize("exec_mode", EXECS)
@pytest.mark.parametrize("copy", COPIES)
def test_config2_recursive_doubling_powers_of_two(dev, P, exec_mode, copy):
    run_case(dev, P, 4096, sp.ALGO_RECURSIVE_DOUBLING, exec_mode, copy, si.BASE_SEED + 2)


@pytest.mark.parametrize("P", [6, 13])
def test_config2_recursive_doubling_refused(P):
    out = ctypes.c_void_p()
    assert binding.lib.sparbit_plan_create(P, 4096, sp.ALGO_RECURSIVE_DOUBLING, 0, ctypes.byref(out)) \
        == sp.ERR_UNSUPPORTED


@pytest.mark.parametrize("P", [6, 8, 14])
@pytest.mark.parametrize("exec_mode", EXECS)
@pytest.mark.parametrize("copy", COPIES)
def test_config2_neighbor_exchange_even_p(dev, P, exec_mode, copy):
    run_case(dev, P, 4096, sp.ALGO_NEIGHBOR_EXCHANGE, exec_mode, copy, si.BASE_SEED + 2)


def test_config2_neighbor_exchange_refused_for_odd_p():
    out = ctypes.c_void_p()
    assert binding.lib.sparbit_plan_create(13, 4096, sp.ALGO_NEIGHBOR_EXCHANGE, 0, ctypes.byref(out)) \
        == sp.ERR_UNSUPPORTED


# ---------------------------------------------------------------- phase-by-phase state
@pytest.mark.parametrize("algo,P", [(sp.ALGO_SPARBIT, 5), (sp.ALGO_SPARBIT, 21), (sp.ALGO_SPARBIT, 32),
                                    (sp.ALGO_BRUCK, 13), (sp.ALGO_RING, 6), (sp.ALGO_RECURSIVE_DOUBLING, 16),
                                    (sp.ALGO_NEIGHBOR_EXCHANGE, 10)])
@pytest.mark.parametrize("exec_mode", [sp.EXEC_PERSISTENT, sp.EXEC_STREAM])
def test_state_after_every_phase(dev, algo, P, exec_mode):
    """Run one phase at a time on both sides; the whole state (sentinel included) must agree."""
    m = 272  # 17 * 16: not a power of two, several vectors per block
    plan = sp.Plan(P, m, algo, exec_mode)
    ref = oracle.Plan(algo, P)
    host_send = si.send_blocks(P, m, 77)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    work = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    if algo == sp.ALGO_BRUCK:
        plan.set_workspace(work, P * P * m)
    want = si.sentinel_buffer(P * P * m)
    scratch = si.sentinel_buffer(P * P * m)
    for ph in range(-1, ref.last_phase + 1):
        plan.allgather_steps(send, recv, ph, ph)
        assert plan.status() == sp.OK
        ref.run(m, host_send.reshape(-1), want, scratch, first=ph, last=ph)
        assert np.array_equal(recv.cpu().numpy(), want), ph
        if algo == sp.ALGO_BRUCK:
            assert np.array_equal(work.cpu().numpy(), scratch), ph


@pytest.mark.parametrize("algo,P", [(sp.ALGO_SPARBIT, 5), (sp.ALGO_SPARBIT, 21), (sp.ALGO_SPARBIT, 32),
                                    (sp.ALGO_SPARBIT, 61), (sp.ALGO_BRUCK, 13), (sp.ALGO_BRUCK, 24),
                                    (sp.ALGO_RING, 6), (sp.ALGO_RECURSIVE_DOUBLING, 32),
                                    (sp.ALGO_NEIGHBOR_EXCHANGE, 28)])
def test_mirror_state_after_every_prefix(dev, algo, P):
    """The mirror executor takes calls that start at the beginning (its on-chip copy starts empty): run
    passes -1..k for every k, each time into sentinel-filled buffers; the whole state in global memory
    (receive and working buffers, sentinel included) must be the oracle's after step k.  P = 5..24
    run in one CTA, P = 28..61 on a cluster (Bruck at 24 too: twice the shared memory)."""
    m = 272
    plan = sp.Plan(P, m, algo, sp.EXEC_MIRROR)
    ref = oracle.Plan(algo, P)
    host_send = si.send_blocks(P, m, 78)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.empty((P * P * m,), dtype=torch.uint8, device=dev)
    work = torch.empty((P * P * m,), dtype=torch.uint8, device=dev)
    if algo == sp.ALGO_BRUCK:
        plan.set_workspace(work, P * P * m)
    for k in range(-1, ref.last_phase + 1):
        recv.fill_(si.SENTINEL)
        work.fill_(si.SENTINEL)
        plan.allgather_steps(send, recv, -1, k)
        assert plan.status() == sp.OK and plan.exec_mode == sp.EXEC_MIRROR
        want = si.sentinel_buffer(P * P * m)
        scratch = si.sentinel_buffer(P * P * m)
        ref.run(m, host_send.reshape(-1), want, scratch, first=-1, last=k)
        assert np.array_equal(recv.cpu().numpy(), want), k
        if algo == sp.ALGO_BRUCK:
            assert np.array_equal(work.cpu().numpy(), scratch), k


@pytest.mark.parametrize("exec_mode", [sp.EXEC_GRAPH, sp.EXEC_STREAM])
@pytest.mark.parametrize("algo,P,m", [(sp.ALGO_SPARBIT, P, m) for P, m in
                                      [(16, 64), (32, 272), (64, 64), (96, 100), (128, 16), (192, 24), (256, 64),
                                       (256, 8), (24, 1000), (40, 6), (512, 16), (1000, 4), (48, 3)]] +
                                     [(sp.ALGO_RECURSIVE_DOUBLING, P, m) for P, m in
                                      [(16, 64), (32, 272), (64, 48), (128, 16), (256, 64), (256, 6), (512, 8)]])
def test_grouped_front_state_after_every_prefix(dev, exec_mode, algo, P, m):
    """The leading passes as independent groups, one CTA each, then the chain (Sparbit: residue
    classes of ranks; recursive doubling: runs of consecutive ranks): run passes -1..k for every k
    into sentinel-filled buffers; the whole receive space must be the oracle's state after step k,
    whether the call ends inside the grouped passes or behind them."""
    plan = sp.Plan(P, m, algo, exec_mode)
    ref = oracle.Plan(algo, P)
    host_send = si.send_blocks(P, m, 79)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.empty((P * P * m,), dtype=torch.uint8, device=dev)
    grouped = 0
    for k in range(-1, ref.last_phase + 1):
        recv.fill_(si.SENTINEL)
        before = plan.launch_counts()[0]
        plan.allgather_steps(send, recv, -1, k)
        assert plan.status() == sp.OK
        launches = plan.launch_counts()[0] - before
        passes = max(1, k + 1)            # the own-block copy is fused into step 0
        grouped = max(grouped, passes - launches)
        want = si.sentinel_buffer(P * P * m)
        ref.run(m, host_send.reshape(-1), want, None, first=-1, last=k)
        assert np.array_equal(recv.cpu().numpy(), want), (P, m, k)
    if P in (16, 32, 64, 128, 256, 512, 96, 192):
        assert grouped >= 1, (algo, P, m)  # some passes did share a kernel
    plan.destroy()


# ---------------------------------------------------------------- brute force over P
ALL_IN_FLOW = {sp.TUNE_FLOW_MIN_PASS_SPANS: 1}     # every pass in the flow kernel
SPLIT_FLOW = {sp.TUNE_FLOW_MIN_PASS_SPANS: 40}     # passes of fewer than 40 spans as kernels in front of it


@pytest.mark.parametrize("exec_mode,m,tune", [(sp.EXEC_PERSISTENT, 16, None), (sp.EXEC_FLOW, 512, ALL_IN_FLOW),
                                              (sp.EXEC_FLOW, 1040, ALL_IN_FLOW), (sp.EXEC_FLOW, 1040, SPLIT_FLOW),
                                              (sp.EXEC_FLOW, 16, None), (sp.EXEC_MIRROR, 16, None),
                                              (sp.EXEC_MIRROR, 52, None), (sp.EXEC_MIRROR, 600, None)])
def test_every_p_up_to_64(dev, exec_mode, m, tune):
    """Every communicator size, on the single-kernel executors.  The flow executor takes blocks
    of at least 32 vectors (512 B: one warp row; 1040 B: two ragged spans per block) and hands
    smaller ones to the graph chain, and by default leaves passes that cannot keep every warp busy
    to per-pass kernels in front of it: the tests set that threshold so that the kernel takes
    every pass, or only those of at least 40 spans; the mirror executor runs in one CTA up to 64 KiB of
    receive buffers (all of these at 16 B) and in a cluster of 2 to 16 CTAs above that (52 B from
    P = 36 on, 600 B from P = 11 on)."""
    for P in range(1, 65):
        ran = sp.EXEC_FLOW if tune is ALL_IN_FLOW else None
        run_case(dev, P, m, sp.ALGO_SPARBIT, exec_mode, sp.COPY_AUTO, 1000 + P, iters=2 if m != 16 else 1, tune=tune,
                 ran=ran)


@pytest.mark.parametrize("algo", [sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK,
                                  sp.ALGO_NEIGHBOR_EXCHANGE])
def test_comparators_many_p(dev, algo):
    for P in [1, 2, 3, 4, 5, 7, 8, 12, 16, 17, 31, 32, 33, 64]:
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        run_case(dev, P, 48, algo, sp.EXEC_PERSISTENT, sp.COPY_AUTO, 2000 + P, iters=1)


# ---------------------------------------------------------------- any block size, any alignment
@pytest.mark.parametrize("m", [1, 2, 3, 6, 10, 20, 100, 1000, 4100, 16400])
@pytest.mark.parametrize("exec_mode", [sp.EXEC_PERSISTENT, sp.EXEC_GRAPH, sp.EXEC_FLOW, sp.EXEC_MIRROR])
def test_odd_block_sizes(dev, m, exec_mode):
    run_case(dev, 7, m, sp.ALGO_SPARBIT, exec_mode, sp.COPY_AUTO, 31 + m, iters=1,
             tune=ALL_IN_FLOW if exec_mode == sp.EXEC_FLOW else None)


@pytest.mark.parametrize("shifts", [(1, 0, 0), (0, 1, 0), (2, 2, 2), (4, 8, 4), (8, 8, 8), (3, 5, 7), (16, 32, 48)])
@pytest.mark.parametrize("algo", [sp.ALGO_SPARBIT, sp.ALGO_BRUCK])
def test_misaligned_buffers(dev, shifts, algo):
    """Buffers at odd addresses must fall back to narrower vectors (and off the bulk engine)."""
    for m in (64, 4096):
        for copy in COPIES:
            run_case(dev, 9, m, algo, sp.EXEC_PERSISTENT, copy, 5, iters=1, shift_send=shifts[0],
                     shift_recv=shifts[1], shift_work=shifts[2])


def test_single_rank_and_empty_blocks(dev):
    for algo in ALGOS:
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE:
            continue  # one rank is not an even number of ranks
        run_case(dev, 1, 256, algo, sp.EXEC_AUTO, sp.COPY_AUTO, 9, iters=1)
    run_case(dev, 2, 256, sp.ALGO_NEIGHBOR_EXCHANGE, sp.EXEC_AUTO, sp.COPY_AUTO, 9, iters=1)
    plan = sp.Plan(8, 0)
    plan.allgather(None, None)
    assert plan.status() == sp.OK


# ---------------------------------------------------------------- larger shapes (several tiles, ragged tails)
@pytest.mark.parametrize("P,m", [(37, 20480 + 16), (128, 8192), (100, 33 * 1024)])
@pytest.mark.parametrize("exec_mode", [sp.EXEC_PERSISTENT, sp.EXEC_GRAPH])
@pytest.mark.parametrize("copy", COPIES)
def test_medium_shapes(dev, P, m, exec_mode, copy):
    run_case(dev, P, m, sp.ALGO_SPARBIT, exec_mode, copy, 4242)


@pytest.mark.parametrize("algo", [sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK,
                                  sp.ALGO_NEIGHBOR_EXCHANGE])
@pytest.mark.parametrize("copy", COPIES)
def test_medium_shapes_comparators(dev, algo, copy):
    run_case(dev, 64, 20480, algo, sp.EXEC_PERSISTENT, copy, 4343, iters=1)


# ---------------------------------------------------------------- the bounded wait of the grid barrier
@pytest.mark.parametrize("copy", COPIES)
def test_grid_barrier_gives_up_instead_of_hanging(dev, copy):
    """With one arrival more expected than there are CTAs the barrier can never complete: the
    kernel must come back with the time-out status, and the plan must work again afterwards."""
    P, m = 16, 4096
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_PERSISTENT)
    plan.set_copy_path(copy)
    host_send = si.send_blocks(P, m, 1)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.set_barrier_test(1, 20_000_000)  # 20 ms
    plan.allgather(send, recv)
    assert plan.status() == sp.ERR_TIMEOUT
    assert plan.status() == sp.OK        # the condition is cleared by reading it
    plan.set_barrier_test(0, 0)
    recv.fill_(si.SENTINEL)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))


def test_flow_wait_gives_up_instead_of_hanging(dev):
    """The flow executor's per-rank waits are bounded too: with counter targets that are never
    reached (the same host-set hook) every waiting warp must leave with the time-out status, and
    the plan must work again afterwards, its counters cleared."""
    P, m = 16, 4096
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_FLOW)
    plan.set_tunable(sp.TUNE_FLOW_MIN_PASS_SPANS, 1)
    host_send = si.send_blocks(P, m, 1)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK and plan.exec_mode == sp.EXEC_FLOW
    plan.set_barrier_test(1, 20_000_000)  # 20 ms
    plan.allgather(send, recv)
    assert plan.status() == sp.ERR_TIMEOUT
    assert plan.status() == sp.OK
    plan.set_barrier_test(0, 0)
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    for _ in range(2):
        recv.fill_(si.SENTINEL)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK
        assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))


def test_flow_launch_forms_and_the_measurement_hook(dev):
    """The flow kernel as a cooperative launch every time (the tunable), as an ordinary launch
    behind a flow launch in the same stream (the default from the second call on), and with its
    waits switched off (a measurement hook: the call must complete and report no error; its result
    is wrong by design and is not looked at)."""
    P, m = 48, 8192
    host_send = si.send_blocks(P, m, 21)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    for coop in (1, 0):
        plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_FLOW)
        plan.set_tunable(sp.TUNE_FLOW_COOPERATIVE, coop)
        for _ in range(3):
            recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
            plan.allgather(send, recv)
            assert plan.status() == sp.OK and plan.exec_mode == sp.EXEC_FLOW
            assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
        plan.destroy()
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_FLOW)
    plan.set_tunable(sp.TUNE_FLOW_SKIP_WAITS, 1)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    plan.set_tunable(sp.TUNE_FLOW_SKIP_WAITS, 0)
    recv.fill_(si.SENTINEL)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
    plan.destroy()


@pytest.mark.parametrize("exec_mode", EXECS + [sp.EXEC_AUTO])
def test_collective_inside_a_captured_graph_replays(dev, exec_mode):
    """A collective enqueued on a stream under capture must replay as often as the caller likes:
    nothing in the captured work may depend on counters of one particular launch.  Each replay
    runs on new send data and into sentinel-filled buffers."""
    for P, m in ((16, 2048), (8, 64), (48, 4096)):
        plan = sp.Plan(P, m, sp.ALGO_SPARBIT, exec_mode)
        send = torch.zeros(P * m, dtype=torch.uint8, device=dev)
        recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            plan.allgather(send, recv, stream)      # the first call allocates the plan's device state
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            graph.capture_begin()
            plan.allgather(send, recv, stream)
            graph.capture_end()
        for it in range(3):
            host_send = si.send_blocks(P, m, 30 + it)
            send.copy_(torch.from_numpy(host_send.reshape(-1)))
            recv.fill_(si.SENTINEL)
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
            assert np.array_equal(recv.cpu().numpy(), want.reshape(-1)), (P, m, exec_mode, it)
        # and the plan still works outside the graph
        recv.fill_(si.SENTINEL)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK
        assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
        del graph
        plan.destroy()


def test_two_flow_collectives_at_once(dev):
    """Two plans, two streams, both on the flow executor at the same time.  Each kernel's waits
    need all of its CTAs resident; the cooperative launch sees to that (the second kernel starts
    when the first has left room), so both must finish, and with the right bytes."""
    cases = [(64, 16384, 11), (48, 32768, 12)]
    plans, sends, recvs, streams, wants = [], [], [], [], []
    for P, m, seed in cases:
        plans.append(sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_FLOW))
        host_send = si.send_blocks(P, m, seed)
        sends.append(torch.from_numpy(host_send.reshape(-1)).to(dev))
        recvs.append(torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev))
        streams.append(torch.cuda.Stream(device=dev))
        wants.append(host_send.reshape(-1))
    torch.cuda.synchronize()
    for it in range(6):
        for plan, send, recv, st in zip(plans, sends, recvs, streams):
            plan.allgather(send, recv, st)
    for (P, m, _), plan, recv, want in zip(cases, plans, recvs, wants):
        assert plan.status() == sp.OK and plan.exec_mode == sp.EXEC_FLOW
        got = recv.cpu().numpy().reshape(P, P * m)
        assert all(np.array_equal(got[r], want) for r in range(P))
        plan.destroy()


@pytest.mark.parametrize("algo", ALGOS)
def test_flow_all_algorithms_changing_data(dev, algo):
    """Every algorithm on the flow executor, several calls in a row on one plan (the counters
    carry over from call to call) with new data and a fresh sentinel fill each time."""
    narrow = dict(ALL_IN_FLOW)
    narrow[sp.TUNE_FLOW_WIDE_MAX_MOVED_BYTES] = 0   # two vectors per lane whatever the block size
    for P, m in ((16, 2048), (12, 1024), (64, 512), (13, 4096), (1, 512), (2, 8192), (5, 4144), (24, 12304)):
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        if algo == sp.ALGO_RING and P > 32:
            continue   # more passes than the flow executor's counter line holds: runs as a graph
        run_case(dev, P, m, algo, sp.EXEC_FLOW, sp.COPY_AUTO, 77 + P, iters=3, tune=ALL_IN_FLOW, ran=sp.EXEC_FLOW)
        run_case(dev, P, m, algo, sp.EXEC_FLOW, sp.COPY_AUTO, 78 + P, iters=2, tune=SPLIT_FLOW)
        if m >= 4096:   # by default these run with four vectors per lane
            run_case(dev, P, m, algo, sp.EXEC_FLOW, sp.COPY_AUTO, 79 + P, iters=2, tune=narrow, ran=sp.EXEC_FLOW)


@pytest.mark.parametrize("algo", ALGOS)
def test_mirror_all_algorithms_changing_data(dev, algo):
    """The mirror executor on every algorithm it takes, up to the largest receive space that
    fits one SM's shared memory, at misaligned addresses too, with new data on every call."""
    for P, m in ((8, 64), (6, 4096), (13, 1024), (16, 800), (2, 32768), (1, 4096), (12, 100), (7, 4500),
                 (16, 4096), (13, 8192), (32, 1000), (64, 208), (128, 64), (100, 96), (253, 24),
                 (40, 100), (40, 70), (40, 75)):   # the last three: clusters on 4-, 2- and 1-byte vectors
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        if algo == sp.ALGO_RING and P > 17 or algo == sp.ALGO_NEIGHBOR_EXCHANGE and P > 32:
            continue   # more passes than the kernel's parameter table holds
        if algo == sp.ALGO_BRUCK and 2 * ((P + 15) // 16) * P * m > 220 * 1024:
            continue   # Bruck mirrors its working buffers as well
        run_case(dev, P, m, algo, sp.EXEC_MIRROR, sp.COPY_AUTO, 90 + P, iters=3, ran=sp.EXEC_MIRROR)
    run_case(dev, 9, 96, algo if algo != sp.ALGO_RECURSIVE_DOUBLING and algo != sp.ALGO_NEIGHBOR_EXCHANGE
             else sp.ALGO_SPARBIT, sp.EXEC_MIRROR, sp.COPY_AUTO, 5, iters=1, shift_send=4, shift_recv=8)
    if algo in (sp.ALGO_SPARBIT, sp.ALGO_BRUCK):
        run_case(dev, 40, 96, algo, sp.EXEC_MIRROR, sp.COPY_AUTO, 6, iters=2, shift_send=4, shift_recv=8, ran=sp.EXEC_MIRROR)
        run_case(dev, 40, 96, algo, sp.EXEC_MIRROR, sp.COPY_AUTO, 7, iters=2, shift_send=2, shift_recv=6, ran=sp.EXEC_MIRROR)


def test_mirror_runs_where_it_fits_and_hands_over_where_not(dev):
    # one CTA up to 227 KB, a cluster of up to 16 CTAs up to 16 x 227 KB, the graph chain beyond
    for P, m, want in ((8, 64, sp.EXEC_MIRROR), (6, 4096, sp.EXEC_MIRROR), (13, 4096, sp.EXEC_MIRROR),
                       (64, 64, sp.EXEC_MIRROR), (20, 16, sp.EXEC_MIRROR), (256, 48, sp.EXEC_MIRROR),
                       (64, 4096, sp.EXEC_GRAPH), (256, 64, sp.EXEC_GRAPH)):
        plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_MIRROR)
        send = torch.from_numpy(si.send_blocks(P, m, 1).reshape(-1)).to(dev)
        recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK and plan.exec_mode == want, (P, m)
        assert all(torch.equal(recv.view(P, P * m)[r], send) for r in range(P))
        plan.destroy()
    # a ring of 20 ranks has 19 passes: more than the kernel's parameter table holds
    plan = sp.Plan(20, 16, sp.ALGO_RING, sp.EXEC_MIRROR)
    send = torch.from_numpy(si.send_blocks(20, 16, 1).reshape(-1)).to(dev)
    recv = torch.full((20 * 20 * 16,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK and plan.exec_mode == sp.EXEC_GRAPH


# ---------------------------------------------------------------- host-buffer entry point, streams, bookkeeping
@pytest.mark.parametrize("algo", [sp.ALGO_SPARBIT, sp.ALGO_BRUCK])
def test_host_entry_point(dev, algo):
    P, m = 24, 2048
    plan = sp.Plan(P, m, algo)
    for it in range(2):
        host_send = si.send_blocks(P, m, 50 + it)
        host_recv = si.sentinel_buffer(P * P * m)
        plan.allgather_host(host_send, host_recv)
        want, _ = oracle.allgather(algo, P, m, host_send)
        assert np.array_equal(host_recv, want.reshape(-1))


@pytest.mark.parametrize("exec_mode", EXECS)
def test_runs_on_a_user_stream_and_counts_launches(dev, exec_mode):
    P, m = 16, 1024
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, exec_mode)
    plan.set_tunable(sp.TUNE_FLOW_MIN_PASS_SPANS, 1)   # the flow kernel takes every pass
    host_send = si.send_blocks(P, m, 3)
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        send = torch.from_numpy(host_send.reshape(-1)).to(dev, non_blocking=False)
        recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        stream.synchronize()
        plan.allgather(send, recv, stream)
        plan.allgather(send, recv, stream)
    assert plan.status() == sp.OK
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
    kernels, graphs = plan.launch_counts()
    phases = plan.num_steps  # the own-block copy and step 0 run as one fused pass
    if exec_mode in (sp.EXEC_PERSISTENT, sp.EXEC_FLOW):
        assert (kernels, graphs) == (2, 0)
    elif exec_mode == sp.EXEC_MIRROR:
        assert (kernels, graphs) == (2, 0)     # 256 KiB of receive buffers: one cluster kernel, launched as itself
        small = sp.Plan(8, 64, sp.ALGO_SPARBIT, sp.EXEC_MIRROR)
        small.allgather(send[: 8 * 64], recv, stream)
        small.allgather(send[: 8 * 64], recv, stream)
        assert small.status() == sp.OK and small.launch_counts() == (2, 0)   # one kernel per call, no graph
        small.destroy()
    elif exec_mode == sp.EXEC_GRAPH:
        assert (kernels, graphs) == (2 * 2, 2)     # three passes as 2 groups of 8 ranks in one kernel, then the last pass
        plain = sp.Plan(P, m, sp.ALGO_SPARBIT, exec_mode)
        plain.set_tunable(sp.TUNE_GROUPED_FRONT, 0)
        plain.allgather(send, recv, stream)
        assert plain.status() == sp.OK and plain.launch_counts() == (phases, 1)   # every pass its own kernel
        assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
        plain.destroy()
    else:
        assert (kernels, graphs) == (2 * 2, 0)
    assert plan.exec_mode == exec_mode


def test_graph_follows_new_pointers(dev):
    """The cached graph must not keep using the buffers of an earlier call."""
    P, m = 12, 4096
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_GRAPH)
    for it in range(3):
        host_send = si.send_blocks(P, m, 600 + it)
        send = torch.from_numpy(host_send.reshape(-1)).to(dev)
        recv = torch.full((P * P * m + 64 * it,), si.SENTINEL, dtype=torch.uint8, device=dev)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK
        want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
        assert np.array_equal(recv[: P * P * m].cpu().numpy(), want.reshape(-1))


@pytest.mark.parametrize("copy", COPIES)
def test_graph_cache_recycles_entries(dev, copy):
    """More buffer sets than the graph cache holds: the least recently used instance is
    re-parameterised in place and must then use the new buffers, not the old ones."""
    P, m = 10, 4096
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_GRAPH)
    plan.set_copy_path(copy)
    sets = []
    for k in range(7):
        host_send = si.send_blocks(P, m, 900 + k)
        sets.append((host_send, torch.from_numpy(host_send.reshape(-1)).to(dev),
                     torch.empty(P * P * m, dtype=torch.uint8, device=dev)))
    for rnd in range(2):
        for host_send, send, recv in sets:
            recv.fill_(si.SENTINEL)
            plan.allgather(send, recv)
        assert plan.status() == sp.OK
        for host_send, send, recv in sets:
            want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
            assert np.array_equal(recv.cpu().numpy(), want.reshape(-1)), rnd
    # partial ranges get graphs of their own and must not disturb the cached full ones
    host_send, send, recv = sets[0]
    recv.fill_(si.SENTINEL)
    plan.allgather_steps(send, recv, -1, 1)
    plan.allgather_steps(send, recv, 2, plan.last_phase)
    assert plan.status() == sp.OK
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))


@pytest.mark.parametrize("copy", COPIES)
def test_persistent_trace_gives_one_stamp_per_pass(dev, copy):
    P, m = 64, 16384
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_PERSISTENT)
    plan.set_copy_path(copy)
    host_send = si.send_blocks(P, m, 21)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    assert len(plan.get_trace()) == 0
    plan.set_trace(True)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    t = plan.get_trace().astype(np.int64)
    assert len(t) == plan.num_steps + 1          # start + one per pass (own block fused with step 0)
    d = np.diff(t)
    assert (d > 0).all()
    assert d[-1] > d[1]                           # the last pass moves 32x the bytes of the second
    assert 10_000 < t[-1] - t[0] < 5_000_000      # tens of microseconds, not garbage
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
    plan.set_trace(False)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK and len(plan.get_trace()) == 0


def test_cluster_mirror_wait_gives_up_instead_of_hanging(dev):
    """The cluster form of the mirror executor waits for a pass's bytes on mbarriers: with more bytes
    expected than ever arrive every wait must time out, the status word must say so, and the plan
    must work again afterwards."""
    P, m = 64, 64
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_MIRROR)
    host_send = si.send_blocks(P, m, 3)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.set_mbarrier_test(16, 5_000_000)   # 5 ms
    plan.allgather(send, recv)
    assert plan.status() == sp.ERR_TIMEOUT
    plan.set_mbarrier_test(0, 0)
    recv.fill_(si.SENTINEL)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK and plan.exec_mode == sp.EXEC_MIRROR
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))


@pytest.mark.parametrize("exec_mode", [sp.EXEC_PERSISTENT, sp.EXEC_STREAM])
def test_bulk_stage_wait_gives_up_instead_of_hanging(dev, exec_mode):
    """The bulk engine's wait for a stage to fill is bounded too: with more bytes expected than
    are ever loaded it must time out, report it through the status word, and leave the plan usable."""
    P, m = 8, 4096
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, exec_mode)
    plan.set_copy_path(sp.COPY_BULK)
    host_send = si.send_blocks(P, m, 2)
    send = torch.from_numpy(host_send.reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.set_mbarrier_test(16, 5_000_000)   # 5 ms
    plan.allgather(send, recv)
    assert plan.status() == sp.ERR_TIMEOUT
    plan.set_mbarrier_test(0, 0)
    recv.fill_(si.SENTINEL)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    want, _ = oracle.allgather(oracle.SPARBIT, P, m, host_send)
    assert np.array_equal(recv.cpu().numpy(), want.reshape(-1))
