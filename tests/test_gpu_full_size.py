"""GPU parity at the benchmark's full sizes, in the launch configurations the benchmark times.

Where the oracle can simulate the whole collective in seconds (configs 3 and 4, and the sweep of
config 5 up to 64 KiB blocks) the comparison is element by element over the whole receive space.
At the 16 GiB point of the sweep the oracle's message lists are traced for a seeded sample of
(rank, slot) outputs, and the whole state is checked on the device against the property that
holds at any size: every receive buffer equals the concatenation of the send blocks.
"""
import numpy as np
import pytest

import oracle
import seeded_inputs as si
import paper_2109_08751_b200 as sp

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    return torch.device("cuda:0")


def full_compare(dev, P, m, algo, exec_mode, copy, seed, iters=2, ran_on=None):
    plan = sp.Plan(P, m, algo, exec_mode)
    plan.set_copy_path(copy)
    ref = oracle.Plan(algo, P)
    recv = torch.empty(P * P * m, dtype=torch.uint8, device=dev)
    work = None
    if algo == sp.ALGO_BRUCK:
        work = torch.empty(P * P * m, dtype=torch.uint8, device=dev)
        plan.set_workspace(work, P * P * m)
    want = np.empty(P * P * m, dtype=np.uint8)
    scratch = np.empty(P * P * m, dtype=np.uint8) if algo == sp.ALGO_BRUCK else None
    for it in range(iters):
        host_send = si.send_blocks(P, m, seed + it).reshape(-1)
        send = torch.from_numpy(host_send).to(dev)
        recv.fill_(si.SENTINEL)
        if work is not None:
            work.fill_(si.SENTINEL)
        plan.allgather(send, recv)
        assert plan.status() == sp.OK
        if ran_on is not None:
            assert (plan.exec_mode, plan.copy_path) == ran_on
        want.fill(si.SENTINEL)
        if scratch is not None:
            scratch.fill(si.SENTINEL)
        ref.run(m, host_send, want, scratch, threads=4)
        # compare on the device, a rank group at a time, to keep host traffic in one direction
        step = max(1, (256 << 20) // (P * m))
        for r0 in range(0, P, step):
            r1 = min(P, r0 + step)
            w = torch.from_numpy(want[r0 * P * m:r1 * P * m]).to(dev)
            assert torch.equal(recv[r0 * P * m:r1 * P * m], w), (P, m, algo, exec_mode, copy, it, r0)
    plan.destroy()


# config 3: bandwidth-bound, persistent executor with a grid barrier per step
@pytest.mark.parametrize("copy", [sp.COPY_BULK, sp.COPY_VECTOR])
def test_config3_p128_m64k_persistent(dev, copy):
    full_compare(dev, 128, 64 * 1024, sp.ALGO_SPARBIT, sp.EXEC_PERSISTENT, copy, si.BASE_SEED + 3)


def test_config3_p128_m64k_flow(dev):
    full_compare(dev, 128, 64 * 1024, sp.ALGO_SPARBIT, sp.EXEC_FLOW, sp.COPY_AUTO, si.BASE_SEED + 3)


def test_config3_auto_is_what_the_benchmark_runs(dev):
    full_compare(dev, 128, 64 * 1024, sp.ALGO_SPARBIT, sp.EXEC_AUTO, sp.COPY_AUTO, si.BASE_SEED + 3, iters=1)


def test_blocks_off_128_byte_lines_auto_keeps_the_bulk_engine(dev):
    # 1.07 GB moved, m a multiple of 16 but not of 128: AUTO leaves the flow executor aside
    full_compare(dev, 128, 32752, sp.ALGO_SPARBIT, sp.EXEC_AUTO, sp.COPY_AUTO, si.BASE_SEED + 3, iters=1,
                 ran_on=(sp.EXEC_GRAPH, sp.COPY_BULK))


# config 4: many small blocks, non-power-of-two; graph chain vs persistent
@pytest.mark.parametrize("exec_mode", [sp.EXEC_PERSISTENT, sp.EXEC_GRAPH, sp.EXEC_AUTO])
def test_config4_p1000_m1k(dev, exec_mode):
    full_compare(dev, 1000, 1024, sp.ALGO_SPARBIT, exec_mode, sp.COPY_AUTO, si.BASE_SEED + 4,
                 iters=2 if exec_mode != sp.EXEC_AUTO else 1)


# config 5: the sweep at P = 256
@pytest.mark.parametrize("m", [8, 64, 512, 4096, 32768])
@pytest.mark.parametrize("algo", [sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK,
                                  sp.ALGO_NEIGHBOR_EXCHANGE])
def test_config5_sweep(dev, m, algo):
    full_compare(dev, 256, m, algo, sp.EXEC_AUTO, sp.COPY_AUTO, si.BASE_SEED + 5, iters=1)


@pytest.mark.parametrize("algo", [sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_NEIGHBOR_EXCHANGE])
def test_config5_comparators_at_64k(dev, algo):
    """The comparators at the headline block size, whole receive space against the oracle."""
    full_compare(dev, 256, 64 * 1024, algo, sp.EXEC_AUTO, sp.COPY_AUTO, si.BASE_SEED + 5, iters=1)


def sampled_compare(dev, plan, ref, P, offsets, host_send, recv, samples=192, seed=12345):
    """Sampled (rank, slot) outputs through the oracle's message lists, then the whole state
    against the property that holds at any size: every receive buffer is the concatenation of
    the send blocks.  offsets[b] .. offsets[b+1] is block b inside a receive buffer."""
    T = int(offsets[P])
    send = torch.from_numpy(host_send).to(dev)
    for k in si.sample_indices(samples, P * P, seed=seed):
        r, b = divmod(int(k), P)
        path = ref.trace(r, b)
        origin = int(path[0]["src_rank"])
        lo, hi = int(offsets[b]), int(offsets[b + 1])
        got = recv[r * T + lo:r * T + hi].cpu().numpy()
        assert np.array_equal(got, host_send[int(offsets[origin]):int(offsets[origin + 1])]), (r, b)
    view = recv.view(P, T)
    for r in range(P):
        assert torch.equal(view[r], send), r


def test_config5_bruck_at_64k_sampled(dev):
    """Bruck at the headline block size: the oracle would need 8 GiB of host memory for its two
    spaces, so sampled outputs are traced through its message lists (rotation included)."""
    P, m = 256, 64 * 1024
    plan = sp.Plan(P, m, sp.ALGO_BRUCK, sp.EXEC_AUTO)
    ref = oracle.Plan(oracle.BRUCK, P)
    host_send = si.send_blocks(P, m, si.BASE_SEED + 5).reshape(-1)
    send = torch.from_numpy(host_send).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    work = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.set_workspace(work, P * P * m)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    sampled_compare(dev, plan, ref, P, np.arange(P + 1, dtype=np.int64) * m, host_send, recv)
    plan.destroy()


# Receive spaces beyond 4 GiB: byte offsets that do not fit 32 bits, on every engine and executor
# (at the headline point P*P*m is exactly 2^32, so no offset there needs the 33rd bit).
BIG_P, BIG_M = 272, 64 * 1024   # 4.85 GB of receive buffers, not a power of two, 9 steps


@pytest.mark.parametrize("exec_mode,copy", [(sp.EXEC_GRAPH, sp.COPY_VECTOR), (sp.EXEC_PERSISTENT, sp.COPY_VECTOR),
                                            (sp.EXEC_PERSISTENT, sp.COPY_BULK), (sp.EXEC_STREAM, sp.COPY_BULK),
                                            (sp.EXEC_FLOW, sp.COPY_VECTOR)])
def test_offsets_beyond_4gib(dev, exec_mode, copy):
    P, m = BIG_P, BIG_M
    assert P * P * m > 1 << 32
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, exec_mode)
    plan.set_copy_path(copy)
    ref = oracle.Plan(oracle.SPARBIT, P)
    host_send = si.send_blocks(P, m, si.BASE_SEED + 6).reshape(-1)
    send = torch.from_numpy(host_send).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    assert plan.copy_path == copy and plan.exec_mode == exec_mode
    for k in si.sample_indices(8, P * P, seed=99):   # hop counts: one per set bit of the distance
        r, b = divmod(int(k), P)
        assert len(ref.trace(r, b)) - 1 == bin((r - b) % P).count("1")
    sampled_compare(dev, plan, ref, P, np.arange(P + 1, dtype=np.int64) * m, host_send, recv)
    plan.destroy()


@pytest.mark.parametrize("exec_mode", [sp.EXEC_GRAPH, sp.EXEC_PERSISTENT])
def test_allgatherv_offsets_beyond_4gib(dev, exec_mode):
    """Blocks of different sizes whose receive space P*T exceeds 4 GiB."""
    P = BIG_P
    counts = si.block_counts(P, 77, kind="mixed", unit=16, scale=BIG_M // 16 * 9 // 13)
    offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    T = int(offsets[P])
    assert P * T > 1 << 32
    plan = sp.Plan.create_v(counts, sp.ALGO_SPARBIT, exec_mode)
    ref = oracle.Plan(oracle.SPARBIT, P)
    host_send = si.send_blocks_v(counts, si.BASE_SEED + 7)
    send = torch.from_numpy(host_send).to(dev)
    recv = torch.full((P * T,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    sampled_compare(dev, plan, ref, P, offsets, host_send, recv)
    plan.destroy()


@pytest.mark.parametrize("exec_mode,copy", [(sp.EXEC_AUTO, sp.COPY_AUTO), (sp.EXEC_GRAPH, sp.COPY_BULK),
                                            (sp.EXEC_PERSISTENT, sp.COPY_VECTOR)])
def test_config5_headline_point_p256_m64k(dev, exec_mode, copy):
    """The point the benchmark's headline number is quoted on (4 GiB of receive buffers)."""
    full_compare(dev, 256, 64 * 1024, sp.ALGO_SPARBIT, exec_mode, copy, si.BASE_SEED + 5, iters=1)


def test_config5_largest_point_p256_m256k_sampled(dev):
    """16 GiB of receive buffers: sampled outputs through the oracle's message lists, and the
    whole state against the result's plain definition, checked on the device."""
    P, m = 256, 256 * 1024
    plan = sp.Plan(P, m)
    ref = oracle.Plan(oracle.SPARBIT, P)
    host_send = si.send_blocks(P, m, si.BASE_SEED + 5).reshape(-1)
    send = torch.from_numpy(host_send).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    blocks = host_send.reshape(P, m)
    for k in si.sample_indices(192, P * P, seed=12345):
        r, b = divmod(int(k), P)
        path = ref.trace(r, b)
        origin = int(path[0]["src_rank"])
        assert len(path) - 1 == bin((r - b) % P).count("1")  # one hop per set bit of the distance
        got = recv[(r * P + b) * m:(r * P + b + 1) * m].cpu().numpy()
        assert np.array_equal(got, blocks[origin]), (r, b)
    view = recv.view(P, P * m)
    for r in range(P):
        assert torch.equal(view[r], send), r
    plan.destroy()


@pytest.mark.parametrize("P,m", [(4097, 3), (20011, 4), (65536, 1), (2, 1 << 30)])
@pytest.mark.parametrize("exec_mode", [sp.EXEC_AUTO, sp.EXEC_PERSISTENT])
def test_extreme_shapes_against_the_plain_definition(dev, P, m, exec_mode):
    """Communicators far larger than any the paper measures (tens of thousands of ranks with
    blocks of a few bytes; a prime P) and blocks of 1 GiB: too many messages for the oracle's lists,
    so the whole state is checked on the device against what holds at any size - every receive
    buffer is the concatenation of the send blocks - after a sentinel fill."""
    plan = sp.Plan(P, m, sp.ALGO_SPARBIT, exec_mode)
    send = torch.from_numpy(si.send_blocks(P, m, si.BASE_SEED + 8).reshape(-1)).to(dev)
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    plan.allgather(send, recv)
    assert plan.status() == sp.OK
    view = recv.view(P, P * m)
    step = max(1, (256 << 20) // (P * m))
    for r0 in range(0, P, step):
        assert bool((view[r0:r0 + step] == send).all()), (P, m, r0)
    plan.destroy()
