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


def full_compare(dev, P, m, algo, exec_mode, copy, seed, iters=2):
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


def test_config3_auto_is_what_the_benchmark_runs(dev):
    full_compare(dev, 128, 64 * 1024, sp.ALGO_SPARBIT, sp.EXEC_AUTO, sp.COPY_AUTO, si.BASE_SEED + 3, iters=1)


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
