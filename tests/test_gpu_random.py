"""Randomised GPU parity: seeded draws over algorithm, P, block size, executor, engine and
buffer alignment, each compared bit for bit with the oracle (sentinel, guard bands and a Bruck
workspace included).  The draws are reproducible from the seed in the test id."""
import numpy as np
import pytest

import seeded_inputs as si
import paper_2109_08751_b200 as sp
from test_gpu_parity import run_case

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    return torch.device("cuda:0")


def draw(seed):
    rng = np.random.default_rng(seed)
    algo = int(rng.integers(0, 5))
    P = int(rng.integers(1, 97))
    if algo == sp.ALGO_RECURSIVE_DOUBLING:
        P = 1 << int(rng.integers(0, 7))
    if algo == sp.ALGO_NEIGHBOR_EXCHANGE:
        P = 2 * int(rng.integers(1, 49))
    if algo == sp.ALGO_RING:
        P = min(P, 40)
    kind = int(rng.integers(0, 4))
    if kind == 0:
        m = int(rng.integers(1, 65))                       # tiny, any size
    elif kind == 1:
        m = 16 * int(rng.integers(1, 257))                 # multiples of 16 up to 4 KiB
    elif kind == 2:
        m = int(rng.integers(1, 20000))                    # anything
    else:
        m = 16 * int(rng.integers(256, 3000))              # 4 .. 47 KiB, several bulk chunks
    exec_mode = int(rng.integers(0, 5))
    copy = int(rng.integers(0, 3))
    shifts = [int(rng.choice([0, 0, 0, 16, 8, 4, 2, 1, 3])) for _ in range(3)]
    return algo, P, m, exec_mode, copy, shifts


@pytest.mark.parametrize("seed", range(60))
def test_random_case(dev, seed):
    algo, P, m, exec_mode, copy, shifts = draw(1000 + seed)
    run_case(dev, P, m, algo, exec_mode, copy, si.BASE_SEED + seed, iters=1,
             shift_send=shifts[0], shift_recv=shifts[1], shift_work=shifts[2])
