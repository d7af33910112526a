"""A seeded random walk over the whole matrix: algorithm x executor x engine x communicator size x
block size x misalignment of each buffer, every case compared with the oracle over the complete
receive (and working) buffers, guard bands and the untouched send buffer included.  The fixed matrices
of test_gpu_parity.py choose their corners by hand; this one does not choose."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2109_08751_b200 as sp
from test_gpu_parity import run_case, is_pow2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda", 0)


ALGOS = [sp.ALGO_SPARBIT, sp.ALGO_SPARBIT, sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK,
         sp.ALGO_NEIGHBOR_EXCHANGE]
EXECS = [sp.EXEC_AUTO, sp.EXEC_PERSISTENT, sp.EXEC_GRAPH, sp.EXEC_STREAM, sp.EXEC_FLOW, sp.EXEC_MIRROR, sp.EXEC_MIRROR]
COPIES = [sp.COPY_AUTO, sp.COPY_VECTOR, sp.COPY_BULK]
BLOCKS = [1, 2, 3, 4, 6, 8, 12, 16, 17, 24, 32, 48, 64, 100, 128, 200, 256, 272, 500, 512, 1000, 1024, 1040, 2048, 4096,
          4100, 8192, 16384, 20000]


@pytest.mark.parametrize("chunk", range(8))
def test_random_cases(dev, chunk):
    rng = np.random.default_rng(20210908 + chunk)
    done = 0
    while done < 40:
        algo = ALGOS[rng.integers(len(ALGOS))]
        P = int(rng.choice([int(rng.integers(1, 20)), int(rng.integers(20, 70)), int(rng.integers(70, 300))],
                           p=[0.45, 0.4, 0.15]))
        if algo == sp.ALGO_RECURSIVE_DOUBLING:
            P = 1 << int(rng.integers(0, 9))
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            P += 1
        if algo in (sp.ALGO_RING, sp.ALGO_NEIGHBOR_EXCHANGE) and P > 64:
            P = 2 * int(rng.integers(1, 33))    # keep the linear schedules short
        m = int(BLOCKS[rng.integers(len(BLOCKS))])
        if P * P * m > (96 << 20):              # the oracle compares every byte: bound the case
            continue
        exec_mode = EXECS[rng.integers(len(EXECS))]
        copy = COPIES[rng.integers(len(COPIES))]
        shifts = [int(rng.choice([0, 0, 1, 2, 4, 8, 16, 24])) for _ in range(3)]
        tune = None
        if exec_mode == sp.EXEC_FLOW and rng.integers(2):
            tune = {sp.TUNE_FLOW_MIN_PASS_SPANS: int(rng.choice([0, 1, 40])),
                    sp.TUNE_FLOW_COOPERATIVE: int(rng.integers(2)),
                    # two vectors per lane, or four wherever blocks are long enough for it
                    sp.TUNE_FLOW_WIDE_MAX_MOVED_BYTES: 0 if done % 2 else 10 ** 12}
        if exec_mode == sp.EXEC_MIRROR and rng.integers(2):
            tune = {sp.TUNE_MIRROR_CTA_VECTORS: int(rng.choice([16, 64, 256, 4096])),
                    sp.TUNE_MIRROR_THREAD_VECTORS: int(rng.choice([1, 2, 4, 8])),
                    sp.TUNE_MIRROR_MAX_BYTES: int(rng.choice([0, 4096, 65536]))}
        assert not (algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P))
        run_case(dev, P, m, algo, exec_mode, copy, 1000 * chunk + done, iters=2, shift_send=shifts[0],
                 shift_recv=shifts[1], shift_work=shifts[2], tune=tune)
        done += 1
