"""Host-side tests of the CUDA library that need no GPU: the C ABI exports what the header
declares, the compact per-phase descriptors expand to exactly the oracle's message sets, and
argument errors are caught on the host."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
import paper_2109_08751_b200 as sp
from paper_2109_08751_b200 import binding

ROOT = Path(__file__).resolve().parent.parent
ALGOS = [sp.ALGO_SPARBIT, sp.ALGO_RING, sp.ALGO_RECURSIVE_DOUBLING, sp.ALGO_BRUCK, sp.ALGO_NEIGHBOR_EXCHANGE]


def is_pow2(p):
    return p & (p - 1) == 0


def test_library_exports_every_declared_symbol():
    header = (ROOT / "include" / "sparbit.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sparbit_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.SYMBOLS), declared ^ set(binding.SYMBOLS)
    lib = ctypes.CDLL(str(ROOT / "paper_2109_08751_b200" / "libsparbit_b200.so"))
    for name in declared:
        assert hasattr(lib, name), name


def as_set(msgs):
    return {tuple(int(x) for x in m) for m in msgs}


def test_binding_constants_match_the_header():
    """Every SPARBIT_* enumerator of the header has the same value under the binding's name for
    it (SPARBIT_ERR_ARG -> ERR_ARG ...): the binding spells the numbers out a second time."""
    import re
    header = (ROOT / "include" / "sparbit.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    seen = 0
    for body in re.findall(r"enum\s*\{(.*?)\}", header, flags=re.S):
        for name, value in re.findall(r"SPARBIT_([A-Z0-9_]+)\s*=\s*(-?\d+)", body):
            if name.endswith("_"):
                continue   # counts, not part of the binding
            assert hasattr(sp, name), name
            assert getattr(sp, name) == int(value), name
            seen += 1
    assert seen >= 45


@pytest.mark.parametrize("algo", ALGOS)
def test_descriptors_expand_to_oracle_message_sets(algo):
    """Per phase, the library's messages equal the oracle's as a set (order inside a phase is free)."""
    for P in list(range(1, 41)) + [64, 100, 127, 128, 129, 255, 256]:
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        if algo == sp.ALGO_RING and P > 64:
            continue
        plan = sp.Plan(P, 16, algo)
        ref = oracle.Plan(algo, P)
        assert plan.num_steps == ref.num_steps
        assert plan.last_phase == ref.last_phase
        for ph in range(-1, ref.last_phase + 1):
            got = plan.messages(ph)
            want = ref.phase_messages(ph)
            assert len(got) == len(want), (algo, P, ph)
            assert as_set(got) == as_set(want), (algo, P, ph)
        plan.destroy()


def test_sparbit_p1000_message_sets():
    plan = sp.Plan(1000, 1024)
    ref = oracle.Plan(oracle.SPARBIT, 1000)
    for ph in range(-1, ref.last_phase + 1):
        got = np.sort(plan.messages(ph), order=list(binding.MSG_DTYPE.names))
        want = np.sort(ref.phase_messages(ph), order=list(oracle.MSG_DTYPE.names))
        assert np.array_equal(got.view(np.int32), want.view(np.int32)), ph


@pytest.mark.parametrize("P", [2, 5, 6, 8, 13, 21, 256, 1000])
def test_step_info_matches_oracle_counts(P):
    plan = sp.Plan(P, 64)
    ref = oracle.Plan(oracle.SPARBIT, P)
    K = plan.num_steps
    held = 1
    for s in range(K):
        d, n, ig = plan.step_info(s)
        assert d == 2 ** (K - 1 - s)
        assert n == len(ref.phase_messages(s)) // P
        assert ig == held - n          # what is withheld is what was held but not sent
        held += n
    assert held == P


def test_plan_errors():
    out = ctypes.c_void_p()
    lib = binding.lib
    assert lib.sparbit_plan_create(0, 16, 0, 0, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create(-3, 16, 0, 0, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create(8, 16, 9, 0, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create(8, 16, 0, 17, ctypes.byref(out)) == sp.ERR_ARG
    assert lib.sparbit_plan_create(8, 16, 0, 0, None) == sp.ERR_ARG
    assert lib.sparbit_plan_create(6, 16, sp.ALGO_RECURSIVE_DOUBLING, 0, ctypes.byref(out)) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_plan_create(13, 16, sp.ALGO_RECURSIVE_DOUBLING, 0, ctypes.byref(out)) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_plan_create(7, 16, sp.ALGO_NEIGHBOR_EXCHANGE, 0, ctypes.byref(out)) == sp.ERR_UNSUPPORTED
    assert lib.sparbit_plan_create(1 << 20, 1 << 40, 0, 0, ctypes.byref(out)) == sp.ERR_OVERFLOW
    assert lib.sparbit_plan_create((1 << 24) + 1, 1, 0, 0, ctypes.byref(out)) == sp.ERR_OVERFLOW
    assert lib.sparbit_plan(0, 16) is None
    assert lib.sparbit_plan_destroy(None) == sp.OK
    assert lib.sparbit_plan_num_steps(None) == -1


def test_argument_checks_happen_before_any_launch():
    """These return on the host before the first CUDA call, so they work without a GPU."""
    lib = binding.lib
    plan = sp.Plan(8, 64)
    h = plan._h
    assert lib.sparbit_allgather(None, 1, 2, None) == sp.ERR_ARG
    assert lib.sparbit_allgather(h, None, 4096, None) == sp.ERR_ARG
    assert lib.sparbit_allgather(h, 4096, None, None) == sp.ERR_ARG
    # send [4096, 4608) overlaps recv [4352, ...)
    assert lib.sparbit_allgather(h, 4096, 4352, None) == sp.ERR_ALIAS
    assert lib.sparbit_allgather_steps(h, 4096, 1 << 20, None, 2, 1) == sp.ERR_ARG
    assert lib.sparbit_allgather_steps(h, 4096, 1 << 20, None, -2, 1) == sp.ERR_ARG
    assert lib.sparbit_allgather_steps(h, 4096, 1 << 20, None, 0, 3) == sp.ERR_ARG
    assert lib.sparbit_plan_step_info(h, 3, None, None, None) == sp.ERR_ARG
    assert lib.sparbit_plan_set_copy_path(h, 7) == sp.ERR_ARG
    # zero-byte blocks: a valid no-op, even with null buffers
    z = sp.Plan(8, 0)
    assert lib.sparbit_allgather(z._h, None, None, None) == sp.OK
    # Bruck needs its workspace
    b = sp.Plan(6, 64, sp.ALGO_BRUCK)
    assert b.workspace_bytes == 6 * 6 * 64
    assert lib.sparbit_allgather(b._h, 4096, 1 << 20, None) == sp.ERR_WORKSPACE
    assert lib.sparbit_plan_set_workspace(b._h, 1 << 22, 100) == sp.ERR_WORKSPACE
    assert lib.sparbit_plan_set_workspace(b._h, 1 << 20, 6 * 6 * 64) == sp.OK
    assert lib.sparbit_allgather(b._h, 4096, 1 << 20, None) == sp.ERR_ALIAS   # workspace == recv
    assert sp.Plan(8, 64).workspace_bytes == 0


def test_strerror_covers_every_code():
    texts = {binding.lib.sparbit_strerror(c).decode() for c in range(0, 10)}
    assert len(texts) == 10 and "unknown error" not in texts
    assert binding.lib.sparbit_strerror(99).decode() == "unknown error"


def test_exec_mode_resolution():
    assert sp.Plan(8, 64).exec_mode == sp.EXEC_MIRROR            # 4 KiB of receive buffers: one CTA, on chip
    assert sp.Plan(32, 64).exec_mode == sp.EXEC_MIRROR           # 64 KiB
    assert sp.Plan(45, 512).exec_mode == sp.EXEC_MIRROR          # 1 MiB, no power of two divides 45: a cluster of CTAs
    assert sp.Plan(253, 1).exec_mode == sp.EXEC_MIRROR           # 63 KiB but 32 Ki one-byte vectors: a cluster too
    assert sp.Plan(32, 128).exec_mode == sp.EXEC_MIRROR          # 128 KiB, 4 Ki vectors in the largest pass: a cluster beats the
                                                                 # chain even with the chain's first four passes in one kernel
    assert sp.Plan(64, 512).exec_mode == sp.EXEC_STREAM          # 2 MiB, 64 Ki vectors: the chain, three passes as 8 groups of 8
                                                                 # ranks, then three: kernel by kernel, not as a graph
    assert sp.Plan(128, 64).exec_mode == sp.EXEC_STREAM          # 1 MiB: the chain, four passes as 8 groups of 16, then three
    assert sp.Plan(256, 64).exec_mode == sp.EXEC_STREAM          # 4 MiB: the chain, five passes as 8 groups of 32, then three
    assert sp.Plan(128, 128).exec_mode == sp.EXEC_STREAM         # 2 MiB
    assert sp.Plan(13, 4096).exec_mode == sp.EXEC_MIRROR         # 676 KiB of 4 KiB blocks, odd P: a cluster
    assert sp.Plan(8, 8192).exec_mode == sp.EXEC_STREAM          # 512 KiB of larger blocks: the chain, three launches
    assert sp.Plan(8, 8192, exec_mode=sp.EXEC_MIRROR).exec_mode == sp.EXEC_MIRROR   # but it fits, on request
    assert sp.Plan(6, 4096, sp.ALGO_BRUCK).exec_mode == sp.EXEC_MIRROR     # 144 KiB, and as much of working buffers
    assert sp.Plan(8, 64, sp.ALGO_BRUCK).exec_mode == sp.EXEC_MIRROR
    assert sp.Plan(256, 65536).exec_mode == sp.EXEC_GRAPH         # 8.6 GB moved: chain + bulk engine
    assert sp.Plan(128, 65536).exec_mode == sp.EXEC_FLOW          # 2.1 GB moved
    assert sp.Plan(1000, 1024).exec_mode == sp.EXEC_FLOW          # 2.0 GB moved
    assert sp.Plan(256, 4096).exec_mode == sp.EXEC_FLOW           # 0.53 GB moved
    assert sp.Plan(128, 8192).exec_mode == sp.EXEC_GRAPH          # 0.27 GB moved, seven launches: a graph
    assert sp.Plan(512, 2048).exec_mode == sp.EXEC_FLOW           # 1.07 GB moved
    assert sp.Plan(300, 1024).exec_mode == sp.EXEC_GRAPH          # 0.18 GB moved, nine launches: a graph
    assert sp.Plan(128, 65520).exec_mode == sp.EXEC_GRAPH         # blocks off 128-byte lines stay on the bulk engine
    assert sp.Plan(128, 65520, ).exec_mode != sp.Plan(128, 65536).exec_mode
    assert sp.Plan(1000, 1008).exec_mode == sp.EXEC_FLOW          # ... where COPY_AUTO would pick it (m >= 8 KiB)
    assert sp.Plan(40000, 1).exec_mode == sp.EXEC_GRAPH           # blocks shorter than a warp row, 16 launches
    short = sp.Plan(128, 64)
    short.set_tunable(sp.TUNE_STREAM_MAX_LAUNCHES, 0)             # never kernel by kernel
    assert short.exec_mode == sp.EXEC_GRAPH
    assert sp.Plan(256, 65536, exec_mode=sp.EXEC_PERSISTENT).exec_mode == sp.EXEC_PERSISTENT


def test_engine_thresholds_are_plan_fields():
    plan = sp.Plan(8, 64)
    assert plan.get_tunable(sp.TUNE_BULK_MIN_BLOCK_BYTES) == 8192
    assert plan.get_tunable(sp.TUNE_BULK_MIN_MOVED_BYTES) == 10 ** 9
    plan.set_tunable(sp.TUNE_BULK_MIN_BLOCK_BYTES, 4096)
    assert plan.get_tunable(sp.TUNE_BULK_MIN_BLOCK_BYTES) == 4096
    assert plan.get_tunable(sp.TUNE_VEC_DENSE_MAX_RECV_BYTES) == 256 << 20
    with pytest.raises(sp.binding.SparbitError):
        plan.set_tunable(99, 1)


def test_environment_overrides_only_the_automatic_choice(monkeypatch):
    monkeypatch.setenv("SPARBIT_EXEC", "persistent")
    assert sp.Plan(8, 64).exec_mode == sp.EXEC_PERSISTENT
    assert sp.Plan(8, 64, exec_mode=sp.EXEC_STREAM).exec_mode == sp.EXEC_STREAM   # explicit wins
    assert sp.Plan.create_v([16, 32]).exec_mode == sp.EXEC_PERSISTENT
    monkeypatch.setenv("SPARBIT_EXEC", "flow")
    assert sp.Plan(8, 64).exec_mode == sp.EXEC_FLOW
    assert sp.Plan.create_v([16, 32]).exec_mode == sp.EXEC_MIRROR                 # flow is not offered there: AUTO's own pick
    assert sp.Plan.create_v([70000, 80000]).exec_mode == sp.EXEC_STREAM              # one launch: a plain one
    monkeypatch.setenv("SPARBIT_EXEC", "nonsense")
    assert sp.Plan(8, 64).exec_mode == sp.EXEC_MIRROR


@pytest.mark.parametrize("algo", ALGOS)
def test_descriptors_are_race_free_and_in_bounds(algo):
    """The library's own host-side check of what the kernels execute (fused first pass included)."""
    for P in list(range(1, 70)) + [100, 127, 128, 253, 256, 1000]:
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        if algo == sp.ALGO_RING and P > 128:
            continue
        sp.Plan(P, 16, algo).validate()
    sp.Plan.create_v([16, 0, 32, 48, 8, 8, 0]).validate()
    with pytest.raises(sp.SparbitError) as e:
        sp.Plan(10000, 16).validate()
    assert e.value.code == sp.ERR_LIMIT


@pytest.mark.parametrize("algo", ALGOS)
def test_flow_units_and_counters_are_consistent(algo):
    """The flow executor's bookkeeping, checked on the host for many communicator sizes, block
    sizes (one span, ragged spans, many spans per block), vector widths and numbers of warps.
    With one warp every pass is large enough for the flow kernel (it then takes the whole
    collective, or its last 32 passes); with more warps the small leading passes are left to
    per-pass kernels, more of them the more warps there are."""
    ran = 0
    for P in list(range(1, 34)) + [61, 64, 100, 128, 253, 256, 1000]:
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        for m, vb in ((512, 16), (1040, 16), (4096, 16), (65536, 16), (1000, 8), (36, 1)):
            if P > 256 and m > 4096:
                continue
            plan = sp.Plan(P, m, algo)
            plan.set_tunable(sp.TUNE_FLOW_MIN_PASS_SPANS, 0)   # a pass needs one span per resident warp
            passes = plan.last_phase + 2 - (1 if algo != sp.ALGO_BRUCK and P > 1 else 0)   # fused first pass
            # spans of four vectors per lane (blocks of 128 vectors and more, up to the given bytes
            # moved) and of two
            for wide_below in (10 ** 12, 0):
                plan.set_tunable(sp.TUNE_FLOW_WIDE_MAX_MOVED_BYTES, wide_below)
                firsts = []
                for warps in (1, 64, 4736):
                    code = plan.validate_flow(vb, warps)
                    assert code in (sp.OK, sp.ERR_UNSUPPORTED)
                    if warps == 1:
                        assert code == sp.OK and plan.first_flow_pass == max(0, passes - 32), (algo, P, m)
                    firsts.append(plan.first_flow_pass if code == sp.OK else passes)
                    ran += code == sp.OK
                assert firsts == sorted(firsts), (algo, P, m, firsts)
            plan.destroy()
    assert ran > 120
    assert sp.Plan(8, 64).validate_flow(16, 1) == sp.ERR_UNSUPPORTED   # blocks shorter than a warp row
    big = sp.Plan(256, 4096)
    assert big.validate_flow(16, 4736) == sp.OK and big.first_flow_pass == 0   # by default every pass
    big.set_tunable(sp.TUNE_FLOW_MIN_PASS_SPANS, 0)
    assert big.get_tunable(sp.TUNE_FLOW_WIDE_MAX_MOVED_BYTES) == 9 * 10 ** 8   # 0.53 GB moved: spans of 2 KiB
    assert big.validate_flow(16, 4736) == sp.OK and big.first_flow_pass == 4   # 8192 of them in pass 4
    big.set_tunable(sp.TUNE_FLOW_WIDE_MAX_MOVED_BYTES, 0)                      # spans of 1 KiB
    assert big.validate_flow(16, 4736) == sp.OK and big.first_flow_pass == 3   # 8192 spans in pass 3


@pytest.mark.parametrize("algo", ALGOS)
def test_every_rank_sends_and_receives_the_same_number_of_blocks_in_a_pass(algo):
    """What the cluster form of the mirror executor counts on: it arms, per pass, an mbarrier in
    every CTA with the bytes that CTA's ranks will receive, computed as ranks x blocks-per-rank x
    block size.  That is right only if, in every pass, every rank receives exactly as many blocks
    as every rank sends (one slot each, no slot twice)."""
    for P in list(range(1, 40)) + [61, 64, 100, 128, 253, 256]:
        if algo == sp.ALGO_RECURSIVE_DOUBLING and not is_pow2(P):
            continue
        if algo == sp.ALGO_NEIGHBOR_EXCHANGE and P % 2:
            continue
        plan = sp.Plan(P, 16, algo)
        for phase in range(-1, plan.last_phase + 1):
            msgs = plan.messages(phase)
            if len(msgs) == 0:
                continue
            sent = np.bincount(msgs["src_rank"], minlength=P)
            got = np.bincount(msgs["dst_rank"], minlength=P)
            assert (sent == sent[0]).all() and (got == sent[0]).all(), (algo, P, phase)
            slots = set(zip(msgs["dst_space"].tolist(), msgs["dst_rank"].tolist(), msgs["dst_slot"].tolist()))
            assert len(slots) == len(msgs), (algo, P, phase)
        plan.destroy()
