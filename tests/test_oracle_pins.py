"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

None of these tests re-types the oracle's own formulae to compare it with itself: each one comes
at the schedule from another side (the plain definition of the result, the paper's worked
examples, an independent recursive construction of the binomial trees, counting arguments).
"""
import math

import numpy as np
import pytest

import oracle
import seeded_inputs as si

ALL_P = list(range(1, 65))
ALGOS = [oracle.SPARBIT, oracle.RING, oracle.RECURSIVE_DOUBLING, oracle.BRUCK, oracle.NEIGHBOR_EXCHANGE]


def defined_for(algo, P):
    """Recursive doubling: powers of two only; neighbor exchange: even P only (Section II-A)."""
    if algo == oracle.RECURSIVE_DOUBLING:
        return P & (P - 1) == 0
    if algo == oracle.NEIGHBOR_EXCHANGE:
        return P % 2 == 0
    return True


def is_pow2(p):
    return p & (p - 1) == 0


def ceil_log2(p):
    return (p - 1).bit_length()


def plan(algo, P):
    return oracle.Plan(algo, P)


def step_sets(pl, spaces=False):
    """per step: set of (src, dst, src_slot, dst_slot) for communication steps only"""
    out = []
    for s in range(pl.num_steps):
        ms = pl.phase_messages(s)
        out.append({(int(m["src_rank"]), int(m["dst_rank"]), int(m["src_slot"]), int(m["dst_slot"]))
                    for m in ms})
        assert len(out[-1]) == len(ms)
    return out


# ------------------------------------------------------------------ the result's plain definition
@pytest.mark.parametrize("algo", ALGOS)
def test_final_state_is_rank_ordered_concatenation(algo):
    """Section II: slot j of every receive buffer holds the block sent by rank j."""
    for P in ALL_P:
        if not defined_for(algo, P):
            continue
        for m in (1, 4, 7, 16):
            send = si.send_blocks(P, m, seed=si.BASE_SEED + P)
            recv, _ = oracle.allgather(algo, P, m, send)
            want = np.broadcast_to(send.reshape(1, P * m), (P, P * m))
            assert np.array_equal(recv, want), (algo, P, m)


def test_blocks_are_distinguishable():
    """The input recipe: no two send blocks, and no two words of a block, compare equal."""
    send = si.send_blocks(64, 16, seed=7).view("<u4")
    assert len(np.unique(send)) == send.size


# ------------------------------------------------------------------ step counts (cost formulae)
@pytest.mark.parametrize("P", ALL_P + [100, 128, 255, 256, 257, 1000])
def test_step_counts(P):
    assert plan(oracle.SPARBIT, P).num_steps == ceil_log2(P)          # ceil(log2 p) alpha
    assert plan(oracle.BRUCK, P).num_steps == ceil_log2(P)            # ceil(log2 p) alpha
    if P <= 257:
        assert plan(oracle.RING, P).num_steps == P - 1                # (p - 1) alpha
    if is_pow2(P):
        assert plan(oracle.RECURSIVE_DOUBLING, P).num_steps == int(math.log2(P))


@pytest.mark.parametrize("P", [3, 5, 6, 7, 13, 21, 100])
def test_recursive_doubling_only_for_powers_of_two(P):
    with pytest.raises(oracle.OracleError):
        plan(oracle.RECURSIVE_DOUBLING, P)


def test_zero_ranks_is_an_error():
    with pytest.raises(oracle.OracleError):
        plan(oracle.SPARBIT, 0)


# ------------------------------------------------------------------ power-of-two behaviour
@pytest.mark.parametrize("P", [2, 4, 8, 16, 32, 64, 256])
def test_sparbit_power_of_two_steps(P):
    """Section III-B: on step s every process sends and receives 2^s blocks to and from peers
    2^(log2 p - (s+1)) away in each direction."""
    pl = plan(oracle.SPARBIT, P)
    L = int(math.log2(P))
    for s, msgs in enumerate(step_sets(pl)):
        d = 2 ** (L - (s + 1))
        sent = np.zeros(P, int)
        got = np.zeros(P, int)
        for src, dst, a, b in msgs:
            assert dst == (src + d) % P
            sent[src] += 1
            got[dst] += 1
        assert (sent == 2 ** s).all() and (got == 2 ** s).all()


# ------------------------------------------------------------------ the paper's P = 5 example
def parse_golden(path):
    rows = []
    for line in path.read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(line)
    return rows


def test_sparbit_p5_walkthrough(golden_dir):
    rows = parse_golden(golden_dir / "sparbit_p5_walkthrough.txt")
    P = 5
    pl = plan(oracle.SPARBIT, P)
    sets = step_sets(pl)
    steps = [tuple(map(int, r.split()[1:])) for r in rows if r.startswith("step")]
    assert pl.num_steps == len(steps) == 3
    sends = {int(r.split()[1]): [int(x) for x in r.split(":")[1].split()] for r in rows if r.startswith("sends")}
    recvs = {int(r.split()[1]): [int(x) for x in r.split(":")[1].split()] for r in rows if r.startswith("recvs")}
    for s, d, n, _ign in steps:
        want = set()
        for r in range(P):
            for k in sends[s]:
                blk = (r - k) % P
                want.add((r, (r + d) % P, blk, blk))
        assert sets[s] == want
        assert len(sends[s]) == n
        # the same step seen from the receivers
        for r in range(P):
            got = sorted((r - b) % P for (src, dst, a, b) in sets[s] if dst == r)
            assert got == sorted(recvs[s])
    # rank 0's held set, step by step, from a real run with sentinel-filled buffers
    held_rows = [r for r in rows if r.startswith("held")]
    m = 8
    send = si.send_blocks(P, m, seed=5)
    for row in held_rows:
        head, blocks = row.split(":")
        want = sorted(int(x) for x in blocks.split())
        last = int(head.split()[3]) if "after" in head else -1
        recv, _ = oracle.allgather(oracle.SPARBIT, P, m, send, last=last)
        r0 = recv[0].reshape(P, m)
        have = [b for b in range(P) if not (r0[b] == si.SENTINEL).all()]
        assert have == want
        for b in have:
            assert np.array_equal(r0[b], send[b])


def test_sparbit_p21_decomposition(golden_dir):
    rows = parse_golden(golden_dir / "sparbit_p21_decomposition.txt")
    P = 21
    subtrees = [int(x) for x in rows[0].split()[1:]]
    assert sum(subtrees) == P
    behaviour = {int(r.split()[1]): r.split()[2] for r in rows[1:]}
    pl = plan(oracle.SPARBIT, P)
    sets = step_sets(pl)
    held = 1  # blocks a rank holds before the step
    for s, msgs in enumerate(sets):
        d = 2 ** (pl.num_steps - 1 - s)
        per_rank = len(msgs) // P
        assert len(msgs) == per_rank * P
        if behaviour[d] == "expand":
            assert per_rank == held          # every held block is sent
            assert d in subtrees
        else:
            assert per_rank == held - 1      # exactly one block withheld
        held += per_rank
    assert held == P


# ------------------------------------------------------------------ independent construction
def binomial_tree_edges(P):
    """Section III-A: the root sends to the rank half the (power-of-two padded) size away and
    both halves recurse in parallel; sends to ranks >= p are dropped.  Returns (step, src, dst)
    with ranks relative to the root, built by literal recursion (no bit tricks)."""
    size = 1
    while size < P:
        size *= 2
    edges = []

    def rec(lo, sz, step):
        if sz == 1:
            return
        half = sz // 2
        if lo + half < P:
            edges.append((step, lo, lo + half))
            rec(lo + half, half, step + 1)
        rec(lo, half, step + 1)

    rec(0, size, 0)
    return edges


@pytest.mark.parametrize("P", ALL_P + [100, 127, 129, 255, 256, 257])
def test_sparbit_is_p_shifted_binomial_trees(P):
    """Section III-B: every process roots a binomial tree for its own block, the trees being the
    same tree shifted by the root's rank with wrap-around; Sparbit is exactly their union."""
    edges = binomial_tree_edges(P)
    assert len(edges) == P - 1
    want = [set() for _ in range(ceil_log2(P))]
    for root in range(P):
        for step, a, b in edges:
            want[step].add(((root + a) % P, (root + b) % P, root, root))
    assert step_sets(plan(oracle.SPARBIT, P)) == want


# ------------------------------------------------------------------ counting invariants
@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("P", [1, 2, 3, 5, 6, 8, 13, 16, 21, 37, 64])
def test_each_block_received_exactly_once(algo, P):
    """Every rank receives (p - 1) blocks, one from each other origin, none twice."""
    if not defined_for(algo, P):
        return
    pl = plan(algo, P)
    msgs = pl.messages
    comm = msgs[msgs["src_rank"] != msgs["dst_rank"]]
    per_dst = np.bincount(comm["dst_rank"], minlength=P)
    assert (per_dst == P - 1).all()
    assert len(comm) == P * (P - 1)
    # no (dst, space, slot) is written twice over the whole collective
    keys = set()
    for m in msgs:
        k = (int(m["dst_rank"]), int(m["dst_space"]), int(m["dst_slot"]))
        assert k not in keys
        keys.add(k)
    # inside one phase nothing is both read and written
    for ph in range(-1, pl.last_phase + 1):
        pm = pl.phase_messages(ph)
        reads = {(int(m["src_rank"]), int(m["src_space"]), int(m["src_slot"])) for m in pm}
        writes = {(int(m["dst_rank"]), int(m["dst_space"]), int(m["dst_slot"])) for m in pm}
        assert not (reads & writes)


@pytest.mark.parametrize("P", ALL_P + [100, 1000])
def test_sparbit_blocks_per_step_closed_form(P):
    """Counting argument: before the step at distance d a rank holds the blocks of the ranks
    0, d', 2d', ... behind it (d' = 2d), i.e. ceil(P / 2d) of them; after it, ceil(P / d).  The
    difference is what it received, which equals what it sent (the pattern is shift-invariant)."""
    pl = plan(oracle.SPARBIT, P)
    K = pl.num_steps
    total = 0
    for s in range(K):
        d = 2 ** (K - 1 - s)
        n = len(pl.phase_messages(s))
        assert n == P * (-(-P // d) - -(-P // (2 * d)))
        total += n
    assert total == P * (P - 1)


@pytest.mark.parametrize("P", [5, 6, 13, 21, 64])
def test_sparbit_held_sets_after_each_step(P):
    """After the step at distance d, rank r holds exactly the blocks {(r - t d) mod P}."""
    m = 4
    send = si.send_blocks(P, m, seed=99)
    K = ceil_log2(P)
    for s in range(K):
        d = 2 ** (K - 1 - s)
        recv, _ = oracle.allgather(oracle.SPARBIT, P, m, send, last=s)
        for r in range(P):
            row = recv[r].reshape(P, m)
            have = {b for b in range(P) if not (row[b] == si.SENTINEL).all()}
            want = {(r - t * d) % P for t in range(-(-P // d))}
            assert have == want
            for b in have:
                assert np.array_equal(row[b], send[b])


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 6, 7, 8, 12, 13, 16, 21, 33, 64])
def test_ignore_pattern_follows_binary_representation(P):
    """Section III-B: steps below the lowest set bit of p never withhold; the step at the lowest
    set bit withholds; above it, a step withholds iff its bit of p is unset."""
    pl = plan(oracle.SPARBIT, P)
    K = pl.num_steps
    low = P & -P
    held = 1
    for s in range(K):
        d = 2 ** (K - 1 - s)
        per_rank = len(pl.phase_messages(s)) // P
        if d < low:
            withhold = False
        elif d == low:
            withhold = True
        else:
            withhold = (P & d) == 0
        assert per_rank == held - (1 if withhold else 0)
        held += per_rank


# ------------------------------------------------------------------ comparators
@pytest.mark.parametrize("P", [2, 3, 5, 6, 8, 13, 16])
def test_ring_shape(P):
    pl = plan(oracle.RING, P)
    for s, msgs in enumerate(step_sets(pl)):
        assert len(msgs) == P                       # one block per rank per step
        for src, dst, a, b in msgs:
            assert dst == (src + 1) % P and a == b
    # the block sent first is the rank's own
    assert {(r, (r + 1) % P, r, r) for r in range(P)} == step_sets(pl)[0]


@pytest.mark.parametrize("P", [2, 4, 8, 16, 64])
def test_recursive_doubling_shape(P):
    pl = plan(oracle.RECURSIVE_DOUBLING, P)
    for s, msgs in enumerate(step_sets(pl)):
        assert len(msgs) == P * 2 ** s              # data doubles
        for src, dst, a, b in msgs:
            assert dst == src ^ (1 << s) and a == b


@pytest.mark.parametrize("P", [2, 3, 5, 6, 8, 13, 16, 21, 100])
def test_bruck_shape(P):
    pl = plan(oracle.BRUCK, P)
    F = P.bit_length() - 1
    sets = step_sets(pl)
    for s, msgs in enumerate(sets):
        dist = 1 << s
        per_rank = dist if s < F else P - (1 << F)  # the additional step sends p - 2^floor blocks
        assert len(msgs) == P * per_rank
        for src, dst, a, b in msgs:
            assert dst == (src - dist) % P
            assert 0 <= a < per_rank                # "the first ... blocks"
    # rotation is purely local and touches every slot once
    rot = pl.phase_messages(pl.num_steps)
    assert len(rot) == P * P and (rot["src_rank"] == rot["dst_rank"]).all()


@pytest.mark.parametrize("P", [2, 4, 6, 8, 10, 14, 16, 30, 64, 100])
def test_neighbor_exchange_shape(P):
    """Section II-A: p/2 steps; on step s an even process r exchanges with r + (-1)^s and an odd
    one with r - (-1)^s, always pairwise; one block on the first step, two on all others, which
    adds up to the p - 1 blocks of the cost formula's bandwidth term."""
    pl = plan(oracle.NEIGHBOR_EXCHANGE, P)
    assert pl.num_steps == P // 2                      # p/2 alpha
    total = 0
    for s, msgs in enumerate(step_sets(pl)):
        per_rank = 1 if s == 0 else 2
        assert len(msgs) == P * per_rank
        partner = {}
        for src, dst, a, b in msgs:
            sign = (-1) ** s
            want = (src + sign) % P if src % 2 == 0 else (src - sign) % P
            assert dst == want and a == b
            partner[src] = dst
        assert all(partner[partner[r]] == r for r in range(P))   # exchanges are pairwise
        total += per_rank
    assert total == P - 1
    # the first step swaps the own blocks of the two neighbours
    assert step_sets(pl)[0] == {(r, r ^ 1, r, r) for r in range(P)}
    if P >= 4:
        # the second step sends the two blocks held so far: the pair {2k, 2k+1}
        assert {(a, src) for src, dst, a, b in step_sets(pl)[1]} == \
            {(2 * (r // 2) + j, r) for r in range(P) for j in (0, 1)}


@pytest.mark.parametrize("P", [3, 5, 7, 13, 21])
def test_neighbor_exchange_only_for_even_p(P):
    with pytest.raises(oracle.OracleError):
        plan(oracle.NEIGHBOR_EXCHANGE, P)


@pytest.mark.parametrize("P", [4, 8, 16, 64])
def test_sparbit_mirrors_bruck_distances(P):
    """Section III: same exchange semantics as Bruck with the distances taken in the opposite
    order, 2^(K-1) down to 1 instead of 1 up to 2^(K-1), data doubling either way."""
    sp = step_sets(plan(oracle.SPARBIT, P))
    br = step_sets(plan(oracle.BRUCK, P))
    sp_d = [{(dst - src) % P for src, dst, _, _ in s} for s in sp]
    br_d = [{(src - dst) % P for src, dst, _, _ in s} for s in br]
    assert sp_d == list(reversed(br_d))
    assert [len(s) for s in sp] == [len(s) for s in br]


# ------------------------------------------------------------------ execution variants
@pytest.mark.parametrize("algo", ALGOS)
def test_threaded_execution_matches_single_thread(algo):
    P, m = 16, 64
    send = si.send_blocks(P, m, seed=3)
    a, sa = oracle.allgather(algo, P, m, send, threads=1)
    b, sb = oracle.allgather(algo, P, m, send, threads=4)
    assert np.array_equal(a, b)
    if sa is not None:
        assert np.array_equal(sa, sb)


def test_partial_runs_compose():
    """Running phases one at a time from the same buffers equals one full run."""
    P, m = 13, 8
    send = si.send_blocks(P, m, seed=11).reshape(-1)
    for algo in (oracle.SPARBIT, oracle.BRUCK, oracle.RING):
        pl = plan(algo, P)
        recv = si.sentinel_buffer(P * P * m)
        scr = si.sentinel_buffer(P * P * m)
        for ph in range(-1, pl.last_phase + 1):
            pl.run(m, send, recv, scr, first=ph, last=ph)
        full, _ = oracle.allgather(algo, P, m, send)
        assert np.array_equal(recv.reshape(P, -1), full)


def test_zero_byte_blocks_are_a_no_op():
    recv, _ = oracle.allgather(oracle.SPARBIT, 8, 0, np.empty((8, 0), np.uint8))
    assert recv.shape == (8, 0)


# ------------------------------------------------------------------ tracing a slot back to its origin
@pytest.mark.parametrize("algo", ALGOS)
def test_trace_leads_back_to_the_owner_of_the_slot(algo):
    """Plan.trace follows the messages that fill (rank, slot) back to a send buffer.  Whatever
    the algorithm, the walk must end at the send block of rank `slot` (Section II: slot j holds
    rank j's block), start with the own-block copy of that rank, and be connected hop to hop."""
    for P in ALL_P:
        if not defined_for(algo, P):
            continue
        pl = plan(algo, P)
        for r in range(P):
            for b in range(P):
                path = pl.trace(r, b)
                assert int(path[0]["src_space"]) == oracle.SPACE_SEND
                assert int(path[0]["src_rank"]) == b, (algo, P, r, b)
                assert (int(path[-1]["dst_space"]), int(path[-1]["dst_rank"]), int(path[-1]["dst_slot"])) \
                    == (oracle.SPACE_RECV, r, b)
                for a, c in zip(path, path[1:]):
                    assert (int(a["dst_space"]), int(a["dst_rank"]), int(a["dst_slot"])) \
                        == (int(c["src_space"]), int(c["src_rank"]), int(c["src_slot"]))
                    assert int(a["phase"]) < int(c["phase"])


@pytest.mark.parametrize("P", ALL_P + [100, 272])
def test_sparbit_trace_has_one_hop_per_set_bit_of_the_distance(P):
    """Sections III-A/B: block b reaches rank b + k through the binomial tree rooted at b, i.e. by
    adding the set bits of k from the most significant down - popcount(k) messages after the
    own-block copy, at strictly decreasing distances that sum to k."""
    pl = plan(oracle.SPARBIT, P)
    pairs = [(r, b) for r in range(P) for b in range(P)] if P <= 64 else \
        [divmod(int(k), P) for k in si.sample_indices(400, P * P, seed=P)]
    for r, b in pairs:
        k = (r - b) % P
        path = pl.trace(r, b)
        hops = path[1:]
        assert len(hops) == bin(k).count("1"), (P, r, b)
        dists = [(int(h["dst_rank"]) - int(h["src_rank"])) % P for h in hops]
        assert dists == sorted(dists, reverse=True) and len(set(dists)) == len(dists)
        assert sum(dists) == k and all(d & (d - 1) == 0 for d in dists)
        assert all(int(h["src_slot"]) == b and int(h["dst_slot"]) == b for h in hops)
