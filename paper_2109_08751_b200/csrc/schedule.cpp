// Host schedule generator.
//
// Sparbit follows Algorithm 1 of the paper: lines 1-5 give the first distance and the bit vector
// of steps that withhold a block, the loop gives each step's distance d and message count
// data - ignore, and the state update (d >>= 1; data = 2*data - ignore) carries them forward.  A
// step's messages are not listed one by one: they are the copies (r, j) -> peer r + d, slot
// r - 2jd on both sides, which the PhaseDesc form states in O(1) bytes.  The counts are
// cross-checked against the counting form ceil(P/d) - ceil(P/2d) before a plan is accepted.
//
// Ring, neighbor exchange, recursive doubling and Bruck (Section II-A) are expressed in the same
// descriptor form.
#include "schedule.h"

#include <string.h>

namespace spb {

static int ceil_log2(uint64_t p) {
    int k = 0;
    while ((1ull << k) < p) k++;
    return k;
}

static int floor_log2(uint64_t p) {
    int k = 0;
    while ((2ull << k) <= p) k++;
    return k;
}

static PhaseDesc blank(uint64_t m) {
    PhaseDesc d;
    memset(&d, 0, sizeof d);
    d.copies = 1;
    d.run = 1;
    d.rank_mask = 0xFFFFFFFFu;
    d.copy_bytes = m;
    return d;
}

// own block: sendbuf[r] -> (space)[r][slot r or 0]
static PhaseDesc own_copy(uint64_t m, bool into_work) {
    PhaseDesc d = blank(m);
    d.src_space = SPACE_SEND;  // one slot per rank: slot 0
    d.dst_space = into_work ? SPACE_WORK : SPACE_RECV;
    d.dst_rcoef = into_work ? 0u : 1u;
    return d;
}

static bool steps_stay_in_range(const PhaseDesc& d, uint32_t P) {
    // (copies-1) * |step| < P keeps base + j*step inside (-P, 2P)
    uint64_t a = (uint64_t)(d.copies - 1) * (uint64_t)(d.src_step < 0 ? -(int64_t)d.src_step : d.src_step);
    uint64_t b = (uint64_t)(d.copies - 1) * (uint64_t)(d.dst_step < 0 ? -(int64_t)d.dst_step : d.dst_step);
    return a < P && b < P && d.src_off < P && d.dst_off < P && d.src_off_odd < P && d.dst_off_odd < P &&
           d.peer_add < P && d.peer_pre < P;
}

static int build_sparbit(uint32_t P, uint64_t m, Schedule& s) {
    const int K = ceil_log2(P);
    s.K = K;
    s.phases.push_back(own_copy(m, false));
    if (K == 0) return SCHED_OK;  // one rank: nothing to exchange
    // Algorithm 1, lines 1-5
    uint32_t data = 1, ignore = 0;
    uint32_t d = 1u << (K - 1);
    uint32_t last_ignore = (uint32_t)__builtin_ctz(P);
    uint32_t ignore_steps = (~(P >> last_ignore) | 1u) << last_ignore;
    for (int i = 0; i < K; i++) {
        if (d & ignore_steps) ignore = 1;
        const uint32_t n = data - ignore;
        // counting form: a rank holds ceil(P/2d) blocks before and ceil(P/d) after the step
        const uint32_t before = (uint32_t)((P + 2ull * d - 1) / (2ull * d));
        const uint32_t after = (P + d - 1) / d;
        if (data != before || n != after - before) return SCHED_INTERNAL;
        PhaseDesc ph = blank(m);
        ph.copies = n;
        ph.peer_add = d;                 // d <= 2^(K-1) < P
        ph.src_space = ph.dst_space = SPACE_RECV;
        ph.src_rcoef = ph.dst_rcoef = 1; // displacement (rank - 2jd) mod P, the same on both sides:
        ph.src_step = ph.dst_step = -(int32_t)(2 * d);  // receiver r+d stores at (r+d) - (2j+1)d
        if (!steps_stay_in_range(ph, P)) return SCHED_INTERNAL;
        s.phases.push_back(ph);
        s.steps.push_back({(int)d, (int)n, (int)ignore});
        d >>= 1;
        data = (data << 1) - ignore;
        ignore = 0;
    }
    if (data != P) return SCHED_INTERNAL;  // every rank ends up holding all P blocks
    return SCHED_OK;
}

static int build_ring(uint32_t P, uint64_t m, Schedule& s) {
    s.K = (int)P - 1;
    s.phases.push_back(own_copy(m, false));
    for (uint32_t st = 0; st + 1 < P; st++) {
        PhaseDesc ph = blank(m);  // r forwards the block of rank r - st to r + 1, same slot there
        ph.peer_add = 1 % P;
        ph.src_space = ph.dst_space = SPACE_RECV;
        ph.src_rcoef = ph.dst_rcoef = 1;
        ph.src_off = ph.dst_off = (P - st % P) % P;
        if (!steps_stay_in_range(ph, P)) return SCHED_INTERNAL;
        s.phases.push_back(ph);
        s.steps.push_back({1, 1, 0});
    }
    return SCHED_OK;
}

static int build_rd(uint32_t P, uint64_t m, Schedule& s) {
    if (P & (P - 1)) return SCHED_UNSUPPORTED;
    const int K = ceil_log2(P);
    s.K = K;
    s.phases.push_back(own_copy(m, false));
    for (int st = 0; st < K; st++) {
        const uint32_t g = 1u << st;  // r and r xor g swap their aligned groups of g slots
        PhaseDesc ph = blank(m);
        ph.peer_xor = g;
        ph.rank_mask = ~(g - 1);
        ph.src_space = ph.dst_space = SPACE_RECV;
        ph.src_rcoef = ph.dst_rcoef = 1;
        ph.src_step = ph.dst_step = 1;
        ph.copies = 1;  // the g slots are contiguous on both sides: one copy of g blocks
        ph.run = g;
        ph.copy_bytes = (uint64_t)g * m;
        if (!steps_stay_in_range(ph, P)) return SCHED_INTERNAL;
        s.phases.push_back(ph);
        s.steps.push_back({(int)g, (int)g, 0});
    }
    return SCHED_OK;
}

static int build_bruck(uint32_t P, uint64_t m, Schedule& s) {
    const int K = ceil_log2(P);
    const int F = floor_log2(P);
    s.K = K;
    s.rotation = true;
    s.phases.push_back(own_copy(m, true));  // working slot i of rank r holds block (r + i) mod P
    for (int st = 0; st < K; st++) {
        const uint32_t dist = 1u << st;
        const uint32_t n = st < F ? dist : P - dist;  // last step of a non-power of two: the rest
        PhaseDesc ph = blank(m);
        ph.peer_add = (P - dist % P) % P;             // sends to r - 2^st
        ph.src_space = ph.dst_space = SPACE_WORK;
        ph.src_off = 0;                               // the first n working slots ...
        ph.dst_off = dist;                            // ... land behind what the receiver holds
        ph.src_step = ph.dst_step = 1;
        ph.copies = 1;
        ph.run = n;
        ph.copy_bytes = (uint64_t)n * m;
        if (!steps_stay_in_range(ph, P) || dist + n > P) return SCHED_INTERNAL;
        s.phases.push_back(ph);
        s.steps.push_back({(int)dist, (int)n, 0});
    }
    PhaseDesc rot = blank(m);  // workspace[r][i] -> recvbuf[r][(r + i) mod P]
    rot.copies = P;
    rot.src_space = SPACE_WORK;
    rot.dst_space = SPACE_RECV;
    rot.src_step = 1;
    rot.dst_rcoef = 1;
    rot.dst_step = 1;
    if (!steps_stay_in_range(rot, P)) return SCHED_INTERNAL;
    s.phases.push_back(rot);
    return SCHED_OK;
}

// Neighbor exchange (Section II-A): P/2 steps, even P only.  On step s an even rank r exchanges
// with r + (-1)^s and an odd rank with r - (-1)^s: the pairing {2k, 2k+1} on even steps, the
// pairing shifted by one, {2k-1, 2k}, on odd steps; both are "add c, flip the lowest bit, subtract
// c" with c = s mod 2.  Step 0 swaps the own blocks, step 1 sends the pair of blocks a rank then
// holds, every later step forwards the pair received on the step before.  Unrolled, a rank whose
// own pair of slots starts at 2k forwards, on step s >= 1, the pair that starts a(s) pairs away:
// even ranks backwards on even steps and forwards on odd ones, odd ranks the other way round,
// with a(s) = s/2 on even steps and (s-1)/2 on odd ones.  Pairs land in their final slots.
static int build_ne(uint32_t P, uint64_t m, Schedule& s) {
    if (P % 2) return SCHED_UNSUPPORTED;
    s.K = (int)(P / 2);
    s.phases.push_back(own_copy(m, false));
    for (uint32_t st = 0; st < P / 2; st++) {
        const uint32_t c = st & 1u;
        PhaseDesc ph = blank(m);
        ph.peer_pre = c;
        ph.peer_xor = 1;
        ph.peer_add = (P - c) % P;
        ph.src_space = ph.dst_space = SPACE_RECV;
        ph.src_rcoef = ph.dst_rcoef = 1;
        if (st == 0) {
            // the own block, slot r on both sides
        } else {
            const uint32_t a = c ? (st - 1) / 2 : st / 2;  // pairs away from the own pair
            const uint32_t away = (2 * a) % P;              // in slots
            const uint32_t back = (P - away) % P;
            ph.rank_mask = ~1u;                             // 2k: first slot of the own pair
            ph.parity_split = 1;
            ph.src_off = ph.dst_off = c ? away : back;          // even ranks
            ph.src_off_odd = ph.dst_off_odd = c ? back : away;  // odd ranks
            ph.src_step = ph.dst_step = 1;
            ph.copies = 1;                                  // the two slots are adjacent: one copy
            ph.run = 2;
            ph.copy_bytes = 2 * m;
        }
        if (!steps_stay_in_range(ph, P)) return SCHED_INTERNAL;
        s.phases.push_back(ph);
        s.steps.push_back({1, st == 0 ? 1 : 2, 0});
    }
    return SCHED_OK;
}

// The first step of Sparbit, ring, neighbor exchange and recursive doubling forwards exactly one
// block per rank, the rank's own, from the slot the own-block copy has just filled.  Reading it from sendbuf instead
// and writing it to both places gives the same state after phase 0 with one pass less.
static void add_fused_first(Schedule& s) {
    if (s.K < 1 || s.rotation) return;
    const PhaseDesc& own = s.phases[0];
    const PhaseDesc& st0 = s.phases[1];
    if (st0.copies != 1 || st0.run != 1 || st0.src_space != SPACE_RECV || st0.dst_space != SPACE_RECV) return;
    // step 0 must read slot r of rank r (what the own-block copy wrote) and store it in slot r
    if (st0.src_rcoef != 1 || st0.src_off != 0 || st0.dst_rcoef != 1 || st0.dst_off != 0) return;
    if (st0.rank_mask != 0xFFFFFFFFu) return;
    PhaseDesc f = st0;
    f.src_space = own.src_space;  // sendbuf[r], one slot per rank
    f.src_rcoef = 0;
    f.src_off = f.src_off_odd = 0;
    f.src_step = 0;
    f.dup_self = 1;
    s.fused_first = f;
    s.has_fused_first = true;
}

int build_schedule(int algo, int64_t P64, uint64_t m, Schedule& out) {
    if (P64 < 1) return SCHED_ARG;
    if (P64 > (1 << 24)) return SCHED_OVERFLOW;
    const uint32_t P = (uint32_t)P64;
    // P * P * m must fit comfortably in 63 bits
    const unsigned __int128 total = (unsigned __int128)P * P * m;
    if (total >> 62) return SCHED_OVERFLOW;
    out = Schedule();
    out.algo = algo;
    out.P = P;
    out.m = m;
    int rc;
    switch (algo) {
        case ALGO_SPARBIT: rc = build_sparbit(P, m, out); break;
        case ALGO_RING: rc = build_ring(P, m, out); break;
        case ALGO_RD: rc = build_rd(P, m, out); break;
        case ALGO_BRUCK: rc = build_bruck(P, m, out); break;
        case ALGO_NE: rc = build_ne(P, m, out); break;
        default: return SCHED_ARG;
    }
    if (rc != SCHED_OK) return rc;
    // one offset for both parities unless a builder split them on purpose
    for (PhaseDesc& ph : out.phases)
        if (!ph.parity_split) {
            ph.src_off_odd = ph.src_off;
            ph.dst_off_odd = ph.dst_off;
        }
    add_fused_first(out);
    return SCHED_OK;
}

uint64_t phase_message_count(const Schedule& s, int phase) {
    const PhaseDesc& d = s.phase(phase);
    return (uint64_t)s.P * d.copies * d.run;
}

void expand_phase(const Schedule& s, int phase, std::vector<Msg>& out) {
    const PhaseDesc& d = s.phase(phase);
    out.clear();
    out.reserve((size_t)phase_message_count(s, phase));
    for (uint32_t r = 0; r < s.P; r++)
        for (uint32_t j = 0; j < d.copies; j++) {
            const CopyLoc c = locate_copy(d, s.P, r, j);
            for (uint32_t k = 0; k < d.run; k++) {  // a run is `run` consecutive slots, no wrap
                Msg msg;
                msg.phase = phase;
                msg.src_rank = (int32_t)c.src_rank;
                msg.dst_rank = (int32_t)c.dst_rank;
                msg.src_space = (int32_t)d.src_space;
                msg.src_slot = (int32_t)(c.src_slot + k);
                msg.dst_space = (int32_t)d.dst_space;
                msg.dst_slot = (int32_t)(c.dst_slot + k);
                out.push_back(msg);
            }
        }
}

void partition_counts(const Schedule& s, int phase, uint32_t G, int mapping, std::vector<uint64_t>& blocks) {
    const PhaseDesc& d = s.phase(phase);
    blocks.assign((size_t)G * G, 0);
    for (uint32_t r = 0; r < s.P; r++) {
        const uint32_t from = rank_device(s.P, G, mapping, r);
        for (uint32_t j = 0; j < d.copies; j++) {
            const CopyLoc c = locate_copy(d, s.P, r, j);
            blocks[(size_t)from * G + rank_device(s.P, G, mapping, c.dst_rank)] += d.run;
        }
    }
}

void partition_messages(const Schedule& s, int phase, uint32_t G, int mapping, uint32_t src_dev, uint32_t dst_dev,
                        std::vector<Msg>& out) {
    std::vector<Msg> all;
    expand_phase(s, phase, all);
    out.clear();
    for (const Msg& msg : all)
        if (rank_device(s.P, G, mapping, (uint32_t)msg.src_rank) == src_dev &&
            rank_device(s.P, G, mapping, (uint32_t)msg.dst_rank) == dst_dev)
            out.push_back(msg);
}

}  // namespace spb
