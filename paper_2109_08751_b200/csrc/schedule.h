// Host schedule generator: turns (algorithm, P, m) into compact per-phase descriptors.
#pragma once
#include <stdint.h>

#include <vector>

#include "phase_desc.h"

namespace spb {

enum Algo { ALGO_SPARBIT = 0, ALGO_RING = 1, ALGO_RD = 2, ALGO_BRUCK = 3, ALGO_NE = 4 };

struct StepInfo {
    int distance;  // ranks between sender and receiver (Algorithm 1's d)
    int blocks;    // messages per rank in the step (Algorithm 1's data - ignore)
    int ignore;    // 1 when the step withholds a block
};

struct Schedule {
    int algo = 0;
    uint32_t P = 0;
    uint64_t m = 0;
    int K = 0;               // communication steps
    bool rotation = false;   // Bruck's final phase
    // phases[0] is phase -1 (own block), phases[1 + s] is step s, phases[1 + K] the rotation
    std::vector<PhaseDesc> phases;
    std::vector<StepInfo> steps;
    // Execution-only shortcut: phases -1 and 0 as ONE pass (sendbuf[r] read once, written to
    // recvbuf[r][r] and to the first peer's slot r).  Valid when has_fused_first; used when a call
    // runs both phases.  The logical schedule (phases, messages) is unchanged by it.
    bool has_fused_first = false;
    PhaseDesc fused_first;
    int last_phase() const { return rotation ? K : K - 1; }
    const PhaseDesc& phase(int ph) const { return phases[(size_t)(ph + 1)]; }
};

// Error codes returned by build_schedule (mapped to the public ones by the caller).
enum { SCHED_OK = 0, SCHED_ARG = 1, SCHED_OVERFLOW = 2, SCHED_UNSUPPORTED = 4, SCHED_INTERNAL = 99 };

int build_schedule(int algo, int64_t P, uint64_t m, Schedule& out);

struct Msg {
    int32_t phase, src_rank, dst_rank, src_space, src_slot, dst_space, dst_slot;
};

// Explicit single-block messages of one phase, through locate_copy (the kernels' index function).
void expand_phase(const Schedule& s, int phase, std::vector<Msg>& out);

// Number of single-block messages of one phase.
uint64_t phase_message_count(const Schedule& s, int phase);

// Placement of the P ranks on G devices (Section III-C).  Sequential keeps neighbouring ranks
// together: device g holds the ranks [floor(g*P/G), floor((g+1)*P/G)).  Cyclic deals them out
// round robin: rank r sits on device r mod G.
enum Mapping { MAP_SEQUENTIAL = 0, MAP_CYCLIC = 1 };

inline uint32_t rank_device(uint32_t P, uint32_t G, int mapping, uint32_t r) {
    if (mapping == MAP_CYCLIC) return r % G;
    return (uint32_t)((((uint64_t)r + 1) * G - 1) / P);
}

// Splits the single-block messages of one phase by (device of the sender, device of the
// receiver).  blocks gets G*G counts, row = sending device; the diagonal is what stays local.
void partition_counts(const Schedule& s, int phase, uint32_t G, int mapping, std::vector<uint64_t>& blocks);

// The messages of one phase that go from device src_dev to device dst_dev (src_dev == dst_dev:
// the local copy list of that device), in the order expand_phase lists them.
void partition_messages(const Schedule& s, int phase, uint32_t G, int mapping, uint32_t src_dev, uint32_t dst_dev,
                        std::vector<Msg>& out);

}  // namespace spb
