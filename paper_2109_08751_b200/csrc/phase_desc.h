// Compact per-phase descriptor shared by the host schedule generator and the copy kernels.
//
// A phase is a set of block copies, one per (rank r, index j) with 0 <= r < P, 0 <= j < copies:
//
//   dst_rank = ((((r + peer_pre) mod P) xor peer_xor) + peer_add) mod P
//   src_slot = wrap(wrap1(src_rcoef * (r & rank_mask) + (r odd ? src_off_odd : src_off)) + j * src_step)
//   dst_slot = wrap(wrap1(dst_rcoef * (r & rank_mask) + (r odd ? dst_off_odd : dst_off)) + j * dst_step)
//
// wrap1 folds a value in [0, 2P) into [0, P); wrap folds a value in (-P, 2P) into [0, P).  The
// schedule generator guarantees those ranges (|j * step| < P), so no division is needed on the
// device.  Each copy moves copy_bytes = run * m bytes: `run` consecutive slots when the phase's
// blocks are contiguous on both sides (recursive doubling, Bruck, neighbor exchange), else one.
//
// A phase with dup_self = 1 writes each copy twice: to (dst_rank, dst_slot) and to (r, dst_slot).
// That is the own-block copy and the first step in one pass: the first step forwards exactly the
// own block, so sendbuf[r] is read once and lands in recvbuf[r][r] and in the first peer's slot r.
//
// This form covers Algorithm 1's steps (peer r + d, slots r - 2jd on both sides), the ring, the
// recursive-doubling exchange (peer r xor 2^s, aligned groups), the neighbor exchange (peer
// r xor 1 on even steps, the pairing shifted by one on odd steps; even and odd ranks forward
// pairs in opposite directions, hence the two offsets), Bruck's steps and rotation, and the
// own-block copy, in O(1) bytes per phase whatever P is.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SPB_HD __host__ __device__ __forceinline__
#else
#define SPB_HD inline
#endif

namespace spb {

enum Space : uint32_t { SPACE_SEND = 0, SPACE_RECV = 1, SPACE_WORK = 2 };

struct PhaseDesc {
    uint32_t copies;      // copies per rank executed by the kernels (= blocks / run)
    uint32_t run;         // blocks per copy
    uint32_t peer_pre;    // in [0, P)
    uint32_t peer_xor;    // 0 = none
    uint32_t peer_add;    // in [0, P)
    uint32_t rank_mask;
    uint32_t src_off;     // in [0, P); for even ranks when parity_split
    uint32_t src_off_odd; // for odd ranks (equal to src_off unless parity_split)
    int32_t  src_step;    // slots between consecutive copies of a rank (signed)
    uint32_t dst_off;
    uint32_t dst_off_odd;
    int32_t  dst_step;
    uint8_t  src_rcoef;   // 0 or 1
    uint8_t  dst_rcoef;
    uint8_t  src_space;
    uint8_t  dst_space;
    uint8_t  dup_self;    // 1: every copy is also written to the SENDING rank's buffer of dst_space,
                          // same slot (the own-block copy fused with the first step)
    uint8_t  parity_split; // host only: the _odd offsets were set on purpose
    uint8_t  pad_[2];
    uint64_t copy_bytes;  // run * m
};
static_assert(sizeof(PhaseDesc) == 64, "PhaseDesc is copied as 16 words and budgeted at 64 bytes");

// Geometry of one collective call: where the three spaces live.
struct Geom {
    uint32_t P;
    uint32_t pad_;
    uint64_t m;               // bytes per block (slot pitch)
    char*    base[3];         // SEND, RECV, WORK
    uint64_t rank_pitch[3];   // bytes between consecutive ranks' buffers: m, P*m, P*m
    // Variable block sizes (allgatherv): m is 0, the send pitch 0 and the receive pitch the sum
    // of all block sizes; the kernels then work from task records that carry byte offsets.
};

struct CopyLoc {
    uint32_t src_rank, dst_rank, src_slot, dst_slot;
};

// All slot arithmetic fits 32 bits: P <= 2^24, bases are below 2P and |j * step| < P.
SPB_HD uint32_t wrap_slot(int32_t v, uint32_t P) {
    if (v < 0) v += (int32_t)P;
    if (v >= (int32_t)P) v -= (int32_t)P;
    return (uint32_t)v;
}

// Where copy j of rank r reads and writes.  The single definition used by the kernels and by the
// host-side expansion into explicit messages.
SPB_HD CopyLoc locate_copy(const PhaseDesc& d, uint32_t P, uint32_t r, uint32_t j) {
    CopyLoc c;
    c.src_rank = r;
    uint32_t t = r + d.peer_pre;
    if (t >= P) t -= P;
    t ^= d.peer_xor;
    t += d.peer_add;
    c.dst_rank = t >= P ? t - P : t;
    const uint32_t rr = r & d.rank_mask;
    const bool odd = (r & 1u) != 0;
    uint32_t s = (d.src_rcoef ? rr : 0u) + (odd ? d.src_off_odd : d.src_off);
    if (s >= P) s -= P;
    c.src_slot = wrap_slot((int32_t)s + (int32_t)j * d.src_step, P);
    uint32_t u = (d.dst_rcoef ? rr : 0u) + (odd ? d.dst_off_odd : d.dst_off);
    if (u >= P) u -= P;
    c.dst_slot = wrap_slot((int32_t)u + (int32_t)j * d.dst_step, P);
    return c;
}

// selects instead of dynamic indexing: kernel parameters stay in the constant bank
SPB_HD char* space_base(const Geom& g, uint32_t space) {
    return space == SPACE_SEND ? g.base[0] : (space == SPACE_RECV ? g.base[1] : g.base[2]);
}
SPB_HD uint64_t space_pitch(const Geom& g, uint32_t space) {
    return space == SPACE_SEND ? g.rank_pitch[0] : (space == SPACE_RECV ? g.rank_pitch[1] : g.rank_pitch[2]);
}

}  // namespace spb
