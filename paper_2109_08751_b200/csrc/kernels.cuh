// Copy kernels of the step executor (sm_100a).
//
// Two copy engines execute one pass (a set of block copies given by a PhaseDesc):
//
//   vector  warp-cooperative ld.global.cg / st.global.cg with 16-, 8-, 4-, 2- or 1-byte vectors.
//           A warp task is a span of one copy (32 lanes x U vectors, index arithmetic once per
//           span) or, for copies shorter than a warp row, rows of several whole copies.  A
//           second form (vec_list_phase) takes a host-built task list, for blocks of different
//           sizes.
//   bulk    cp.async.bulk global -> shared -> global through a ring of shared-memory stages, one
//           elected lane per warp driving its own ring; completion of loads through mbarriers,
//           of stores through bulk async-groups.  Every load fills one CTA's own shared memory and
//           every block has one destination (two in the fused first pass, issued as two stores).
//
// and five ways to sequence passes: one kernel per pass, chained by programmatic dependent launch
// (plain stream launches or a CUDA graph); one persistent cooperative kernel with a bounded-wait
// grid barrier after every pass; one kernel in which every rank's Waitall is a set of per-rank
// counters instead of a barrier (flow); and, for small collectives, one CTA or one cluster of
// CTAs that keeps a copy of the receive buffers in (distributed) shared memory and feeds every
// pass from there (mirror).
//
// Loads never use the non-coherent path or L1: data written in one pass is read by other SMs in
// the next one, possibly inside the same launch.
//
// Both engines are tuned to about 32 KiB of loads in flight per SM, the measured sweet spot of a
// copy on B200 (more in flight lowers the achieved HBM bandwidth).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "phase_desc.h"

namespace spb {

// device status word values
enum : unsigned { DEV_OK = 0u, DEV_BARRIER_TIMEOUT = 1u, DEV_MBARRIER_TIMEOUT = 2u };

struct BarrierCtl {
    unsigned* counter;        // monotonically increasing arrival counter
    unsigned* status;         // device status word (DEV_*)
    unsigned  base;           // counter value when this launch starts
    unsigned  expected;       // arrivals that complete one barrier (grid size, + test extra)
    unsigned long long timeout_ns;
    unsigned  mbar_extra_tx;  // test hook: bytes added to every expected transaction count, so
                              // that no mbarrier of the bulk engine ever completes (0 = off)
    unsigned long long* trace;  // optional: CTA 0 stores %globaltimer at kernel start and after
                                // every pass it leaves (passes + 1 entries); null = off
};

// Tunables (overridable at compile time for experiments).
#ifndef SPB_BULK_STAGES
#define SPB_BULK_STAGES 4   // stages per ring
#endif
#ifndef SPB_BULK_LOADS
#define SPB_BULK_LOADS 2    // loads in flight per ring; the other stages hold pending stores
#endif
#ifndef SPB_VEC_UNROLL
#define SPB_VEC_UNROLL 2    // vectors per lane per warp task
#endif
#ifndef SPB_PERSIST_MIN_CTAS
#define SPB_PERSIST_MIN_CTAS 2  // CTAs of 512 threads per SM the persistent vector kernel is built for
#endif
constexpr int kBulkStages = SPB_BULK_STAGES;
constexpr int kBulkLoadsAhead = SPB_BULK_LOADS;
constexpr int kVecUnroll = SPB_VEC_UNROLL;
static_assert(kBulkLoadsAhead >= 1 && kBulkLoadsAhead < kBulkStages, "a ring needs stages for loads and for stores");

// ------------------------------------------------------------------------------------------------
// small PTX helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_relaxed_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned* p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() {
    asm volatile("fence.proxy.async;" ::: "memory");
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_dst),
        "l"(gsrc), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// vector engine
// ------------------------------------------------------------------------------------------------
template <typename V>
__device__ __forceinline__ V ld_cg(const V* p);
template <typename V>
__device__ __forceinline__ void st_cg(V* p, V v);

template <>
__device__ __forceinline__ uint4 ld_cg<uint4>(const uint4* p) { return __ldcg(p); }
template <>
__device__ __forceinline__ uint2 ld_cg<uint2>(const uint2* p) { return __ldcg(p); }
template <>
__device__ __forceinline__ unsigned ld_cg<unsigned>(const unsigned* p) { return __ldcg(p); }
template <>
__device__ __forceinline__ unsigned short ld_cg<unsigned short>(const unsigned short* p) { return __ldcg(p); }
template <>
__device__ __forceinline__ unsigned char ld_cg<unsigned char>(const unsigned char* p) { return __ldcg(p); }
template <>
__device__ __forceinline__ void st_cg<uint4>(uint4* p, uint4 v) { __stcg(p, v); }
template <>
__device__ __forceinline__ void st_cg<uint2>(uint2* p, uint2 v) { __stcg(p, v); }
template <>
__device__ __forceinline__ void st_cg<unsigned>(unsigned* p, unsigned v) { __stcg(p, v); }
template <>
__device__ __forceinline__ void st_cg<unsigned short>(unsigned short* p, unsigned short v) { __stcg(p, v); }
template <>
__device__ __forceinline__ void st_cg<unsigned char>(unsigned char* p, unsigned char v) { __stcg(p, v); }

// One phase on the vector engine.  warp_id / n_warps enumerate all warps taking part.
// Requires P * copies * ceil(vectors_per_copy / (32*U)) < 2^32 (checked on the host).
template <typename V, int U = kVecUnroll>
__device__ __forceinline__ void vec_phase(const Geom& g, const PhaseDesc& d, uint32_t warp_id, uint32_t n_warps,
                                          uint32_t lane) {
    const uint32_t P = g.P;
    const uint64_t vpc64 = d.copy_bytes / sizeof(V);  // vectors per copy
    const uint32_t n_copies = P * d.copies;            // copies in the phase (< 2^32, host-checked)
    const char* sbase = space_base(g, d.src_space);
    char* dbase = space_base(g, d.dst_space);
    const uint64_t spitch = space_pitch(g, d.src_space);
    const uint64_t dpitch = space_pitch(g, d.dst_space);

    if (vpc64 >= 32) {
        // a task is one span of 32*U vectors inside one copy
        const uint32_t span = 32u * U;
        const uint32_t spc = (uint32_t)((vpc64 + span - 1) / span);  // spans per copy
        const uint64_t tasks = (uint64_t)n_copies * spc;
        for (uint64_t w = warp_id; w < tasks; w += n_warps) {
            const uint32_t w32 = (uint32_t)w;
            const uint32_t q = w32 / spc;
            const uint32_t sp = w32 - q * spc;
            const uint32_t r = q / d.copies;
            const uint32_t j = q - r * d.copies;
            const CopyLoc c = locate_copy(d, P, r, j);
            const V* src = reinterpret_cast<const V*>(sbase + ((uint64_t)c.src_rank * spitch + (uint64_t)c.src_slot * g.m));
            V* dst = reinterpret_cast<V*>(dbase + ((uint64_t)c.dst_rank * dpitch + (uint64_t)c.dst_slot * g.m));
            V* dst2 = reinterpret_cast<V*>(dbase + ((uint64_t)r * dpitch + (uint64_t)c.dst_slot * g.m));
            const uint64_t v0 = (uint64_t)sp * span + lane;
            V regs[U];
#pragma unroll
            for (int k = 0; k < U; k++) {
                const uint64_t v = v0 + 32u * k;
                if (v < vpc64) regs[k] = ld_cg<V>(src + v);
            }
#pragma unroll
            for (int k = 0; k < U; k++) {
                const uint64_t v = v0 + 32u * k;
                if (v < vpc64) {
                    st_cg<V>(dst + v, regs[k]);
                    if (d.dup_self) st_cg<V>(dst2 + v, regs[k]);
                }
            }
        }
    } else if (vpc64 > 0) {
        // a copy is shorter than a warp row: a row holds cpw whole copies, a task is U rows
        const uint32_t vpc = (uint32_t)vpc64;
        const uint32_t cpw = 32u / vpc;
        const uint32_t sub = lane / vpc;       // which copy of the row
        const uint32_t v = lane - sub * vpc;   // which vector of that copy
        const bool lane_on = sub < cpw;
        const uint32_t per_task = cpw * U;
        const uint64_t tasks = ((uint64_t)n_copies + per_task - 1) / per_task;
        for (uint64_t w = warp_id; w < tasks; w += n_warps) {
            V regs[U];
            V* dsts[U];
            V* dsts2[U];
#pragma unroll
            for (int k = 0; k < U; k++) {
                const uint64_t q64 = (w * U + k) * cpw + sub;
                dsts[k] = nullptr;
                if (lane_on && q64 < n_copies) {
                    const uint32_t q = (uint32_t)q64;
                    const uint32_t r = q / d.copies;
                    const uint32_t j = q - r * d.copies;
                    const CopyLoc c = locate_copy(d, P, r, j);
                    const V* src =
                        reinterpret_cast<const V*>(sbase + ((uint64_t)c.src_rank * spitch + (uint64_t)c.src_slot * g.m));
                    dsts[k] = reinterpret_cast<V*>(dbase + ((uint64_t)c.dst_rank * dpitch + (uint64_t)c.dst_slot * g.m)) + v;
                    dsts2[k] = reinterpret_cast<V*>(dbase + ((uint64_t)r * dpitch + (uint64_t)c.dst_slot * g.m)) + v;
                    regs[k] = ld_cg<V>(src + v);
                }
            }
#pragma unroll
            for (int k = 0; k < U; k++)
                if (dsts[k]) {
                    st_cg<V>(dsts[k], regs[k]);
                    if (d.dup_self) st_cg<V>(dsts2[k], regs[k]);
                }
        }
    }
}

// One phase with blocks of DIFFERENT sizes (allgatherv).  The host lists the phase's work as tasks
// of at most kVarSegmentBytes, each a self-contained record: where the bytes are read (offset
// inside the phase's source space), where they go (offset inside its destination space), how
// many, and - for the fused first pass - how many ranks away the second destination is.  Empty
// blocks have no entry.  Every task is about the same size, so handing task t to warp
// t mod n_warps balances the warps whatever the mix of block sizes is, and a task needs no
// index arithmetic and no size table on the device.
constexpr uint32_t kVarSegmentBytes = 4096;

struct VarTask {
    unsigned long long a;  // bits 0..47 source byte offset, bits 48..63 byte count - 1
    unsigned long long b;  // bits 0..47 destination byte offset, bits 48..63 (signed) rank distance
                           // of the second destination in a dup_self phase
};
static_assert(sizeof(VarTask) == 16, "a task is read with one 16-byte load");
constexpr unsigned long long kVarOffsetMask = (1ull << 48) - 1;

__device__ __forceinline__ VarTask ld_task(const VarTask* p) {
    const ulonglong2 v = __ldg(reinterpret_cast<const ulonglong2*>(p));
    VarTask t;
    t.a = v.x;
    t.b = v.y;
    return t;
}

template <typename V>
__device__ __forceinline__ void vec_list_phase(const Geom& g, const PhaseDesc& d, const VarTask* __restrict__ list,
                                               uint64_t count, uint32_t warp_id, uint32_t n_warps, uint32_t lane) {
    // four vectors per lane: blocks of arbitrary sizes rarely start on 128-byte lines, which makes
    // every load slower, and more of them in flight make up for part of it (uniformly random sizes
    // around 4 KiB at P = 256: 113.7 us against 128.4 with two; around 1 KiB at P = 1000: 452 against 486)
    constexpr int U = 4;
    constexpr uint32_t span = 32u * U;  // vectors per warp iteration
    const char* sbase = space_base(g, d.src_space);
    char* dbase = space_base(g, d.dst_space);
    const long long dpitch = (long long)space_pitch(g, d.dst_space);
    if (warp_id >= count) return;
    VarTask next = ld_task(list + warp_id);
    for (uint64_t t = warp_id; t < count; t += n_warps) {
        const VarTask e = next;
        if (t + n_warps < count) next = ld_task(list + t + n_warps);  // in flight while this task is copied
        const V* src = reinterpret_cast<const V*>(sbase + (e.a & kVarOffsetMask));
        V* dst = reinterpret_cast<V*>(dbase + (e.b & kVarOffsetMask));
        V* dst2 = reinterpret_cast<V*>(reinterpret_cast<char*>(dst) + (long long)(short)(e.b >> 48) * dpitch);
        const uint32_t vectors = ((uint32_t)(e.a >> 48) + 1u) / (uint32_t)sizeof(V);
#pragma unroll 1
        for (uint32_t first = 0; first < vectors; first += span) {
            V regs[U];
#pragma unroll
            for (int k = 0; k < U; k++) {
                const uint32_t v = first + lane + 32u * k;
                if (v < vectors) regs[k] = ld_cg<V>(src + v);
            }
#pragma unroll
            for (int k = 0; k < U; k++) {
                const uint32_t v = first + lane + 32u * k;
                if (v < vectors) {
                    st_cg<V>(dst + v, regs[k]);
                    if (d.dup_self) st_cg<V>(dst2 + v, regs[k]);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// bulk engine
// ------------------------------------------------------------------------------------------------
struct BulkPipe {
    uint32_t ring;      // shared address of this warp's first stage
    uint32_t bars;      // shared address of this warp's first mbarrier (kBulkStages of them)
    uint32_t meta;      // shared address of per-stage {dst pointer, bytes, second-dst delta, pad} records (32 B: v2.u64 accesses need 16-byte alignment)
    uint32_t taskq;     // shared address of this ring's queue of prefetched task-list entries (kTaskQueue x 16 B)
    uint32_t it;        // stages used so far by this ring (carried across phases)
};
constexpr int kTaskQueue = 8;   // entries of the queue
constexpr int kTaskAhead = 6;   // list entries in flight ahead of the task being issued

// Bounded wait on one mbarrier phase.  Returns false (after setting the status word) on time-out
// or when another CTA already reported a failure.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, unsigned* status,
                                                  unsigned long long timeout_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    unsigned polls = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 63u) == 0) {
            if (ld_relaxed_gpu(status) != DEV_OK) return false;
            if (globaltimer_ns() - t0 > timeout_ns) {
                atomicCAS(status, DEV_OK, DEV_MBARRIER_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// One phase on the bulk engine, driven by ONE thread (the elected lane of a warp).  pipe_id /
// n_pipes enumerate all rings taking part.  All addresses and sizes are multiples of 16 bytes
// (host-checked).  Returns false if a wait gave up.
//
// With a task list (blocks of different sizes) a task is one list entry (at most one stage, host-
// checked) instead of a chunk of a copy located through the descriptor; the entry of the task
// after the one being issued is fetched one step ahead.
template <bool kList = false>
__device__ __forceinline__ bool bulk_phase(const Geom& g, const PhaseDesc& d, uint32_t stage_bytes, uint32_t pipe_id,
                                           uint32_t n_pipes, BulkPipe& pp, unsigned* status,
                                           unsigned long long timeout_ns, uint32_t extra_tx = 0,
                                           const VarTask* __restrict__ list = nullptr, uint64_t count = 0) {
    constexpr int S = kBulkStages;
    constexpr int L = kBulkLoadsAhead;
    const uint32_t P = g.P;
    const uint64_t cpc = kList ? 1 : (d.copy_bytes + stage_bytes - 1) / stage_bytes;  // chunks per copy
    const uint64_t tasks = kList ? count : (uint64_t)P * d.copies * cpc;
    if (pipe_id >= tasks) return true;
    // equal chunks (rounded up to 128 B) instead of full stages plus a short tail
    const uint32_t chunk = kList ? 0u : (uint32_t)((((d.copy_bytes + cpc - 1) / cpc) + 127u) & ~127ull);
    // A list entry costs a memory round trip and the ring issues a task every third of one, so the
    // entries of the next kTaskAhead tasks are kept in flight, copied asynchronously into a small
    // shared-memory queue (one async group per entry, empty past the end of the list).
    auto fetch_entry = [&](uint64_t k) {
        if (k < tasks) {
            const uint64_t n = (k - pipe_id) / n_pipes;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(pp.taskq + (uint32_t)(n % kTaskQueue) * 16u),
                         "l"(list + k)
                         : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (kList)
        for (int k = 0; k < kTaskAhead; k++) fetch_entry(pipe_id + (uint64_t)k * n_pipes);
    fence_proxy_async_all();  // what other CTAs wrote before the barrier -> visible to bulk loads
    const uint64_t mine = (tasks - pipe_id + n_pipes - 1) / n_pipes;      // tasks of this ring
    const bool small = (tasks >> 32) == 0;
    const char* sbase = space_base(g, d.src_space);
    char* dbase = space_base(g, d.dst_space);
    const uint64_t spitch = space_pitch(g, d.src_space);
    const uint64_t dpitch = space_pitch(g, d.dst_space);
    bool ok = true;

    for (uint64_t i = 0; i < mine + L; i++) {
        if (i < mine) {
            const uint32_t slot_it = pp.it + (uint32_t)i;
            const uint32_t st = slot_it % S;
            // the store that last used this stage (S tasks ago) must have finished reading shared
            // memory: stores are committed one group per task, L tasks behind the loads
            bulk_wait_read<S - L - 1>();
            const uint64_t w = pipe_id + i * n_pipes;
            const char* src;
            char* dst;
            uint32_t bytes;
            long long delta2;  // second destination of a dup_self phase, as a byte delta from the first
            if constexpr (kList) {
                fetch_entry(w + (uint64_t)kTaskAhead * n_pipes);
                asm volatile("cp.async.wait_group %0;" ::"n"(kTaskAhead) : "memory");  // entry i has landed
                VarTask e;
                asm volatile("ld.shared.v2.u64 {%0, %1}, [%2];" : "=l"(e.a), "=l"(e.b)
                             : "r"(pp.taskq + (uint32_t)(i % kTaskQueue) * 16u)
                             : "memory");
                src = sbase + (e.a & kVarOffsetMask);
                dst = dbase + (e.b & kVarOffsetMask);
                bytes = (uint32_t)(e.a >> 48) + 1u;
                delta2 = (long long)(short)(e.b >> 48) * (long long)dpitch;
            } else {
                uint64_t q, ch;
                uint32_t r, j;
                if (small) {  // everything fits 32 bits: four cheap divisions instead of four long ones
                    const uint32_t w32 = (uint32_t)w, cpc32 = (uint32_t)cpc;
                    const uint32_t q32 = w32 / cpc32;
                    ch = w32 - q32 * cpc32;
                    r = q32 / d.copies;
                    j = q32 - r * d.copies;
                    q = q32;
                } else {
                    q = w / cpc;
                    ch = w - q * cpc;
                    r = (uint32_t)(q / d.copies);
                    j = (uint32_t)(q - (uint64_t)r * d.copies);
                }
                const CopyLoc c = locate_copy(d, P, r, j);
                const uint64_t off = ch * chunk;
                const uint64_t left = d.copy_bytes - off;
                bytes = left < chunk ? (uint32_t)left : chunk;
                src = sbase + ((uint64_t)c.src_rank * spitch + (uint64_t)c.src_slot * g.m) + off;
                dst = dbase + ((uint64_t)c.dst_rank * dpitch + (uint64_t)c.dst_slot * g.m) + off;
                delta2 = ((long long)r - (long long)c.dst_rank) * (long long)dpitch;
            }
            const uint32_t bar = pp.bars + st * 8u;
            // remember where this stage goes
            asm volatile("st.shared.v2.u64 [%0], {%1, %2};" ::"r"(pp.meta + st * 32u), "l"(dst),
                         "l"((unsigned long long)bytes)
                         : "memory");
            asm volatile("st.shared.u64 [%0], %1;" ::"r"(pp.meta + st * 32u + 16u), "l"(delta2) : "memory");
            mbar_expect_tx(bar, bytes + extra_tx);
            bulk_load(pp.ring + st * stage_bytes, src, bytes, bar);
        }
        if (i >= (uint64_t)L) {
            const uint32_t slot_it = pp.it + (uint32_t)(i - L);
            const uint32_t st = slot_it % S;
            const uint32_t parity = (slot_it / S) & 1u;
            if (!mbar_wait_bounded(pp.bars + st * 8u, parity, status, timeout_ns)) {
                ok = false;
                break;
            }
            unsigned long long dst, bytes;
            asm volatile("ld.shared.v2.u64 {%0, %1}, [%2];" : "=l"(dst), "=l"(bytes) : "r"(pp.meta + st * 32u)
                         : "memory");
            bulk_store(reinterpret_cast<void*>(dst), pp.ring + st * stage_bytes, (uint32_t)bytes);
            if (d.dup_self) {
                long long delta2;
                asm volatile("ld.shared.u64 %0, [%1];" : "=l"(delta2) : "r"(pp.meta + st * 32u + 16u) : "memory");
                bulk_store(reinterpret_cast<void*>(dst + delta2), pp.ring + st * stage_bytes, (uint32_t)bytes);
            }
            bulk_commit();
        }
    }
    pp.it += (uint32_t)mine;
    // all stores of this phase complete (written, not only read) before anyone is told about it
    bulk_wait_all();
    fence_proxy_async_all();
    return ok;
}

// ------------------------------------------------------------------------------------------------
// bounded-wait grid barrier (persistent executor)
// ------------------------------------------------------------------------------------------------
// All threads of all CTAs call it; `epoch` counts the barriers this launch has passed.  Returns
// false when the wait gave up or another CTA reported a failure: the caller must then leave the
// kernel.  Co-residency of the grid is guaranteed by the cooperative launch.
template <bool kAsyncProxy>
__device__ __forceinline__ bool grid_barrier(const BarrierCtl& ctl, unsigned& epoch, int* smem_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        epoch++;
        const unsigned target = ctl.base + epoch * ctl.expected;
        if (kAsyncProxy) fence_proxy_async_all();  // bulk stores of this CTA -> visible before the release
        red_release_gpu_add(ctl.counter, 1u);
        bool ok = true;
        unsigned polls = 0;
        unsigned long long t0 = 0;
        while ((int)(ld_acquire_gpu(ctl.counter) - target) < 0) {
            if ((++polls & 31u) == 0) {
                if (t0 == 0) t0 = globaltimer_ns();
                if (ld_relaxed_gpu(ctl.status) != DEV_OK) {
                    ok = false;
                    break;
                }
                if (globaltimer_ns() - t0 > ctl.timeout_ns) {
                    atomicCAS(ctl.status, DEV_OK, DEV_BARRIER_TIMEOUT);
                    ok = false;
                    break;
                }
            }
        }
        if (kAsyncProxy) fence_proxy_async_all();  // later bulk loads see what the other CTAs wrote
        *smem_flag = ok ? 1 : 0;
    }
    __syncthreads();
    return *smem_flag != 0;
}

// ------------------------------------------------------------------------------------------------
// kernels
// ------------------------------------------------------------------------------------------------
// Per-phase kernels are chained with programmatic dependent launch: a kernel waits until the
// previous phase's grid has completed and its writes are visible (griddepcontrol.wait) before it
// touches memory, and lets the next phase's kernel start launching with
// griddepcontrol.launch_dependents - the vector kernel once its own copies are issued (measured on
// B200: triggering at its start costs 3-4 % of bandwidth at large blocks), the bulk kernel at
// once.  Both instructions are no-ops for a launch without the attribute.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// one phase, vector engine
template <typename V>
__global__ void __launch_bounds__(512, 2) phase_vec_kernel(Geom g, PhaseDesc d) {
    chain_wait();
    const uint32_t wpb = blockDim.x >> 5;
    vec_phase<V>(g, d, blockIdx.x * wpb + (threadIdx.x >> 5), gridDim.x * wpb, threadIdx.x & 31u);
    chain_trigger();
}

// one phase, vector engine, variable block sizes (task list built by the host)
template <typename V>
__global__ void __launch_bounds__(512, 2) phase_vec_list_kernel(Geom g, PhaseDesc d, const VarTask* list,
                                                                unsigned long long count) {
    chain_wait();
    const uint32_t wpb = blockDim.x >> 5;
    vec_list_phase<V>(g, d, list, count, blockIdx.x * wpb + (threadIdx.x >> 5), gridDim.x * wpb, threadIdx.x & 31u);
    chain_trigger();
}

// shared-memory layout of the bulk kernels: [rings | mbarriers | meta], ring stages 128-B aligned
__device__ __forceinline__ BulkPipe make_pipe(unsigned char* smem, uint32_t stage_bytes, uint32_t warps,
                                              uint32_t warp) {
    BulkPipe pp;
    const uint32_t base = smem_u32(smem);
    const uint32_t rings = warps * kBulkStages * stage_bytes;
    pp.ring = base + warp * kBulkStages * stage_bytes;
    pp.bars = base + rings + warp * kBulkStages * 8u;
    pp.meta = base + rings + warps * kBulkStages * 8u + warp * kBulkStages * 32u;
    pp.taskq = base + rings + warps * kBulkStages * 40u + warp * kTaskQueue * 16u;
    pp.it = 0;
    return pp;
}
__device__ __forceinline__ void init_pipe(const BulkPipe& pp) {
    for (int s = 0; s < kBulkStages; s++) mbar_init(pp.bars + s * 8u, 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_all();
}

// one phase, bulk engine
__global__ void __launch_bounds__(256) phase_bulk_kernel(Geom g, PhaseDesc d, uint32_t stage_bytes, unsigned* status,
                                                         unsigned long long timeout_ns, uint32_t extra_tx) {
    extern __shared__ __align__(128) unsigned char smem[];
    // the bulk kernel leaves room on the SM for its successor (4 warps, 66 KB), and measures
    // best when the successor is let in at once and sets up its rings during this phase
    chain_trigger();
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31u) == 0) {
        BulkPipe pp = make_pipe(smem, stage_bytes, warps, warp);
        init_pipe(pp);
        chain_wait();
        bulk_phase(g, d, stage_bytes, blockIdx.x * warps + warp, gridDim.x * warps, pp, status, timeout_ns,
                   extra_tx);
    }
}

// one phase, bulk engine, variable block sizes (same task list as the vector form)
__global__ void __launch_bounds__(256) phase_bulk_list_kernel(Geom g, PhaseDesc d, uint32_t stage_bytes,
                                                              unsigned* status, unsigned long long timeout_ns,
                                                              uint32_t extra_tx, const VarTask* list,
                                                              unsigned long long count) {
    extern __shared__ __align__(128) unsigned char smem[];
    chain_trigger();
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31u) == 0) {
        BulkPipe pp = make_pipe(smem, stage_bytes, warps, warp);
        init_pipe(pp);
        chain_wait();
        bulk_phase<true>(g, d, stage_bytes, blockIdx.x * warps + warp, gridDim.x * warps, pp, status, timeout_ns,
                         extra_tx, list, count);
    }
}

// Where the task list of each entry of the device descriptor table starts, and how long it is
// (variable block sizes; the persistent kernels walk the table).
struct VarRange {
    unsigned long long lo, count;
};

// Descriptors of a multi-phase kernel live in shared memory, double-buffered: the next phase's
// descriptor is fetched while the current phase runs, so no phase starts with a global load on
// its critical path, and the copy loops need no registers to hold it.
__device__ __forceinline__ void fetch_desc(PhaseDesc* dst, const PhaseDesc* __restrict__ src) {
    static_assert(sizeof(PhaseDesc) == 64, "PhaseDesc is copied as 16 words");
    if (threadIdx.x < 16)
        reinterpret_cast<uint32_t*>(dst)[threadIdx.x] = reinterpret_cast<const uint32_t*>(src)[threadIdx.x];
}

// phases first..last (indices into descs), vector engine, grid barrier between phases
template <typename V, bool kList = false>
__global__ void __launch_bounds__(512, SPB_PERSIST_MIN_CTAS) persistent_vec_kernel(Geom g, const PhaseDesc* __restrict__ descs,
                                                                int first, int last, BarrierCtl ctl,
                                                                const VarTask* __restrict__ tasks = nullptr,
                                                                const VarRange* __restrict__ ranges = nullptr) {
    __shared__ int flag;
    __shared__ PhaseDesc sd[2];
    if (ld_relaxed_gpu(ctl.status) != DEV_OK) return;  // an earlier failure was not cleared yet
    const uint32_t wpb = blockDim.x >> 5;
    const uint32_t warp_id = blockIdx.x * wpb + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * wpb;
    unsigned epoch = 0;
    const bool tracer = ctl.trace != nullptr && blockIdx.x == 0 && threadIdx.x == 0;
    if (tracer) ctl.trace[0] = globaltimer_ns();
    fetch_desc(&sd[0], &descs[first]);
    __syncthreads();
    for (int ph = first; ph <= last; ph++) {
        const int cur = (ph - first) & 1;
        if (ph != last) fetch_desc(&sd[cur ^ 1], &descs[ph + 1]);
        if (kList) {
            const VarRange vr = ranges[ph];
            vec_list_phase<V>(g, sd[cur], tasks + vr.lo, vr.count, warp_id, n_warps, threadIdx.x & 31u);
        } else {
            vec_phase<V>(g, sd[cur], warp_id, n_warps, threadIdx.x & 31u);
        }
        if (ph != last && !grid_barrier<false>(ctl, epoch, &flag)) return;
        if (tracer) ctl.trace[ph - first + 1] = globaltimer_ns();
    }
}

// phases first..last, bulk engine, grid barrier between phases
template <bool kList = false>
__global__ void __launch_bounds__(256) persistent_bulk_kernel(Geom g, const PhaseDesc* __restrict__ descs, int first,
                                                              int last, uint32_t stage_bytes, BarrierCtl ctl,
                                                              const VarTask* __restrict__ tasks = nullptr,
                                                              const VarRange* __restrict__ ranges = nullptr) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int flag;
    __shared__ PhaseDesc sd[2];
    if (ld_relaxed_gpu(ctl.status) != DEV_OK) return;
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5;
    const bool driver = (threadIdx.x & 31u) == 0;
    BulkPipe pp = make_pipe(smem, stage_bytes, warps, warp);
    if (driver) init_pipe(pp);
    unsigned epoch = 0;
    const bool tracer = ctl.trace != nullptr && blockIdx.x == 0 && threadIdx.x == 0;
    if (tracer) ctl.trace[0] = globaltimer_ns();
    fetch_desc(&sd[0], &descs[first]);
    __syncthreads();
    for (int ph = first; ph <= last; ph++) {
        const int cur = (ph - first) & 1;
        if (ph != last) fetch_desc(&sd[cur ^ 1], &descs[ph + 1]);
        if (driver) {
            if (kList) {
                const VarRange vr = ranges[ph];
                bulk_phase<true>(g, sd[cur], stage_bytes, blockIdx.x * warps + warp, gridDim.x * warps, pp, ctl.status,
                                 ctl.timeout_ns, ctl.mbar_extra_tx, tasks + vr.lo, vr.count);
            } else {
                bulk_phase<false>(g, sd[cur], stage_bytes, blockIdx.x * warps + warp, gridDim.x * warps, pp,
                                  ctl.status, ctl.timeout_ns, ctl.mbar_extra_tx);
            }
        }
        if (ph != last && !grid_barrier<true>(ctl, epoch, &flag)) return;
        if (tracer) ctl.trace[ph - first + 1] = globaltimer_ns();
    }
}

// ------------------------------------------------------------------------------------------------
// mirror executor: a whole SMALL collective in one CTA, the receive buffers mirrored on chip
// ------------------------------------------------------------------------------------------------
// In the latency regime a pass costs two memory round trips (the loads, then the acknowledged
// stores: 1.6-2.3 us on B200) however passes are separated.  When all P receive buffers together
// fit into one SM's shared memory, this kernel keeps a copy of them there: every block that is
// written to a receive buffer is written to global memory AND to the same place of the on-chip
// copy, and every forwarded block is read from the on-chip copy of the SENDING rank's receive
// buffer - the slot the schedule names, with the bytes that were stored there one or more passes
// earlier - instead of from global memory.  The schedule, the passes and their order are
// unchanged; a pass boundary is the CTA's barrier, and a pass costs a shared-memory access.
// Only the own blocks are read from global memory (the send buffer).  Bruck's working buffers are
// mirrored the same way (twice the shared memory).
constexpr int kMirrorMaxPasses = 16;
struct MirrorArgs {
    PhaseDesc d[kMirrorMaxPasses];
    int n;
    uint32_t work_at;  // Bruck: where, in vectors, the on-chip copy of the working buffers starts
    uint32_t extra_tx;  // cluster form, test hook: bytes expected on top of a pass's own (never arrive)
    int aligned;        // grouped form: 0 = a group is a residue class mod G, 1 = a run of P/G consecutive ranks
    unsigned* status;   // cluster form: device status word (DEV_*)
    unsigned long long timeout_ns;
    // ceil(2^40 / x) for x = vectors per copy and x = copies per rank of each pass, so that t / x
    // is a multiplication and a shift (exact while t * x < 2^40; t counts the vectors sent in a
    // pass, fewer than the shared memory holds bytes: 2^18)
    unsigned long long magic_vpc[kMirrorMaxPasses];
    unsigned long long magic_copies[kMirrorMaxPasses];
};

// kWork: the collective has working buffers (Bruck); without them every pass writes the receive
// space and the space look-ups fold away.
template <typename V, bool kWork>
__global__ void __launch_bounds__(1024, 1) mirror_vec_kernel(Geom g, const __grid_constant__ MirrorArgs ma) {
    // [P][P] slots of m bytes, laid out as the RECV space; for Bruck a second such array for its
    // working buffers behind it
    extern __shared__ __align__(16) unsigned char mirror[];
    chain_trigger();
    chain_wait();
    const uint32_t P = g.P;
    const uint32_t vps = (uint32_t)(g.m / sizeof(V));  // vectors per slot
    V* mir = reinterpret_cast<V*>(mirror);
    for (int i = 0; i < ma.n; i++) {
        if (i) __syncthreads();
        const PhaseDesc& d = ma.d[i];
        const uint32_t vpc = (uint32_t)(d.copy_bytes / sizeof(V));
        const uint32_t total = P * d.copies * vpc;  // fits: the whole receive space is below 256 KiB
        const bool from_send = d.src_space == SPACE_SEND;
        const V* msrc = mir + (kWork && d.src_space == SPACE_WORK ? ma.work_at : 0u);
        V* mdst = mir + (kWork && d.dst_space == SPACE_WORK ? ma.work_at : 0u);
        V* gdst = reinterpret_cast<V*>(kWork ? space_base(g, d.dst_space) : g.base[SPACE_RECV]);
        const unsigned long long mv = ma.magic_vpc[i], mc = ma.magic_copies[i];
        for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
            const uint32_t q = (uint32_t)((t * mv) >> 40);  // t / vpc
            const uint32_t v = t - q * vpc;
            const uint32_t r = (uint32_t)((q * mc) >> 40);  // q / copies
            const uint32_t j = q - r * d.copies;
            const CopyLoc c = locate_copy(d, P, r, j);
            const V x = from_send ? ld_cg<V>(reinterpret_cast<const V*>(g.base[SPACE_SEND] + (uint64_t)r * g.m) + v)
                                  : msrc[(c.src_rank * P + c.src_slot) * vps + v];
            const uint32_t at = (c.dst_rank * P + c.dst_slot) * vps + v;
            mdst[at] = x;
            st_cg<V>(gdst + at, x);
            if (d.dup_self) {
                const uint32_t at2 = (r * P + c.dst_slot) * vps + v;
                mdst[at2] = x;
                st_cg<V>(gdst + at2, x);
            }
        }
    }
}

// The first passes of a collective as INDEPENDENT small collectives.  Sparbit: while the step distance
// is still a multiple of G (a power of two that divides P), a rank only ever exchanges blocks with
// ranks of its own residue class mod G, and only blocks whose index is in that class too: the P
// ranks fall into G groups of R = P / G ranks that do not talk to each other.  Recursive doubling
// starts at the other end: while the distance is below R = 2^s, partners (r xor 2^i) and slots stay
// inside the aligned run of R consecutive ranks r belongs to.  Either way each group's part of the
// receive buffers - R ranks x R slots - is small even when the whole is not, so one CTA per group
// runs those passes from an on-chip copy exactly as mirror_vec_kernel does for a whole collective
// (same copies, same slots, written through to global memory); the passes after them run as the
// usual per-pass kernels and read what this kernel wrote.  grid = G CTAs.
template <typename V>
__global__ void __launch_bounds__(1024, 1) grouped_mirror_vec_kernel(Geom g, const __grid_constant__ MirrorArgs ma) {
    // [R][R] slots of m bytes.  Residue classes: local rank i is rank c + i * G, local slot k is
    // slot c + k * G.  Aligned runs: local rank i is rank c * R + i, local slot k is slot c * R + k.
    extern __shared__ __align__(16) unsigned char mirror[];
    chain_trigger();
    chain_wait();
    const uint32_t P = g.P;
    const uint32_t c = blockIdx.x;
    const uint32_t lgG = 31u - (uint32_t)__clz(gridDim.x);
    const uint32_t R = P >> lgG;
    const bool aligned = ma.aligned != 0;
    const uint32_t vps = (uint32_t)(g.m / sizeof(V));  // vectors per slot
    V* mir = reinterpret_cast<V*>(mirror);
    const V* gsend = reinterpret_cast<const V*>(g.base[SPACE_SEND]);
    V* grecv = reinterpret_cast<V*>(g.base[SPACE_RECV]);
    auto local = [&](uint32_t x) { return aligned ? x - c * R : x >> lgG; };  // of a rank or slot of this group
    for (int i = 0; i < ma.n; i++) {
        if (i) __syncthreads();
        const PhaseDesc& d = ma.d[i];
        const uint32_t vpc = (uint32_t)(d.copy_bytes / sizeof(V));
        const uint32_t total = R * d.copies * vpc;
        const bool from_send = d.src_space == SPACE_SEND;
        const unsigned long long mv = ma.magic_vpc[i], mc = ma.magic_copies[i];
        for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
            const uint32_t q = (uint32_t)((t * mv) >> 40);   // t / vpc
            const uint32_t v = t - q * vpc;
            const uint32_t li = (uint32_t)((q * mc) >> 40);  // q / copies: local rank of the sender
            const uint32_t j = q - li * d.copies;
            const uint32_t r = aligned ? c * R + li : c + (li << lgG);
            const CopyLoc loc = locate_copy(d, P, r, j);
            const V x = from_send ? ld_cg<V>(gsend + (uint64_t)r * vps + v) : mir[(li * R + local(loc.src_slot)) * vps + v];
            const uint32_t ls = local(loc.dst_slot);
            mir[(local(loc.dst_rank) * R + ls) * vps + v] = x;
            st_cg<V>(grecv + ((uint64_t)loc.dst_rank * P + loc.dst_slot) * vps + v, x);
            if (d.dup_self) {
                mir[(li * R + ls) * vps + v] = x;
                st_cg<V>(grecv + ((uint64_t)r * P + loc.dst_slot) * vps + v, x);
            }
        }
    }
}

// The same for blocks of DIFFERENT sizes (allgatherv), in one CTA: the passes' work comes as the task
// lists the list kernels use (byte offsets inside the source and destination space, at most
// kVarSegmentBytes each), a group of lanes per task; the on-chip copy is laid out like the receive space
// (rank r's buffer at r times the sum of all block sizes).
struct MirrorListPass {
    const VarTask* list;
    unsigned long long count;
    uint32_t src_space, dst_space, dup_self;
    uint32_t group;  // lanes that share a task (a power of two, 4..32): about the vectors of an average task
};
struct MirrorListArgs {
    MirrorListPass pass[kMirrorMaxPasses];
    int n;
    int pad_[3];
};

template <typename V>
__global__ void __launch_bounds__(1024, 1) mirror_list_kernel(Geom g, const __grid_constant__ MirrorListArgs ma) {
    extern __shared__ __align__(16) unsigned char mirror[];
    chain_trigger();
    chain_wait();
    V* mir = reinterpret_cast<V*>(mirror);
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t n_warps = blockDim.x >> 5;
    const long long pitch = (long long)g.rank_pitch[SPACE_RECV];  // bytes of one receive buffer
    for (int i = 0; i < ma.n; i++) {
        if (i) __syncthreads();
        const MirrorListPass& ps = ma.pass[i];
        const bool from_send = ps.src_space == SPACE_SEND;
        const char* sbase = g.base[SPACE_SEND];
        char* dbase = g.base[SPACE_RECV];
        const uint32_t G = ps.group, sub = lane & (G - 1u), grp = lane / G, groups = 32u / G;
        // a warp fetches 32 task records at once (one per lane: one trip to memory instead of 32),
        // then its groups of G lanes take them one after the other
        // (each warp takes a contiguous slice of the list, as even as they come)
        const uint32_t count = (uint32_t)ps.count;  // a list has fewer than 2^27 entries (host-checked)
        const uint32_t per = (count + n_warps - 1u) / n_warps;
        const uint32_t lo = warp * per;
        const uint32_t hi = lo + per < count ? lo + per : count;
        for (uint32_t t0 = lo; t0 < hi; t0 += 32u) {
            VarTask mine;
            mine.a = mine.b = 0;
            if (t0 + lane < hi) mine = ld_task(ps.list + t0 + lane);
            const uint32_t have = hi - t0 < 32u ? hi - t0 : 32u;
            for (uint32_t k0 = 0; k0 < have; k0 += groups) {
                const uint32_t k = k0 + grp;
                VarTask e;
                e.a = __shfl_sync(0xffffffffu, mine.a, (int)(k & 31u));
                e.b = __shfl_sync(0xffffffffu, mine.b, (int)(k & 31u));
                if (k >= have) continue;
                const unsigned long long soff = e.a & kVarOffsetMask;
                const unsigned long long doff = e.b & kVarOffsetMask;
                const long long doff2 = (long long)doff + (long long)(short)(e.b >> 48) * pitch;  // dup_self: the sender's own buffer
                const uint32_t vectors = ((uint32_t)(e.a >> 48) + 1u) / (uint32_t)sizeof(V);
                for (uint32_t v = sub; v < vectors; v += G) {
                    const V x = from_send ? ld_cg<V>(reinterpret_cast<const V*>(sbase + soff) + v) : mir[soff / sizeof(V) + v];
                    mir[doff / sizeof(V) + v] = x;
                    st_cg<V>(reinterpret_cast<V*>(dbase + doff) + v, x);
                    if (ps.dup_self) {
                        mir[(unsigned long long)doff2 / sizeof(V) + v] = x;
                        st_cg<V>(reinterpret_cast<V*>(dbase + doff2) + v, x);
                    }
                }
            }
        }
    }
}

// The same idea on a thread-block CLUSTER, for collectives whose receive buffers fit into the
// shared memory of up to 16 SMs together: rank r's on-chip copy lives in CTA r mod C of the cluster
// (ranks c, c+C, c+2C, ... one after the other).  A CTA executes the copies its own ranks SEND: it
// reads the block from its local shared memory and stores it into the destination rank's CTA through
// distributed shared memory (st.shared::cluster) and into global memory; the hardware cluster barrier
// (arrive.release / wait.acquire) is the Waitall.  A pass costs a shared-memory read, a posted remote
// write and that barrier.  The last barrier keeps every CTA alive until nobody writes into it any more.
// (The barrier's release also waits for the pass's global stores, one of the two round trips the
// mirror is there to avoid: this form runs vectors of 1 and 2 bytes only, which st.async does not
// move; wider vectors take cluster_mirror_async_kernel below.)
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_shared_addr, uint32_t cta) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_shared_addr), "r"(cta));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
template <typename V>
__device__ __forceinline__ void st_cluster(uint32_t addr, V v);
template <>
__device__ __forceinline__ void st_cluster<uint4>(uint32_t addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
template <>
__device__ __forceinline__ void st_cluster<uint2>(uint32_t addr, uint2 v) {
    asm volatile("st.shared::cluster.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(v.x), "r"(v.y) : "memory");
}
template <>
__device__ __forceinline__ void st_cluster<unsigned>(uint32_t addr, unsigned v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
template <>
__device__ __forceinline__ void st_cluster<unsigned short>(uint32_t addr, unsigned short v) {
    asm volatile("st.shared::cluster.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
template <>
__device__ __forceinline__ void st_cluster<unsigned char>(uint32_t addr, unsigned char v) {
    asm volatile("st.shared::cluster.u8 [%0], %1;" ::"r"(addr), "r"((uint32_t)v) : "memory");
}

template <typename V>
__global__ void __launch_bounds__(1024, 1) cluster_mirror_vec_kernel(Geom g, const __grid_constant__ MirrorArgs ma) {
    // this CTA's ranks (c, c + C, ...), each [P] slots of m bytes; for Bruck the working buffers behind
    extern __shared__ __align__(16) unsigned char mirror[];
    chain_trigger();
    chain_wait();
    const uint32_t P = g.P;
    const uint32_t C = cluster_nctarank();
    const uint32_t c = cluster_ctarank();
    const uint32_t mine = c < P ? (P - c + C - 1) / C : 0u;  // ranks this CTA holds
    const uint32_t vps = (uint32_t)(g.m / sizeof(V));        // vectors per slot
    V* mir = reinterpret_cast<V*>(mirror);
    const uint32_t mir_base = smem_u32(mirror);
    for (int i = 0; i < ma.n; i++) {
        // every CTA of the cluster passes here the same number of times: the Waitall, and before
        // the first pass the guarantee that all CTAs of the cluster have started
        cluster_sync_all();
        const PhaseDesc& d = ma.d[i];
        const uint32_t vpc = (uint32_t)(d.copy_bytes / sizeof(V));
        const uint32_t total = mine * d.copies * vpc;
        const bool from_send = d.src_space == SPACE_SEND;
        const uint32_t src_at = d.src_space == SPACE_WORK ? ma.work_at : 0u;
        const uint32_t dst_at = d.dst_space == SPACE_WORK ? ma.work_at : 0u;
        V* gdst = reinterpret_cast<V*>(space_base(g, d.dst_space));
        for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
            const uint32_t q = t / vpc;
            const uint32_t v = t - q * vpc;
            const uint32_t lr = q / d.copies;  // which of this CTA's ranks sends
            const uint32_t j = q - lr * d.copies;
            const uint32_t r = c + lr * C;
            const CopyLoc loc = locate_copy(d, P, r, j);
            const V x = from_send ? ld_cg<V>(reinterpret_cast<const V*>(g.base[SPACE_SEND] + (uint64_t)r * g.m) + v)
                                  : mir[src_at + (lr * P + loc.src_slot) * vps + v];
            // the receiving rank's copy: CTA dst_rank mod C, its (dst_rank / C)-th rank
            const uint32_t there = dst_at + ((loc.dst_rank / C) * P + loc.dst_slot) * vps + v;
            st_cluster<V>(map_to_cta(mir_base + there * (uint32_t)sizeof(V), loc.dst_rank % C), x);
            st_cg<V>(gdst + (loc.dst_rank * P + loc.dst_slot) * vps + v, x);
            if (d.dup_self) {
                mir[dst_at + (lr * P + loc.dst_slot) * vps + v] = x;
                st_cg<V>(gdst + (r * P + loc.dst_slot) * vps + v, x);
            }
        }
    }
    cluster_sync_all();  // nobody leaves while a neighbour may still store into its shared memory
}

// The cluster form without a barrier between the passes, for vectors of 4, 8 and 16 bytes.  A copy
// is pushed with st.async: the store into the receiving CTA's shared memory completes bytes on an
// mbarrier IN THAT CTA, one mbarrier per pass, armed at the start with the bytes the CTA's ranks
// receive in that pass (every rank receives `copies` blocks of `copy_bytes` per pass, twice that
// when the pass also files the own block).  What a rank sends in pass i it has received in passes
// before i, and its on-chip copy sits in the CTA that sends for it, so a CTA's Waitall is a wait on
// its OWN mbarriers of the passes before: no round trip, no cluster-wide barrier, and the global
// stores of a pass are not waited for before the next one starts (nobody reads them in this
// kernel; they are complete when the kernel is).  No slot is written twice within a collective, so
// a CTA that runs ahead cannot overwrite what a slower one still reads.  Waits are bounded; a wait
// that gives up sets the status word and the thread goes to the final cluster barrier.
template <typename V>
__device__ __forceinline__ void st_async_cluster(uint32_t addr, V v, uint32_t bar);
template <>
__device__ __forceinline__ void st_async_cluster<uint4>(uint32_t addr, uint4 v, uint32_t bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
                 "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(bar)
                 : "memory");
}
template <>
__device__ __forceinline__ void st_async_cluster<uint2>(uint32_t addr, uint2 v, uint32_t bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];" ::"r"(addr), "r"(v.x),
                 "r"(v.y), "r"(bar)
                 : "memory");
}
template <>
__device__ __forceinline__ void st_async_cluster<unsigned>(uint32_t addr, unsigned v, uint32_t bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(addr), "r"(v), "r"(bar)
                 : "memory");
}

template <typename V>
__global__ void __launch_bounds__(1024, 1) cluster_mirror_async_kernel(Geom g, const __grid_constant__ MirrorArgs ma) {
    extern __shared__ __align__(16) unsigned char mirror[];
    __shared__ __align__(8) unsigned long long pass_bar[kMirrorMaxPasses];
    chain_trigger();
    const uint32_t P = g.P;
    const uint32_t C = cluster_nctarank();
    const uint32_t c = cluster_ctarank();
    const uint32_t mine = c < P ? (P - c + C - 1) / C : 0u;  // ranks this CTA holds
    const uint32_t vps = (uint32_t)(g.m / sizeof(V));        // vectors per slot
    V* mir = reinterpret_cast<V*>(mirror);
    const uint32_t mir_base = smem_u32(mirror);
    const uint32_t bar_base = smem_u32(pass_bar);
    const uint32_t lgC = 31u - (uint32_t)__clz(C);  // cluster sizes are powers of two
    if (threadIdx.x == 0) {
        for (int i = 0; i < ma.n; i++) mbar_init(bar_base + 8u * i, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < ma.n; i++) {
            const PhaseDesc& d = ma.d[i];
            mbar_expect_tx(bar_base + 8u * i, mine * d.copies * (uint32_t)d.copy_bytes * (d.dup_self ? 2u : 1u) + ma.extra_tx);
        }
    }
    cluster_sync_all();  // every CTA of the cluster runs and its mbarriers are armed
    chain_wait();        // (all of the above touches no global memory: it overlaps the kernel before)
    bool ok = true;
    for (int i = 0; i < ma.n && ok; i++) {
        // the Waitall of the pass before, for this CTA's ranks (all threads, so that a thread
        // without work in some pass has still seen every earlier pass arrive)
        // (every thread polls: measured faster than one poller per warp or per CTA handing the
        // result on)
        if (i > 0) ok = mbar_wait_bounded(bar_base + 8u * (i - 1), 0u, ma.status, ma.timeout_ns);
        if (!ok) break;
        const PhaseDesc& d = ma.d[i];
        const uint32_t vpc = (uint32_t)(d.copy_bytes / sizeof(V));
        const uint32_t total = mine * d.copies * vpc;
        const bool from_send = d.src_space == SPACE_SEND;
        const uint32_t src_at = d.src_space == SPACE_WORK ? ma.work_at : 0u;
        const uint32_t dst_at = d.dst_space == SPACE_WORK ? ma.work_at : 0u;
        const uint32_t bar = bar_base + 8u * i;
        V* gdst = reinterpret_cast<V*>(space_base(g, d.dst_space));
        const unsigned long long mv = ma.magic_vpc[i], mc = ma.magic_copies[i];
        const V* gsend = reinterpret_cast<const V*>(g.base[SPACE_SEND]);
        for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
            const uint32_t q = (uint32_t)((t * mv) >> 40);   // t / vpc
            const uint32_t v = t - q * vpc;
            const uint32_t lr = (uint32_t)((q * mc) >> 40);  // q / copies: which of this CTA's ranks sends
            const uint32_t j = q - lr * d.copies;
            const uint32_t r = c + (lr << lgC);
            const CopyLoc loc = locate_copy(d, P, r, j);
            const V x = from_send ? ld_cg<V>(gsend + (uint64_t)r * vps + v) : mir[src_at + (lr * P + loc.src_slot) * vps + v];
            // the receiving rank's copy: CTA dst_rank mod C, its (dst_rank / C)-th rank
            const uint32_t to = loc.dst_rank & (C - 1u);
            const uint32_t there = dst_at + ((loc.dst_rank >> lgC) * P + loc.dst_slot) * vps + v;
            st_async_cluster<V>(map_to_cta(mir_base + there * (uint32_t)sizeof(V), to), x, map_to_cta(bar, to));
            st_cg<V>(gdst + (loc.dst_rank * P + loc.dst_slot) * vps + v, x);
            if (d.dup_self) {
                const uint32_t here = dst_at + (lr * P + loc.dst_slot) * vps + v;
                st_async_cluster<V>(map_to_cta(mir_base + here * (uint32_t)sizeof(V), c), x, map_to_cta(bar, c));
                st_cg<V>(gdst + (r * P + loc.dst_slot) * vps + v, x);
            }
        }
    }
    // nothing may still be on its way into this CTA when it leaves, and no CTA leaves before the others
    if (ok) mbar_wait_bounded(bar_base + 8u * (ma.n - 1), 0u, ma.status, ma.timeout_ns);
    __syncwarp();  // threads that gave up in different passes meet again before the aligned barrier
    cluster_sync_all();
}

// ------------------------------------------------------------------------------------------------
// flow executor: the whole collective in one cooperative kernel WITHOUT grid-wide barriers
// ------------------------------------------------------------------------------------------------
// Algorithm 1 ends every step with MPI_Waitall, but what a rank sends in step i+1 depends only on
// what THAT rank has received in the steps before.  So the Waitall is kept per rank instead of per
// grid: a (rank, pass) counter counts the finished work units that wrote into that rank's buffer
// in that pass, and a unit that reads rank r in pass i first waits until the counters of rank r
// for every earlier pass that writes the space it reads have reached their final value.  Blocks
// still travel exactly as the schedule says (each forwarded block is read from the sending
// rank's receive buffer after that rank has received it); only the idle time at the pass
// boundaries goes away, because warps that are done with pass i start on pass i+1 while others
// are still busy.
//
// A unit is up to `us` consecutive warp spans (32*U vectors each) of the copies ONE rank sends
// in one pass: one source rank, one destination rank, hence one dependency and one counter.
// Units are numbered pass by pass and dealt to the warps round robin, every warp taking its units
// in increasing order; the unit with the smallest number that is not finished never waits for a
// later one, so the scheme cannot deadlock while all CTAs are resident (cooperative launch).
// Within a pass the ranks are enumerated from `rot` on, chosen by the host so that a unit's
// producers sit at about the same relative position of the pass before.
//
// Counters are never reset between collectives: the host passes, per pass, the value they reach
// at the end of THIS launch (launch number times units per rank).
constexpr int kFlowMaxPasses = 32;  // a rank's counters fill one 128-byte line

struct FlowPass {
    uint32_t upr;       // units per source rank
    uint32_t us;        // spans per unit (the last unit of a rank may hold fewer)
    uint32_t spc;       // spans per copy
    uint32_t rot;       // position x of the pass handles source rank (x + rot) mod P
    uint32_t target;    // counter value of a (rank, this pass) when all its units of this launch are done
    uint32_t dep_mask;  // bit k: pass k (< this one) writes the space this pass reads
    uint32_t eager;     // 1: no warp has a second unit in this pass - signal a unit as soon as it is stored
    uint32_t pad_;
};
struct FlowArgs {
    FlowPass pass[kFlowMaxPasses];
    uint32_t n;
    uint32_t pad_;
    unsigned* cnt;      // [P][kFlowMaxPasses]
    unsigned* status;
    unsigned long long timeout_ns;
};

__device__ __forceinline__ void red_relaxed_gpu_add(unsigned* p, unsigned v) {
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

template <typename V, int U>
__global__ void __launch_bounds__(512, 2) flow_vec_kernel(Geom g, const PhaseDesc* __restrict__ descs, int first_idx,
                                                          const __grid_constant__ FlowArgs fa) {
    __shared__ PhaseDesc sd[kFlowMaxPasses];
    __shared__ uint32_t s_target[kFlowMaxPasses];
    for (uint32_t k = threadIdx.x; k < fa.n * 16u; k += blockDim.x)
        reinterpret_cast<uint32_t*>(sd)[k] = reinterpret_cast<const uint32_t*>(descs + first_idx)[k];
    if (threadIdx.x < kFlowMaxPasses) s_target[threadIdx.x] = threadIdx.x < fa.n ? fa.pass[threadIdx.x].target : 0u;
    __syncthreads();
    chain_trigger();
    chain_wait();  // the collective before this one in the stream is complete
    if (ld_relaxed_gpu(fa.status) != DEV_OK) return;  // an earlier failure was not cleared yet
    const uint32_t P = g.P;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wpb = blockDim.x >> 5;
    const uint32_t n_warps = gridDim.x * wpb;
    const uint32_t warp_id = blockIdx.x * wpb + (threadIdx.x >> 5);
    constexpr uint32_t span = 32u * U;

    // completion of the unit before: signalled after the next unit's first loads are on their
    // way (the fence then waits for stores that have long been issued), or before any wait
    unsigned* pend0 = nullptr;
    unsigned* pend1 = nullptr;
    auto flush = [&]() {
        if (pend0) {
            __syncwarp();
            if (lane == 0) {
                fence_acq_rel_gpu();  // the unit's stores (all lanes, ordered by the warp barrier) first
                red_relaxed_gpu_add(pend0, 1u);
                if (pend1) red_relaxed_gpu_add(pend1, 1u);
            }
            pend0 = pend1 = nullptr;
        }
    };

    uint64_t g0 = 0;  // number of the pass's first unit
    for (uint32_t i = 0; i < fa.n; i++) {
        const FlowPass fp = fa.pass[i];
        const PhaseDesc& d = sd[i];
        const uint32_t units = P * fp.upr;  // < 2^32, host-checked
        const uint32_t spans_per_rank = d.copies * fp.spc;
        const uint64_t vpc64 = d.copy_bytes / sizeof(V);
        const char* sbase = space_base(g, d.src_space);
        char* dbase = space_base(g, d.dst_space);
        const uint64_t spitch = space_pitch(g, d.src_space);
        const uint64_t dpitch = space_pitch(g, d.dst_space);
        const bool polls = lane < i && ((fp.dep_mask >> lane) & 1u);
        uint32_t w = (warp_id + n_warps - (uint32_t)(g0 % n_warps)) % n_warps;
        for (; w < units; w += n_warps) {
            const uint32_t x = w / fp.upr;
            const uint32_t k = w - x * fp.upr;
            uint32_t r = x + fp.rot;
            if (r >= P) r -= P;
            // the Waitall of rank r: everything it receives before this pass has arrived
            if (fp.dep_mask) {
                const unsigned* line = fa.cnt + (size_t)r * kFlowMaxPasses;
                bool ok = !polls || (int)(ld_acquire_gpu(line + lane) - s_target[lane]) >= 0;
                if (!__all_sync(0xffffffffu, ok)) {
                    flush();
                    const unsigned long long t0 = globaltimer_ns();
                    unsigned tries = 0;
                    for (;;) {
                        ok = !polls || (int)(ld_acquire_gpu(line + lane) - s_target[lane]) >= 0;
                        if (__all_sync(0xffffffffu, ok)) break;
                        if ((++tries & 15u) == 0) {
                            bool give_up = false;
                            if (lane == 0) {
                                if (ld_relaxed_gpu(fa.status) != DEV_OK) give_up = true;
                                else if (globaltimer_ns() - t0 > fa.timeout_ns) {
                                    atomicCAS(fa.status, DEV_OK, DEV_BARRIER_TIMEOUT);
                                    give_up = true;
                                }
                            }
                            if (__any_sync(0xffffffffu, give_up)) return;
                        }
                    }
                }
                __syncwarp();  // what one lane acquired, all lanes may read
            }
            const uint32_t s0 = k * fp.us;
            uint32_t s1 = s0 + fp.us;
            if (s1 > spans_per_rank) s1 = spans_per_rank;
            uint32_t j = s0 / fp.spc;
            uint32_t sp = s0 - j * fp.spc;
            uint32_t dst_rank = 0;
            for (uint32_t s = s0; s < s1; s++) {
                const CopyLoc c = locate_copy(d, P, r, j);
                dst_rank = c.dst_rank;
                const V* src = reinterpret_cast<const V*>(sbase + ((uint64_t)c.src_rank * spitch + (uint64_t)c.src_slot * g.m));
                V* dst = reinterpret_cast<V*>(dbase + ((uint64_t)c.dst_rank * dpitch + (uint64_t)c.dst_slot * g.m));
                V* dst2 = reinterpret_cast<V*>(dbase + ((uint64_t)r * dpitch + (uint64_t)c.dst_slot * g.m));
                const uint64_t v0 = (uint64_t)sp * span + lane;
                V regs[U];
#pragma unroll
                for (int q = 0; q < U; q++) {
                    const uint64_t v = v0 + 32u * q;
                    if (v < vpc64) regs[q] = ld_cg<V>(src + v);
                }
                if (s == s0) flush();
#pragma unroll
                for (int q = 0; q < U; q++) {
                    const uint64_t v = v0 + 32u * q;
                    if (v < vpc64) {
                        st_cg<V>(dst + v, regs[q]);
                        if (d.dup_self) st_cg<V>(dst2 + v, regs[q]);
                    }
                }
                if (++sp == fp.spc) {
                    sp = 0;
                    j++;
                }
            }
            pend0 = fa.cnt + (size_t)dst_rank * kFlowMaxPasses + i;
            pend1 = d.dup_self && dst_rank != r ? fa.cnt + (size_t)r * kFlowMaxPasses + i : nullptr;
            if (fp.eager) flush();
        }
        g0 += units;
    }
    flush();
}

}  // namespace spb
