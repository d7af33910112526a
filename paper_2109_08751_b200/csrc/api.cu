// C ABI of the step executor: plans, argument checks, executor selection and launches.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "../../include/sparbit.h"
#include "kernels.cuh"
#include "schedule.h"

using namespace spb;

namespace {

thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", what, cudaGetErrorString(e));
    return SPARBIT_ERR_CUDA;
}
#define CU(call)                                         \
    do {                                                 \
        cudaError_t e_ = (call);                         \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

constexpr unsigned long long kDefaultTimeoutNs = 2000000000ull;  // 2 s
constexpr int kVecBlock = 512;
// Dynamic shared memory a per-pass vector kernel with a FULL grid (two CTAs per SM) asks for
// without using it: it caps the kernel at two CTAs per SM whatever its register count, so that a
// chained successor cannot squeeze a third CTA onto some SMs while the others get one (measured at
// P = 1000, m = 1 KiB: 348 us without the cap, 339 us with it).  Small grids do not ask for it:
// there the early residency of the successor is what keeps a pass at 2.6 us.
constexpr size_t kVecOccupancySmem = 100 * 1024;

struct GraphKey {
    const void* send = nullptr;
    void* recv = nullptr;
    void* work = nullptr;
    int first = 0, last = -2;
    int path = 0, vec = 0, exec = 0;
    unsigned long long timeout_ns = 0;
    unsigned extra_tx = 0;
    bool same_shape(const GraphKey& o) const {
        return first == o.first && last == o.last && path == o.path && vec == o.vec && exec == o.exec &&
               timeout_ns == o.timeout_ns && extra_tx == o.extra_tx;
    }
    bool same_buffers(const GraphKey& o) const { return send == o.send && recv == o.recv && work == o.work; }
};

}  // namespace

struct sparbit_plan_s {
    Schedule sched;
    int exec_req = SPARBIT_EXEC_AUTO;
    int copy_req = SPARBIT_COPY_AUTO;
    int copy_last = SPARBIT_COPY_AUTO;
    int exec_last = SPARBIT_EXEC_AUTO;
    void* work = nullptr;
    size_t work_bytes = 0;

    // variable block sizes (allgatherv): prefix sums of the byte counts, P+1 entries
    bool variable = false;
    std::vector<uint64_t> voff;
    uintptr_t voff_bits = 0;  // OR of all prefix sums: decides the vector width
    // task lists of the variable-size kernels, one per descriptor of the device table order
    // (phases in order, then the fused first pass): entries, and where each list starts
    std::vector<VarTask> vtasks;
    std::vector<size_t> vtask_lo, vtask_hi;  // per device-table index: [lo, hi) inside vtasks
    VarTask* d_vtasks = nullptr;
    VarRange* d_vranges = nullptr;           // the same ranges on the device (persistent executor)

    size_t send_bytes() const { return variable ? (size_t)voff.back() : (size_t)sched.P * sched.m; }
    size_t recv_bytes() const { return (size_t)sched.P * send_bytes(); }

    // device side, created by the first launch
    bool dev_ready = false;
    bool dev_touched = false;  // set-up was attempted: something may have been allocated
    int device = -1;
    int sm_count = 0;
    int coop = 0;
    int max_smem_optin = 0;
    PhaseDesc* d_descs = nullptr;
    unsigned* d_ctl = nullptr;  // [0] barrier counter, [1] status word
    unsigned* d_flow_cnt = nullptr;  // flow executor: [P][kFlowMaxPasses] unit counters
    unsigned flow_epoch = 0;         // flow launches since the counters were last cleared
    int flow_vbytes = 0;             // vector width and vectors per lane (width * 16 + unroll) of those launches
    // what resolve() gave for (vector width, phase range) under the current settings: the automatic
    // choices walk the schedule several times, too much for every call of a 2 us collective
    struct {
        bool valid = false;
        int vbytes = 0, first = 0, last = 0;
        uint64_t version = 0;
        int exec = 0, copy = 0;
    } resolved;
    uint64_t settings_version = 0;  // bumped by every setter the automatic choices depend on
    // the grouped front of the stream executor for (vector width, phase range), under the same version
    struct {
        bool valid = false;
        int vbytes = 0, first = 0, last = 0;
        uint64_t version = 0;
        int front = 0;
        uint32_t groups = 1;
    } front_cache;
    unsigned bar_base = 0;
    int extra_arrivals = 0;
    unsigned long long timeout_ns = kDefaultTimeoutNs;
    unsigned mbar_extra_tx = 0;  // test hook of the bulk engine's bounded mbarrier wait

    // bulk engine geometry
    // measured on B200: about 32 KiB of loads in flight per SM is the sweet spot for a copy (more
    // lowers the achieved HBM bandwidth): 4 rings x 2 loads x 4 KiB
    uint32_t bulk_warps = 4;
    uint32_t bulk_stage_bytes = 4096;

    // thresholds of the automatic choices (sparbit_plan_set_tunable); defaults from measured sweeps
    uint64_t tune[SPARBIT_TUNE_COUNT_] = {
        8u << 10,     // BULK_MIN_BLOCK_BYTES
        1000000000u,  // BULK_MIN_MOVED_BYTES
        1,            // FLOW_UNITS_PER_WARP
        8,            // FLOW_MAX_UNIT_SPANS
        400000000u,   // FLOW_MIN_MOVED_BYTES
        6000000000ull,  // FLOW_MAX_MOVED_BYTES
        64u << 10,    // MIRROR_MAX_BYTES
        1,            // FLOW_MIN_PASS_SPANS (every pass; 0: passes of at least one span per resident warp)
        65536,        // MIRROR_MAX_VECTORS
        4096,         // MIRROR_CLUSTER_MAX_BLOCK
        256,          // MIRROR_CTA_VECTORS
        4,            // MIRROR_THREAD_VECTORS
        0,            // FLOW_COOPERATIVE
        0,            // FLOW_SKIP_WAITS
        1,            // GROUPED_FRONT
        900000000u,   // FLOW_WIDE_MAX_MOVED_BYTES
        256u << 20,   // VEC_DENSE_MAX_RECV_BYTES
        6,            // STREAM_MAX_LAUNCHES
    };

    // cached graphs: one instantiated chain per (buffers, phase range, engine), a few of them so
    // that callers alternating between buffer sets never re-instantiate
    struct GraphEntry {
        GraphKey key;
        cudaGraphExec_t exec = nullptr;
        uint64_t stamp = 0;
        uint64_t kernels = 0;  // kernel nodes of the graph
    };
    std::vector<GraphEntry> gcache;
    uint64_t gstamp = 0;
    cudaStream_t capture_stream = nullptr;

    // host-buffer entry point
    void* stage_send = nullptr;
    void* stage_recv = nullptr;
    void* stage_work = nullptr;

    // per-pass time stamps of the persistent executor (off by default)
    bool trace_on = false;
    unsigned long long* d_trace = nullptr;
    size_t trace_cap = 0, trace_len = 0;

    cudaStream_t last_stream = nullptr;
    bool launched = false;
    uint64_t kernel_launches = 0, graph_launches = 0;
};

namespace {

// SPARBIT_EXEC / SPARBIT_COPY in the environment override what AUTO would pick (not an explicit
// request): persistent|graph|stream|flow|mirror and vector|bulk.  Anything else is ignored.
int env_choice(const char* name, const char* const* words, const int* values, int n, int fallback) {
    const char* v = getenv(name);
    if (!v) return fallback;
    for (int i = 0; i < n; i++)
        if (strcmp(v, words[i]) == 0) return values[i];
    return fallback;
}
int env_exec(int fallback) {
    static const char* const w[] = {"persistent", "graph", "stream", "flow", "mirror"};
    static const int x[] = {SPARBIT_EXEC_PERSISTENT, SPARBIT_EXEC_GRAPH, SPARBIT_EXEC_STREAM, SPARBIT_EXEC_FLOW,
                            SPARBIT_EXEC_MIRROR};
    return env_choice("SPARBIT_EXEC", w, x, 5, fallback);
}
int env_copy(int fallback) {
    static const char* const w[] = {"vector", "bulk"};
    static const int x[] = {SPARBIT_COPY_VECTOR, SPARBIT_COPY_BULK};
    return env_choice("SPARBIT_COPY", w, x, 2, fallback);
}

int map_sched_err(int e) {
    switch (e) {
        case SCHED_OK: return SPARBIT_OK;
        case SCHED_ARG: return SPARBIT_ERR_ARG;
        case SCHED_OVERFLOW: return SPARBIT_ERR_OVERFLOW;
        case SCHED_UNSUPPORTED: return SPARBIT_ERR_UNSUPPORTED;
        default: return SPARBIT_ERR_ARG;
    }
}

size_t bulk_smem_bytes(const sparbit_plan_s* p) {
    return (size_t)p->bulk_warps * (kBulkStages * (p->bulk_stage_bytes + 8 + 32) + kTaskQueue * 16);
}

const void* pick_phase_vec(int vbytes);

int ensure_device(sparbit_plan_s* p) {
    if (p->dev_ready) {
        // a plan belongs to the device of its first launch
        int cur = -1;
        CU(cudaGetDevice(&cur));
        return cur == p->device ? SPARBIT_OK : SPARBIT_ERR_ARG;
    }
    p->dev_touched = true;
    CU(cudaGetDevice(&p->device));
    CU(cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device));
    CU(cudaDeviceGetAttribute(&p->coop, cudaDevAttrCooperativeLaunch, p->device));
    CU(cudaDeviceGetAttribute(&p->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, p->device));
    // shrink the bulk ring if this device offers less shared memory than planned
    while (bulk_smem_bytes(p) > (size_t)p->max_smem_optin && p->bulk_stage_bytes > 1024) p->bulk_stage_bytes -= 1024;
    // descriptor table: the phases in order, then (if the schedule has one) the same sequence with
    // phases -1 and 0 replaced by the fused first pass
    std::vector<PhaseDesc> table = p->sched.phases;
    if (p->sched.has_fused_first) {
        table.push_back(p->sched.fused_first);
        table.insert(table.end(), p->sched.phases.begin() + 2, p->sched.phases.end());
    }
    // a set-up that failed half way is run again by the next launch: what it already allocated is
    // kept and filled again, never allocated twice
    const size_t n = table.size();
    if (!p->d_descs) CU(cudaMalloc((void**)&p->d_descs, n * sizeof(PhaseDesc)));
    CU(cudaMemcpy(p->d_descs, table.data(), n * sizeof(PhaseDesc), cudaMemcpyHostToDevice));
    if (p->variable) {
        const size_t nt = p->vtasks.size() ? p->vtasks.size() : 1;
        if (!p->d_vtasks) CU(cudaMalloc((void**)&p->d_vtasks, nt * sizeof(VarTask)));
        if (p->vtasks.size())
            CU(cudaMemcpy(p->d_vtasks, p->vtasks.data(), p->vtasks.size() * sizeof(VarTask), cudaMemcpyHostToDevice));
        std::vector<VarRange> ranges(p->vtask_lo.size());
        for (size_t i = 0; i < ranges.size(); i++) {
            ranges[i].lo = p->vtask_lo[i];
            ranges[i].count = p->vtask_hi[i] - p->vtask_lo[i];
        }
        if (!p->d_vranges) CU(cudaMalloc((void**)&p->d_vranges, ranges.size() * sizeof(VarRange)));
        CU(cudaMemcpy(p->d_vranges, ranges.data(), ranges.size() * sizeof(VarRange), cudaMemcpyHostToDevice));
    }
    if (!p->d_ctl) CU(cudaMalloc((void**)&p->d_ctl, 2 * sizeof(unsigned)));
    CU(cudaMemset(p->d_ctl, 0, 2 * sizeof(unsigned)));
    for (int vb = 1; vb <= 16; vb *= 2) {
        CU(cudaFuncSetAttribute(pick_phase_vec(vb), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kVecOccupancySmem));
    }
    CU(cudaFuncSetAttribute(phase_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            (int)bulk_smem_bytes(p)));
    CU(cudaFuncSetAttribute(persistent_bulk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            (int)bulk_smem_bytes(p)));
    CU(cudaFuncSetAttribute(persistent_bulk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            (int)bulk_smem_bytes(p)));
    CU(cudaFuncSetAttribute(phase_bulk_list_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            (int)bulk_smem_bytes(p)));
    p->dev_ready = true;
    return SPARBIT_OK;
}

bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb) {
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
    return x < y + nb && y < x + na;
}

// largest power-of-two vector width (<= 16) that divides every address and m
int pick_vector_bytes(const sparbit_plan_s* p, const void* send, const void* recv) {
    uintptr_t bits = (uintptr_t)send | (uintptr_t)recv;
    bits |= p->variable ? p->voff_bits : (uintptr_t)p->sched.m;
    if (p->sched.algo == ALGO_BRUCK) bits |= (uintptr_t)p->work;
    int v = 16;
    while (v > 1 && (bits & (uintptr_t)(v - 1))) v >>= 1;
    return v;
}

// warp tasks of one phase on the vector engine (mirrors vec_phase)
uint64_t vec_tasks(const PhaseDesc& d, uint32_t P, int vbytes, int unroll = kVecUnroll) {
    const uint64_t vpc = d.copy_bytes / (uint64_t)vbytes;
    const uint64_t n_copies = (uint64_t)P * d.copies;
    if (n_copies >> 32) return ~0ull;  // the kernels index copies with 32 bits
    if (vpc >= 32) {
        const uint64_t span = 32ull * unroll;
        return n_copies * ((vpc + span - 1) / span);
    }
    if (vpc == 0) return 0;
    const uint64_t per_task = (32 / vpc) * unroll;
    return (n_copies + per_task - 1) / per_task;
}

uint64_t bulk_tasks(const PhaseDesc& d, uint32_t P, uint32_t stage_bytes) {
    return (uint64_t)P * d.copies * ((d.copy_bytes + stage_bytes - 1) / stage_bytes);
}

template <typename V>
const void* phase_vec_fn() { return (const void*)phase_vec_kernel<V>; }
template <typename V>
const void* persistent_vec_fn(bool list) {
    return list ? (const void*)persistent_vec_kernel<V, true> : (const void*)persistent_vec_kernel<V, false>;
}

const void* pick_phase_vec(int vbytes) {
    switch (vbytes) {
        case 16: return phase_vec_fn<uint4>();
        case 8: return phase_vec_fn<uint2>();
        case 4: return phase_vec_fn<unsigned>();
        case 2: return phase_vec_fn<unsigned short>();
        default: return phase_vec_fn<unsigned char>();
    }
}
template <typename V>
const void* phase_vec_var_fn() { return (const void*)phase_vec_list_kernel<V>; }
const void* pick_phase_vec_var(int vbytes) {
    switch (vbytes) {
        case 16: return phase_vec_var_fn<uint4>();
        case 8: return phase_vec_var_fn<uint2>();
        case 4: return phase_vec_var_fn<unsigned>();
        case 2: return phase_vec_var_fn<unsigned short>();
        default: return phase_vec_var_fn<unsigned char>();
    }
}
const void* pick_persistent_vec(int vbytes, bool list = false) {
    switch (vbytes) {
        case 16: return persistent_vec_fn<uint4>(list);
        case 8: return persistent_vec_fn<uint2>(list);
        case 4: return persistent_vec_fn<unsigned>(list);
        case 2: return persistent_vec_fn<unsigned short>(list);
        default: return persistent_vec_fn<unsigned char>(list);
    }
}
template <typename V>
const void* mirror_vec_fn(bool work) {
    return work ? (const void*)mirror_vec_kernel<V, true> : (const void*)mirror_vec_kernel<V, false>;
}
const void* pick_mirror_vec(int vbytes, bool work) {
    switch (vbytes) {
        case 16: return mirror_vec_fn<uint4>(work);
        case 8: return mirror_vec_fn<uint2>(work);
        case 4: return mirror_vec_fn<unsigned>(work);
        case 2: return mirror_vec_fn<unsigned short>(work);
        default: return mirror_vec_fn<unsigned char>(work);
    }
}
template <typename V>
const void* cluster_mirror_vec_fn() { return (const void*)cluster_mirror_vec_kernel<V>; }
template <typename V>
const void* cluster_mirror_async_fn() { return (const void*)cluster_mirror_async_kernel<V>; }
// st.async moves 4, 8 or 16 bytes: smaller vectors take the form with a cluster barrier per pass
const void* pick_cluster_mirror_vec(int vbytes) {
    switch (vbytes) {
        case 16: return cluster_mirror_async_fn<uint4>();
        case 8: return cluster_mirror_async_fn<uint2>();
        case 4: return cluster_mirror_async_fn<unsigned>();
        case 2: return cluster_mirror_vec_fn<unsigned short>();
        default: return cluster_mirror_vec_fn<unsigned char>();
    }
}
constexpr int kFlowWideUnroll = 4;  // vectors per lane of the flow kernel's wide form
template <typename V>
const void* flow_vec_fn(int unroll) {
    return unroll == kFlowWideUnroll ? (const void*)flow_vec_kernel<V, kFlowWideUnroll>
                                     : (const void*)flow_vec_kernel<V, kVecUnroll>;
}
const void* pick_flow_vec(int vbytes, int unroll) {
    switch (vbytes) {
        case 16: return flow_vec_fn<uint4>(unroll);
        case 8: return flow_vec_fn<uint2>(unroll);
        case 4: return flow_vec_fn<unsigned>(unroll);
        case 2: return flow_vec_fn<unsigned short>(unroll);
        default: return flow_vec_fn<unsigned char>(unroll);
    }
}

Geom make_geom(const sparbit_plan_s* p, const void* send, void* recv) {
    Geom g;
    memset(&g, 0, sizeof g);
    g.P = p->sched.P;
    g.m = p->sched.m;
    g.base[SPACE_SEND] = (char*)const_cast<void*>(send);
    g.base[SPACE_RECV] = (char*)recv;
    g.base[SPACE_WORK] = (char*)p->work;
    g.rank_pitch[SPACE_SEND] = g.m;
    g.rank_pitch[SPACE_RECV] = (uint64_t)g.P * g.m;
    g.rank_pitch[SPACE_WORK] = (uint64_t)g.P * g.m;
    if (p->variable) {
        g.m = 0;
        g.rank_pitch[SPACE_SEND] = 0;                 // send blocks sit at voff[rank]
        g.rank_pitch[SPACE_RECV] = p->voff.back();    // every receive buffer holds all blocks
        g.rank_pitch[SPACE_WORK] = 0;
    }
    return g;
}

// What a call that asks for phases first..last executes: the phases one by one, or, when it asks
// for both phase -1 and phase 0 and the schedule allows it, the fused first pass followed by
// phases 1..last.
struct ExecSeq {
    const Schedule* s;
    bool fused;
    int first, last;
    int count() const { return last - first + 1 - (fused ? 1 : 0); }
    const PhaseDesc& item(int i) const {
        if (!fused) return s->phase(first + i);
        return i == 0 ? s->fused_first : s->phase(i);
    }
    // position in the device table (see ensure_device)
    size_t table_index(int i) const {
        return fused ? s->phases.size() + (size_t)i : (size_t)(first + 1 + i);
    }
};

ExecSeq make_seq(const sparbit_plan_s* p, int first, int last) {
    ExecSeq q;
    q.s = &p->sched;
    q.first = first;
    q.last = last;
    q.fused = first == -1 && last >= 0 && p->sched.has_fused_first;
    return q;
}

struct Resolved {
    int exec;    // SPARBIT_EXEC_* (never AUTO)
    int copy;    // SPARBIT_COPY_VECTOR or _BULK
    int vbytes;  // vector width for the vector engine
};

// Shared memory one CTA of a cluster of C needs for the mirror executor: the receive buffers (and,
// for Bruck, working buffers) of its ceil(P / C) ranks.  C = 1: the single-CTA form.
unsigned __int128 mirror_smem_per_cta(const sparbit_plan_s* p, uint32_t C) {
    const uint32_t ranks = (p->sched.P + C - 1) / C;
    unsigned __int128 bytes = (unsigned __int128)ranks * p->sched.P * p->sched.m;
    if (p->sched.algo == ALGO_BRUCK) bytes *= 2;
    return bytes;
}

constexpr uint32_t kMirrorMaxCluster = 16;  // the largest cluster a B200 places (non-portable size)

// The mirror executor takes whole collectives of fixed-size blocks whose P receive buffers fit
// into the shared memory of one CTA, or of the CTAs of one cluster, together.
bool mirror_possible(const sparbit_plan_s* p, int first, int last, size_t smem_limit) {
    if (first != -1) return false;  // the on-chip copy starts empty: a call has to begin at the beginning
    if (smem_limit < 1024) return false;
    smem_limit -= 1024;  // the kernels' own static shared memory (mbarriers) comes out of the same limit
    const ExecSeq seq = make_seq(p, first, last);
    if (seq.count() < 1 || seq.count() > kMirrorMaxPasses) return false;
    if (p->variable)  // blocks of different sizes: one CTA only
        return (unsigned __int128)p->sched.P * p->voff.back() <= (unsigned __int128)smem_limit;
    return mirror_smem_per_cta(p, kMirrorMaxCluster) <= (unsigned __int128)smem_limit;
}

// Which passes of a call the flow kernel takes: the longest run of passes at the END of the
// executed sequence that it can take (fixed-size blocks of at least 32 vectors, at most
// kFlowMaxPasses of them) and that have at least FLOW_MIN_PASS_SPANS warp spans in all (0 stands
// for one per resident warp).  The passes before run as chained per-pass kernels.  A small pass
// alone is cheaper behind a kernel boundary than behind a counter hand-off, but in the collectives
// the flow executor is chosen for (1 GB moved and more) taking every pass measured equal or up to
// 2 % faster than any split (one launch instead of several, and the small passes overlap their
// neighbours), so the default is 1.  Returns the position of the first flow pass, or the sequence
// length if there is none.
// Vectors per lane and warp span in the flow kernel.  A collective that moves less than
// FLOW_WIDE_MAX_MOVED_BYTES in blocks of at least one wide span (2 KiB in 16-byte vectors) runs
// with four instead of two: half of such a collective lives in L2, which answers faster than the
// 32 KiB of loads in flight per SM that suit DRAM can keep busy (P = 256, m = 4 KiB: 85.0 us
// against 90.3; P = 362, m = 2 KiB: 85.5 against 91.4; P = 128, m = 16 KiB: 84.3 against 88.0;
// P = 256, m = 6 KiB: 125.6 against 129.7).  From about 1 GB moved the narrow form wins (P = 256,
// m = 8 KiB: 168.6 us against 174.4; P = 128, m = 64 KiB: 330.7 against 346.7), and blocks shorter
// than one wide span would leave it half empty.
int flow_unroll(const sparbit_plan_s* p, int vbytes) {
    if (p->variable) return kVecUnroll;
    const uint64_t m = p->sched.m;
    const unsigned __int128 moved = (unsigned __int128)2 * p->sched.P * (p->sched.P - 1) * m;
    if (moved < (unsigned __int128)p->tune[SPARBIT_TUNE_FLOW_WIDE_MAX_MOVED_BYTES] &&
        m / (uint64_t)vbytes >= 32ull * kFlowWideUnroll)
        return kFlowWideUnroll;
    return kVecUnroll;
}

int flow_first_pass(const sparbit_plan_s* p, const ExecSeq& seq, int vbytes, uint64_t max_warps) {
    const uint64_t span = 32ull * flow_unroll(p, vbytes);
    const int n = seq.count();
    int f = n;
    for (int i = n - 1; i >= 0 && n - i <= kFlowMaxPasses; i--) {
        const PhaseDesc& d = seq.item(i);
        const uint64_t vpc = d.copy_bytes / (uint64_t)vbytes;
        if (vpc < 32) break;
        const uint64_t spc = (vpc + span - 1) / span;
        const uint64_t spans = (uint64_t)p->sched.P * d.copies * spc;
        if (spans >> 31) break;
        const uint64_t least = p->tune[SPARBIT_TUNE_FLOW_MIN_PASS_SPANS] ? p->tune[SPARBIT_TUNE_FLOW_MIN_PASS_SPANS] : max_warps;
        if (spans < least) break;
        f = i;
    }
    return f;
}

constexpr uint64_t kFlowWarpsB200 = 148 * 2 * 16;  // resident warps of the flow kernel on a B200

bool flow_possible(const sparbit_plan_s* p, int vbytes, int first, int last, bool assume_b200 = false) {
    if (p->variable || !(p->coop || assume_b200)) return false;
    if (first != -1 || last != p->sched.last_phase()) return false;
    const ExecSeq seq = make_seq(p, first, last);
    if (seq.count() < 1) return false;
    const uint64_t warps = assume_b200 || !p->sm_count ? kFlowWarpsB200 : (uint64_t)p->sm_count * 2 * (kVecBlock / 32);
    return flow_first_pass(p, seq, vbytes, warps) < seq.count();
}

// Executor for SPARBIT_EXEC_AUTO, from measurements on B200.
//  - Up to 64 KiB of receive buffers in all, the mirror executor: one CTA, passes separated by its
//    own barrier and fed from shared memory (GPU time per collective, back to back: P = 8, m = 64 B
//    2.5 us against 4.7 for the chain; P = 32, m = 64 B: 5.5 against 9.1).  Above that one CTA's
//    bandwidth eats the gain, and a cluster of CTAs with the copies in distributed shared memory
//    takes over, up to 64 Ki vectors in the largest pass (2 MiB of receive buffers in 16-byte
//    vectors; blocks of a few bytes make as many vectors of a few bytes: P = 253, m = 1 B runs on a
//    cluster too, 13.6 against 18.5 for the chain and 36.8 in one CTA) with blocks of at most 4 KiB
//    (P = 64, m = 64 B: 6.1 against 11.5; P = 181, m = 64 B: 14.2 against 18.5; P = 16, m = 4 KiB: 7.2
//    either way): a pass is one push through the SM-to-SM network and an mbarrier, about 0.8 us.
//    Beyond that sixteen SMs' bandwidth eats the gain (P = 100, m = 200 B: 16.4 either way).
//  - A pass costs 1.6-2.3 us of GPU time in the latency regime whichever way it is separated from
//    the next one (kernel boundary with programmatic dependent launch, a CTA's own barrier, a grid
//    barrier, per-rank counters: two memory round trips - the loads, then the acknowledged stores
//    - are most of it), so there the launches decide.  One graph launch costs the host the same
//    whatever the graph holds, which a long chain needs; but back-to-back graph launches start a
//    microsecond or two apart where plain launches with programmatic stream serialisation overlap,
//    so a chain of at most STREAM_MAX_LAUNCHES kernels is launched kernel by kernel (chain_exec),
//    and so are the one-kernel executors.
//  - From about 0.4 GB moved (65 us and more) the flow executor is 1-7 % ahead of the chain: the
//    start-up and drain of every pass overlap with its neighbours (P = 256, m = 4 KiB: 85.0 us
//    against 92.1; P = 160, m = 8 KiB: 69.6 against 71.1; P = 1000, m = 1 KiB: 324.7 against 336.5;
//    P = 509, m = 4 KiB: 331.1 against 347.1; P = 128, m = 64 KiB: 332.4 against 338.7 on the bulk
//    engine).  At 0.33 GB it is behind (P = 200, m = 4 KiB: 58.5 against 56.8; P = 64, m = 40 KiB:
//    57.4 against 53.9).
//  - From about 6 GB moved the chain on the bulk engine wins again by 1-2 %: the pass boundaries
//    no longer matter and the bulk engine moves a byte a little cheaper than the vector engine,
//    which is the only one the flow executor has.
// Where the mirror executor is the fastest (measured): what decides is the number of vectors of
// the largest pass, which sixteen SMs have to push - at most MIRROR_MAX_VECTORS (1 MiB of receive
// buffers in 16-byte vectors; far less in blocks of a few bytes, which make vectors of a few
// bytes) - and, beyond the MIRROR_MAX_BYTES that one CTA takes, blocks of at most
// MIRROR_CLUSTER_MAX_BLOCK bytes (larger blocks mean few ranks and few passes: the chain is cheap).
bool mirror_wins(const sparbit_plan_s* p, int vbytes, int first, int last) {
    if (p->variable)  // one CTA: up to what one CTA takes of equal blocks
        return (unsigned __int128)p->sched.P * p->voff.back() <= (unsigned __int128)p->tune[SPARBIT_TUNE_MIRROR_MAX_BYTES];
    const ExecSeq seq = make_seq(p, first, last);
    uint64_t most = 0;
    for (int i = 0; i < seq.count(); i++) {
        const PhaseDesc& d = seq.item(i);
        const uint64_t v = (uint64_t)p->sched.P * d.copies * (d.copy_bytes / (uint64_t)vbytes);
        if (v > most) most = v;
    }
    if (most > p->tune[SPARBIT_TUNE_MIRROR_MAX_VECTORS]) return false;
    const unsigned __int128 all = (unsigned __int128)p->sched.P * p->sched.P * p->sched.m;
    return all <= (unsigned __int128)p->tune[SPARBIT_TUNE_MIRROR_MAX_BYTES] ||
           p->sched.m <= p->tune[SPARBIT_TUNE_MIRROR_CLUSTER_MAX_BLOCK];
}

int front_passes(const sparbit_plan_s* p, const ExecSeq& seq, int vbytes, uint32_t* groups);

// The executor for a small collective, or -1 if it is none.  One CTA where everything is small
// enough for it.  Beyond that the mirror executor on a cluster (about 3.5 us + 0.8 us per pass) or
// the chain with its leading passes in the grouped mirror kernel (4.2-6.2 us for those + 2.05 us
// per pass after them), whichever comes out shorter: the chain when at most three passes follow
// the grouped ones and the largest pass has more than 16 Ki vectors (measured, GPU time per
// collective: P = 256, m = 8 B 9.8 us against 11.7; P = 128, m = 128 B 10.0 against 13.3; P = 64,
// m = 512 B 8.6 against 12.6; but P = 64, m = 64 B 6.7 against 6.1 on the cluster, P = 32, m = 512 B
// 6.7 against 6.1, P = 16, m = 1 KiB 5.6 against 5.0).  P without a suitable power-of-two divisor
// has no groups: the cluster it is (P = 253, m = 1 B 13.6 against 18.5 for the plain chain;
// P = 181, m = 64 B 14.2 against 18.5).
int small_collective_exec(const sparbit_plan_s* p, int vbytes, int first, int last, size_t smem_limit) {
    if (!mirror_possible(p, first, last, smem_limit) || !mirror_wins(p, vbytes, first, last)) return -1;
    if (p->variable) return SPARBIT_EXEC_MIRROR;
    const ExecSeq seq = make_seq(p, first, last);
    uint64_t most = 0;
    for (int i = 0; i < seq.count(); i++) {
        const PhaseDesc& d = seq.item(i);
        const uint64_t v = (uint64_t)p->sched.P * d.copies * (d.copy_bytes / (uint64_t)vbytes);
        if (v > most) most = v;
    }
    if (mirror_smem_per_cta(p, 1) <= (unsigned __int128)p->tune[SPARBIT_TUNE_MIRROR_MAX_BYTES] &&
        most <= 8 * p->tune[SPARBIT_TUNE_MIRROR_CTA_VECTORS])
        return SPARBIT_EXEC_MIRROR;
    uint32_t groups = 1;
    const int s = front_passes(p, seq, vbytes, &groups);
    if (s >= 3 && seq.count() - s <= 3 && most > 16384) return SPARBIT_EXEC_GRAPH;
    return SPARBIT_EXEC_MIRROR;
}

// COPY_AUTO gives this plan the bulk engine and its blocks do not start on 128-byte lines.  The
// vector engine pays 10-30 % for such blocks (every warp row straddles lines; P = 128, m = 65520 B:
// 406 us in the chain, 363 in the flow kernel, against 331 at m = 65536 B), the bulk engine 2 %
// (345 us): the flow executor, which runs on the vector engine only, is then not worth leaving
// the bulk engine for.
bool bulk_off_line(const sparbit_plan_s* p, int vbytes) {
    if (p->variable || p->copy_req != SPARBIT_COPY_AUTO || vbytes != 16) return false;
    const uint64_t m = p->sched.m;
    const unsigned __int128 moved = (unsigned __int128)2 * p->sched.P * (p->sched.P - 1) * m;
    return (m & 127u) != 0 && m >= p->tune[SPARBIT_TUNE_BULK_MIN_BLOCK_BYTES] &&
           moved >= (unsigned __int128)p->tune[SPARBIT_TUNE_BULK_MIN_MOVED_BYTES];
}

int auto_exec(const sparbit_plan_s* p, int vbytes, int first, int last) {
    const int small = small_collective_exec(p, vbytes, first, last, (size_t)p->max_smem_optin);
    if (small >= 0) return small;
    const unsigned __int128 moved = (unsigned __int128)2 * p->sched.P * (p->sched.P - 1) * p->sched.m;
    if (moved >= (unsigned __int128)p->tune[SPARBIT_TUNE_FLOW_MIN_MOVED_BYTES] &&
        moved < (unsigned __int128)p->tune[SPARBIT_TUNE_FLOW_MAX_MOVED_BYTES] && !bulk_off_line(p, vbytes) &&
        flow_possible(p, vbytes, first, last))
        return SPARBIT_EXEC_FLOW;
    return SPARBIT_EXEC_GRAPH;
}

// Kernels a call launches on the chain (graph or stream executor, vector engine): one per pass,
// the grouped front counting as one.
int chain_launches(const sparbit_plan_s* p, int vbytes, int first, int last) {
    const ExecSeq seq = make_seq(p, first, last);
    uint32_t groups = 1;
    const int f = front_passes(p, seq, vbytes, &groups);
    return f ? 1 + seq.count() - f : seq.count();
}

// GRAPH or STREAM for a chain on the vector engine.  Back-to-back graph launches start on a grid
// of about 2 us; plain launches with programmatic stream serialisation overlap, which is worth 1-2 us
// of GPU time per collective (P = 256, m = 8 B, three launches: 9.8 us against 11.8; P = 64, m = 64 B,
// two: 6.7 against 8.2; P = 64, m = 4 KiB, six: 13.4 against 14.4).  But a graph launch costs the
// host 1.8 us whatever the graph holds and a plain launch of these kernels 2-3 us each (5 us into a
// queue that is already deep), so a caller that issues collectives back to back becomes bound by
// its own launches once they add up to more than the collective takes on the GPU.  Measured with
// the host feeding the loop, six launches still come out ahead of the graph (13.4 us against 14.4
// at P = 64, m = 4 KiB; five: 10.3 either way at P = 32, m = 4 KiB); eight would cost the host
// about 20 us where P = 256, m = 64 B without its grouped front takes the GPU 17.5.  Hence kernel by
// kernel up to STREAM_MAX_LAUNCHES (6), as a graph beyond.
int chain_exec(const sparbit_plan_s* p, int vbytes, int first, int last) {
    return (uint64_t)chain_launches(p, vbytes, first, last) <= p->tune[SPARBIT_TUNE_STREAM_MAX_LAUNCHES]
               ? SPARBIT_EXEC_STREAM
               : SPARBIT_EXEC_GRAPH;
}

bool auto_copy_is_bulk(const sparbit_plan_s* p, int vbytes) {
    if (p->copy_req != SPARBIT_COPY_AUTO) return p->copy_req == SPARBIT_COPY_BULK && vbytes == 16;
    if (vbytes != 16) return false;
    const uint64_t block = p->variable ? p->voff.back() / p->sched.P : p->sched.m;
    const unsigned __int128 moved = p->variable ? (unsigned __int128)2 * (p->sched.P - 1) * p->voff.back()
                                                : (unsigned __int128)2 * p->sched.P * (p->sched.P - 1) * p->sched.m;
    return block >= p->tune[SPARBIT_TUNE_BULK_MIN_BLOCK_BYTES] &&
           moved >= (unsigned __int128)p->tune[SPARBIT_TUNE_BULK_MIN_MOVED_BYTES];
}

int auto_exec_before_launch(const sparbit_plan_s* p, int vbytes) {
    const int small = small_collective_exec(p, vbytes, -1, p->sched.last_phase(), 227u << 10);
    if (small == SPARBIT_EXEC_GRAPH) return chain_exec(p, vbytes, -1, p->sched.last_phase());
    if (small >= 0) return small;
    const unsigned __int128 moved = (unsigned __int128)2 * p->sched.P * (p->sched.P - 1) * p->sched.m;
    if (moved >= (unsigned __int128)p->tune[SPARBIT_TUNE_FLOW_MIN_MOVED_BYTES] &&
        moved < (unsigned __int128)p->tune[SPARBIT_TUNE_FLOW_MAX_MOVED_BYTES] && !bulk_off_line(p, vbytes) &&
        flow_possible(p, vbytes, -1, p->sched.last_phase(), true))
        return SPARBIT_EXEC_FLOW;
    return auto_copy_is_bulk(p, vbytes) ? SPARBIT_EXEC_GRAPH : chain_exec(p, vbytes, -1, p->sched.last_phase());
}

Resolved resolve(const sparbit_plan_s* p, const void* send, const void* recv, int first, int last) {
    Resolved r;
    r.vbytes = pick_vector_bytes(p, send, recv);
    const uint64_t m = p->sched.m;
    const bool bulk_possible = r.vbytes == 16;
    int copy = p->copy_req;
    // measured on B200 (P = 61 .. 509, m = 4 KiB .. 256 KiB): with about 32 KiB of loads in flight per
    // SM both engines reach the copy peak; the bulk engine is 1-4 % ahead once blocks are >= 8 KiB
    // and the collective is in the bandwidth regime (about 1 GB moved or more); below that its
    // per-pass set-up (ring and mbarrier initialisation) and per-operation cost show and the
    // vector engine wins
    if (copy == SPARBIT_COPY_AUTO) {
        const unsigned __int128 moved = (unsigned __int128)2 * p->sched.P * (p->sched.P - 1) * m;
        copy = (bulk_possible && m >= p->tune[SPARBIT_TUNE_BULK_MIN_BLOCK_BYTES] &&
                moved >= (unsigned __int128)p->tune[SPARBIT_TUNE_BULK_MIN_MOVED_BYTES])
                   ? SPARBIT_COPY_BULK
                   : SPARBIT_COPY_VECTOR;
    }
    if (p->variable && p->copy_req == SPARBIT_COPY_AUTO) {
        // the same rule on the average block size, with 2*(P-1)*T bytes moved
        const uint64_t T = p->voff.back();
        const unsigned __int128 moved = (unsigned __int128)2 * (p->sched.P - 1) * T;
        copy = (bulk_possible && T / p->sched.P >= p->tune[SPARBIT_TUNE_BULK_MIN_BLOCK_BYTES] &&
                moved >= (unsigned __int128)p->tune[SPARBIT_TUNE_BULK_MIN_MOVED_BYTES])
                   ? SPARBIT_COPY_BULK
                   : SPARBIT_COPY_VECTOR;
    }
    if (copy == SPARBIT_COPY_BULK && !bulk_possible) copy = SPARBIT_COPY_VECTOR;
    r.copy = copy;
    int exec = p->exec_req;
    if (exec == SPARBIT_EXEC_AUTO) {
        exec = auto_exec(p, r.vbytes, first, last);
        if (exec == SPARBIT_EXEC_GRAPH && r.copy == SPARBIT_COPY_VECTOR) exec = chain_exec(p, r.vbytes, first, last);
    }
    if (exec == SPARBIT_EXEC_PERSISTENT && !p->coop) exec = SPARBIT_EXEC_GRAPH;
    if (exec == SPARBIT_EXEC_MIRROR && !mirror_possible(p, first, last, (size_t)p->max_smem_optin))
        exec = SPARBIT_EXEC_GRAPH;
    if (exec == SPARBIT_EXEC_MIRROR) r.copy = SPARBIT_COPY_VECTOR;
    if (exec == SPARBIT_EXEC_FLOW) {
        // the flow executor runs whole collectives of fixed-size blocks on the vector engine, every
        // copy at least one warp row long; anything else goes to the graph chain
        if (flow_possible(p, r.vbytes, first, last)) r.copy = SPARBIT_COPY_VECTOR;
        else exec = SPARBIT_EXEC_GRAPH;
    }
    r.exec = exec;
    return r;
}

// launch geometry of one phase as its own kernel
struct PhaseLaunch {
    const void* fn;
    dim3 grid, block;
    size_t smem;
};

int plan_phase_launch(sparbit_plan_s* p, const Resolved& rs, const PhaseDesc& d, PhaseLaunch& pl,
                      uint64_t var_tasks = 0) {
    const uint32_t P = p->sched.P;
    if (p->variable && rs.copy == SPARBIT_COPY_BULK) {
        uint64_t ctas = (var_tasks + p->bulk_warps - 1) / p->bulk_warps;
        if (ctas > (uint64_t)p->sm_count) ctas = p->sm_count;
        if (ctas < 1) ctas = 1;
        pl.fn = (const void*)phase_bulk_list_kernel;
        pl.grid = dim3((unsigned)ctas);
        pl.block = dim3(p->bulk_warps * 32);
        pl.smem = bulk_smem_bytes(p);
        return SPARBIT_OK;
    }
    if (p->variable) {
        const uint64_t wpb = kVecBlock / 32;
        uint64_t ctas = (var_tasks + wpb - 1) / wpb;
        const uint64_t cap = (uint64_t)p->sm_count * 2;
        if (ctas > cap) ctas = cap;
        if (ctas < 1) ctas = 1;
        pl.fn = pick_phase_vec_var(rs.vbytes);
        pl.grid = dim3((unsigned)ctas);
        pl.block = dim3(kVecBlock);
        pl.smem = 0;  // no occupancy cap here: this kernel reads its task list and the size table
                      // through L1, which a large shared-memory carve-out would shrink (measured)
        return SPARBIT_OK;
    }
    if (rs.copy == SPARBIT_COPY_BULK) {
        const uint64_t tasks = bulk_tasks(d, P, p->bulk_stage_bytes);
        uint64_t ctas = (tasks + p->bulk_warps - 1) / p->bulk_warps;
        if (ctas > (uint64_t)p->sm_count) ctas = p->sm_count;
        if (ctas < 1) ctas = 1;
        pl.fn = (const void*)phase_bulk_kernel;
        pl.grid = dim3((unsigned)ctas);
        pl.block = dim3(p->bulk_warps * 32);
        pl.smem = bulk_smem_bytes(p);
    } else {
        const uint64_t tasks = vec_tasks(d, P, rs.vbytes);
        if (tasks >> 32) return SPARBIT_ERR_OVERFLOW;
        const uint64_t wpb = kVecBlock / 32;
        uint64_t ctas = (tasks + wpb - 1) / wpb;
        // 1024 threads x 2 vectors in flight per SM suit DRAM.  Receive buffers of up to about twice the
        // L2 are served by L2 for a good part, which rewards a third CTA per SM (what the kernel's 40
        // registers allow): P = 256, m = 2 KiB 45.4 us against 46.7; P = 512, m = 512 B 61.4 against
        // 64.9; P = 512, m = 1 KiB 89.9 against 91.2; a fourth (fewer registers) gave nothing.
        const bool dense = (unsigned __int128)P * P * p->sched.m <=
                           (unsigned __int128)p->tune[SPARBIT_TUNE_VEC_DENSE_MAX_RECV_BYTES];
        const uint64_t cap = (uint64_t)p->sm_count * (dense ? 3 : 2);
        if (ctas > cap) ctas = cap;
        if (ctas < 1) ctas = 1;
        pl.fn = pick_phase_vec(rs.vbytes);
        pl.grid = dim3((unsigned)ctas);
        pl.block = dim3(kVecBlock);
        pl.smem = ctas == cap && !dense ? kVecOccupancySmem : 0;
    }
    return SPARBIT_OK;
}

struct PhaseArgs {
    Geom g;
    PhaseDesc d;
    uint32_t stage_bytes;
    unsigned* status;
    unsigned long long timeout_ns;
    uint32_t extra_tx;
    const VarTask* list;  // variable block sizes: this pass's task list
    unsigned long long count;
    void* ptrs[8];
    void fill(bool bulk, bool variable = false) {
        ptrs[0] = &g;
        ptrs[1] = &d;
        if (bulk) {
            ptrs[2] = &stage_bytes;
            ptrs[3] = &status;
            ptrs[4] = &timeout_ns;
            ptrs[5] = &extra_tx;
            ptrs[6] = &list;   // the list form of the bulk kernel only
            ptrs[7] = &count;
        } else if (variable) {
            ptrs[2] = &list;
            ptrs[3] = &count;
        }
    }
};

// How many leading passes of a call run in the grouped mirror kernel (0: none).  Sparbit's step
// distances are descending powers of two; while they are multiples of a G that divides P the
// ranks fall into G independent groups of R = P / G (see grouped_mirror_vec_kernel).  Recursive
// doubling's are ascending: after s steps a rank has only talked inside its aligned run of 2^s.  The largest
// such run of passes whose group state, R*R*m bytes, one CTA handles well (MIRROR_MAX_BYTES, and
// eight times MIRROR_CTA_VECTORS vectors in its largest pass); at least two passes.
int front_passes(const sparbit_plan_s* p, const ExecSeq& seq, int vbytes, uint32_t* groups) {
    const Schedule& sc = p->sched;
    if (!p->tune[SPARBIT_TUNE_GROUPED_FRONT] || p->variable || !seq.fused) return 0;
    if (sc.algo != ALGO_SPARBIT && sc.algo != ALGO_RD) return 0;
    const int n = seq.count();  // item i is step i (item 0 with the own-block copy fused in)
    int best = 0;
    for (int s = 2; s <= n && s <= kMirrorMaxPasses; s++) {
        // Sparbit: G = the distance of the last grouped step, a power of two that must divide P.
        // Recursive doubling (P a power of two): runs of R = twice that distance.
        const uint64_t dist = (uint64_t)sc.steps[(size_t)s - 1].distance;
        if (dist < 1 || (dist & (dist - 1))) continue;
        const uint64_t G = sc.algo == ALGO_SPARBIT ? dist : sc.P / (2 * dist);
        if (G < 1 || sc.P % G || G > 65535) continue;
        const uint64_t R = sc.P / G;
        if ((unsigned __int128)R * R * sc.m > (unsigned __int128)p->tune[SPARBIT_TUNE_MIRROR_MAX_BYTES]) break;  // groups only grow
        uint64_t most = 0;
        for (int i = 0; i < s; i++) {
            const PhaseDesc& d = seq.item(i);
            const uint64_t v = R * d.copies * (d.copy_bytes / (uint64_t)vbytes);
            if (v > most) most = v;
        }
        if (most > 8 * p->tune[SPARBIT_TUNE_MIRROR_CTA_VECTORS]) break;
        best = s;
        *groups = (uint32_t)G;
    }
    return best >= 2 ? best : 0;  // two grouped passes: 3.5 us where two chained passes cost 4 (P = 64, m = 2 KiB: 11.6 us against 12.5)
}

template <typename V>
const void* grouped_mirror_fn() { return (const void*)grouped_mirror_vec_kernel<V>; }
const void* pick_grouped_mirror(int vbytes) {
    switch (vbytes) {
        case 16: return grouped_mirror_fn<uint4>();
        case 8: return grouped_mirror_fn<uint2>();
        case 4: return grouped_mirror_fn<unsigned>();
        case 2: return grouped_mirror_fn<unsigned short>();
        default: return grouped_mirror_fn<unsigned char>();
    }
}

int grant_max_smem(const sparbit_plan_s* p, const void* fn, int slot, bool big_cluster);
int vec_slot(int vbytes);

int launch_grouped_front(sparbit_plan_s* p, const Resolved& rs, const Geom& g, const ExecSeq& seq, int front,
                         uint32_t groups, cudaStream_t st) {
    MirrorArgs ma;
    memset(&ma, 0, sizeof ma);
    ma.n = front;
    ma.aligned = p->sched.algo == ALGO_RD ? 1 : 0;
    const uint64_t R = p->sched.P / groups;
    uint64_t most = 1;
    for (int i = 0; i < front; i++) {
        ma.d[i] = seq.item(i);
        const uint64_t vpc = ma.d[i].copy_bytes / (uint64_t)rs.vbytes;
        const uint64_t v = R * ma.d[i].copies * vpc;
        if (v > most) most = v;
        ma.magic_vpc[i] = ((1ull << 40) + vpc - 1) / (vpc ? vpc : 1);
        ma.magic_copies[i] = ((1ull << 40) + ma.d[i].copies - 1) / (ma.d[i].copies ? ma.d[i].copies : 1);
    }
    const void* fn = pick_grouped_mirror(rs.vbytes);
    int rc = grant_max_smem(p, fn, 24 + vec_slot(rs.vbytes), false);
    if (rc) return rc;
    const uint64_t per_thread = p->tune[SPARBIT_TUNE_MIRROR_THREAD_VECTORS];
    uint64_t threads = (most + per_thread - 1) / per_thread;
    threads = (threads + 63) / 64 * 64;
    if (threads > 1024) threads = 1024;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(groups);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = (size_t)(R * R * p->sched.m);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    Geom gg = g;
    void* args[] = {&gg, &ma};
    CU(cudaLaunchKernelExC(&cfg, fn, args));
    p->kernel_launches++;
    return SPARBIT_OK;
}

// One kernel per phase on `st`.  Consecutive phases are launched with programmatic stream
// serialisation: a phase kernel lets its successor start launching at once
// (griddepcontrol.launch_dependents) and itself waits for its predecessor to complete and flush
// (griddepcontrol.wait) before it touches memory, so the launch latency of phase i+1 hides behind
// phase i while the Waitall between phases stays intact.
int launch_stream(sparbit_plan_s* p, const Resolved& rs, const Geom& g, int first, int last, cudaStream_t st,
                  int seq_end = -1) {
    const ExecSeq seq = make_seq(p, first, last);
    const int end = seq_end < 0 ? seq.count() : seq_end;  // only the first seq_end passes, if given
    int front = 0;
    if (seq_end < 0 && rs.copy == SPARBIT_COPY_VECTOR) {
        uint32_t groups = 1;
        auto& fc = p->front_cache;
        if (fc.valid && fc.vbytes == rs.vbytes && fc.first == first && fc.last == last &&
            fc.version == p->settings_version) {
            front = fc.front;
            groups = fc.groups;
        } else {
            front = front_passes(p, seq, rs.vbytes, &groups);
            fc.valid = true;
            fc.vbytes = rs.vbytes;
            fc.first = first;
            fc.last = last;
            fc.version = p->settings_version;
            fc.front = front;
            fc.groups = groups;
        }
        if (front) {
            int rc = launch_grouped_front(p, rs, g, seq, front, groups, st);
            if (rc) return rc;
        }
    }
    for (int i = front; i < end; i++) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        // The bulk kernel lets its dependents launch at once; across two calls that would bring the
        // next collective's kernels onto the SMs while this one's last, largest pass still needs
        // every slot (measured: 242 us against 175 at P = 256, m = 8 KiB back to back).  So the first
        // kernel of a call on that engine is an ordinary launch.
        cfg.numAttrs = (i == 0 && rs.copy == SPARBIT_COPY_BULK) ? 0 : 1;
        PhaseArgs a;
        a.g = g;
        a.d = seq.item(i);
        a.stage_bytes = p->bulk_stage_bytes;
        a.status = p->d_ctl + 1;
        a.timeout_ns = p->timeout_ns;
        a.extra_tx = p->mbar_extra_tx;
        a.list = nullptr;
        a.count = 0;
        if (p->variable) {
            const size_t ti = seq.table_index(i);
            a.list = p->d_vtasks + p->vtask_lo[ti];
            a.count = p->vtask_hi[ti] - p->vtask_lo[ti];
        }
        a.fill(rs.copy == SPARBIT_COPY_BULK, p->variable);
        PhaseLaunch pl;
        int rc = plan_phase_launch(p, rs, a.d, pl, a.count);
        if (rc) return rc;
        cfg.gridDim = pl.grid;
        cfg.blockDim = pl.block;
        cfg.dynamicSmemBytes = pl.smem;
        CU(cudaLaunchKernelExC(&cfg, pl.fn, a.ptrs));
        p->kernel_launches++;
    }
    return SPARBIT_OK;
}

void drop_graph(sparbit_plan_s* p) {
    for (auto& e : p->gcache)
        if (e.exec) cudaGraphExecDestroy(e.exec);
    p->gcache.clear();
}

constexpr size_t kGraphCacheEntries = 4;

int launch_mirror(sparbit_plan_s* p, const Resolved& rs, const Geom& g, int first, int last, cudaStream_t st);

int launch_graph(sparbit_plan_s* p, const Resolved& rs, const Geom& g, int first, int last, cudaStream_t st) {
    GraphKey key;
    key.send = g.base[SPACE_SEND];
    key.recv = g.base[SPACE_RECV];
    key.work = g.base[SPACE_WORK];
    key.first = first;
    key.last = last;
    key.path = rs.copy;
    key.vec = rs.vbytes;
    key.exec = rs.exec;
    key.timeout_ns = p->timeout_ns;
    key.extra_tx = p->mbar_extra_tx;
    sparbit_plan_s::GraphEntry* hit = nullptr;
    for (auto& e : p->gcache)
        if (e.key.same_shape(key) && e.key.same_buffers(key)) hit = &e;
    if (!hit) {
        // capture the chain of per-phase launches (programmatic edges included) into a graph
        if (!p->capture_stream) CU(cudaStreamCreateWithFlags(&p->capture_stream, cudaStreamNonBlocking));
        const uint64_t launches_before = p->kernel_launches;
        CU(cudaStreamBeginCapture(p->capture_stream, cudaStreamCaptureModeThreadLocal));
        int rc = rs.exec == SPARBIT_EXEC_MIRROR ? launch_mirror(p, rs, g, first, last, p->capture_stream)
                                                : launch_stream(p, rs, g, first, last, p->capture_stream);
        cudaGraph_t graph = nullptr;
        cudaError_t ce = cudaStreamEndCapture(p->capture_stream, &graph);
        const uint64_t captured = p->kernel_launches - launches_before;
        p->kernel_launches = launches_before;  // captured, not launched
        if (rc) {
            if (graph) cudaGraphDestroy(graph);
            return rc;
        }
        if (ce != cudaSuccess) return cuda_fail(ce, "cudaStreamEndCapture");
        if (p->gcache.size() < kGraphCacheEntries) {
            p->gcache.emplace_back();
            hit = &p->gcache.back();
        } else {
            // recycle the least recently used entry: same topology -> update it in place
            hit = &p->gcache[0];
            for (auto& e : p->gcache)
                if (e.stamp < hit->stamp) hit = &e;
            if (hit->exec && hit->key.same_shape(key)) {
                cudaGraphExecUpdateResultInfo info;
                if (cudaGraphExecUpdate(hit->exec, graph, &info) != cudaSuccess) {
                    (void)cudaGetLastError();
                    cudaGraphExecDestroy(hit->exec);
                    hit->exec = nullptr;
                }
            } else if (hit->exec) {
                cudaGraphExecDestroy(hit->exec);
                hit->exec = nullptr;
            }
        }
        if (!hit->exec) {
            cudaError_t ie = cudaGraphInstantiate(&hit->exec, graph, 0);
            if (ie != cudaSuccess) {
                cudaGraphDestroy(graph);
                hit->exec = nullptr;
                hit->key = GraphKey();
                return cuda_fail(ie, "cudaGraphInstantiate");
            }
        }
        cudaGraphDestroy(graph);
        hit->key = key;
        hit->kernels = captured;
    }
    hit->stamp = ++p->gstamp;
    CU(cudaGraphLaunch(hit->exec, st));
    p->graph_launches++;
    p->kernel_launches += hit->kernels;
    return SPARBIT_OK;
}

int launch_persistent(sparbit_plan_s* p, const Resolved& rs, const Geom& g, int first, int last, cudaStream_t st) {
    const uint32_t P = p->sched.P;
    const ExecSeq seq = make_seq(p, first, last);
    // grid: enough CTAs for the largest phase, at most what is co-resident
    uint64_t need = 1;
    const void* fn;
    dim3 block;
    size_t smem = 0;
    int per_sm = 0;
    // tasks of pass i: listed (variable block sizes) or counted from the descriptor
    auto list_tasks = [&](int i) {
        const size_t ti = seq.table_index(i);
        return (uint64_t)(p->vtask_hi[ti] - p->vtask_lo[ti]);
    };
    if (rs.copy == SPARBIT_COPY_BULK) {
        fn = p->variable ? (const void*)persistent_bulk_kernel<true> : (const void*)persistent_bulk_kernel<false>;
        block = dim3(p->bulk_warps * 32);
        smem = bulk_smem_bytes(p);
        for (int i = 0; i < seq.count(); i++) {
            const uint64_t tasks = p->variable ? list_tasks(i) : bulk_tasks(seq.item(i), P, p->bulk_stage_bytes);
            uint64_t t = (tasks + p->bulk_warps - 1) / p->bulk_warps;
            if (t > need) need = t;
        }
    } else {
        fn = pick_persistent_vec(rs.vbytes, p->variable);
        block = dim3(kVecBlock);
        for (int i = 0; i < seq.count(); i++) {
            const uint64_t tasks = p->variable ? list_tasks(i) : vec_tasks(seq.item(i), P, rs.vbytes);
            if (tasks >> 32) return SPARBIT_ERR_OVERFLOW;
            uint64_t t = (tasks + kVecBlock / 32 - 1) / (kVecBlock / 32);
            if (t > need) need = t;
        }
    }
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, (int)block.x, smem));
    if (per_sm < 1) return cuda_fail(cudaErrorLaunchOutOfResources, "persistent kernel does not fit on an SM");
    // one CTA of rings per SM keeps the loads in flight at the measured sweet spot; more would fit
    if (rs.copy == SPARBIT_COPY_BULK) per_sm = 1;
    uint64_t grid = (uint64_t)per_sm * p->sm_count;
    if (grid > need) grid = need;
    BarrierCtl ctl;
    ctl.counter = p->d_ctl;
    ctl.status = p->d_ctl + 1;
    ctl.base = p->bar_base;
    ctl.expected = (unsigned)grid + (unsigned)p->extra_arrivals;
    ctl.timeout_ns = p->timeout_ns;
    ctl.mbar_extra_tx = p->mbar_extra_tx;
    ctl.trace = nullptr;
    if (p->trace_on) {
        const size_t need_entries = (size_t)seq.count() + 1;
        if (need_entries > p->trace_cap) {  // (re)allocate; the first traced call is not capturable
            cudaFree(p->d_trace);
            p->d_trace = nullptr;
            p->trace_cap = 0;
            CU(cudaMalloc((void**)&p->d_trace, need_entries * sizeof(unsigned long long)));
            p->trace_cap = need_entries;
        }
        ctl.trace = p->d_trace;
        p->trace_len = need_entries;
    }
    int first_idx = (int)seq.table_index(0), last_idx = (int)seq.table_index(seq.count() - 1);
    Geom gg = g;
    const PhaseDesc* descs = p->d_descs;
    uint32_t stage = p->bulk_stage_bytes;
    const VarTask* vtasks = p->d_vtasks;   // null unless the plan has variable block sizes
    const VarRange* vranges = p->d_vranges;
    void* args_vec[] = {&gg, &descs, &first_idx, &last_idx, &ctl, &vtasks, &vranges};
    void* args_bulk[] = {&gg, &descs, &first_idx, &last_idx, &stage, &ctl, &vtasks, &vranges};
    CU(cudaLaunchCooperativeKernel(fn, dim3((unsigned)grid), block,
                                   rs.copy == SPARBIT_COPY_BULK ? args_bulk : args_vec, smem, st));
    p->bar_base += (unsigned)(last_idx - first_idx) * ctl.expected;  // one barrier between consecutive passes
    p->kernel_launches++;
    return SPARBIT_OK;
}

// The whole collective in one CTA, or in one cluster of CTAs, with the receive buffers mirrored in
// (distributed) shared memory.
// The mirror kernels take their dynamic shared memory up to the device's opt-in maximum.  The limit
// is a property of the function, not of a plan: it is raised once per device and kernel, to the
// maximum (asking for less per launch costs nothing), so that no plan can lower it under another.
constexpr int kSmemDevices = 64;
std::mutex g_smem_mutex;
bool g_smem_granted[kSmemDevices][40];
int vec_slot(int vbytes) { return vbytes == 16 ? 4 : vbytes == 8 ? 3 : vbytes == 4 ? 2 : vbytes == 2 ? 1 : 0; }
int grant_max_smem(const sparbit_plan_s* p, const void* fn, int slot, bool big_cluster) {
    std::lock_guard<std::mutex> lock(g_smem_mutex);
    const int dev = p->device >= 0 && p->device < kSmemDevices ? p->device : 0;
    if (g_smem_granted[dev][slot]) return SPARBIT_OK;
    cudaFuncAttributes fa;
    CU(cudaFuncGetAttributes(&fa, fn));  // the limit covers static and dynamic shared memory together
    CU(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, p->max_smem_optin - (int)fa.sharedSizeBytes));
    if (big_cluster) CU(cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    g_smem_granted[dev][slot] = true;
    return SPARBIT_OK;
}

template <typename V>
const void* mirror_list_fn() { return (const void*)mirror_list_kernel<V>; }
const void* pick_mirror_list(int vbytes) {
    switch (vbytes) {
        case 16: return mirror_list_fn<uint4>();
        case 8: return mirror_list_fn<uint2>();
        case 4: return mirror_list_fn<unsigned>();
        case 2: return mirror_list_fn<unsigned short>();
        default: return mirror_list_fn<unsigned char>();
    }
}

// blocks of different sizes: one CTA, a warp per listed task
int launch_mirror_list(sparbit_plan_s* p, const Resolved& rs, const Geom& g, const ExecSeq& seq, cudaStream_t st) {
    MirrorListArgs ma;
    memset(&ma, 0, sizeof ma);
    ma.n = seq.count();
    uint64_t most = 1;  // tasks of the largest pass
    for (int i = 0; i < ma.n; i++) {
        const PhaseDesc& d = seq.item(i);
        const size_t ti = seq.table_index(i);
        ma.pass[i].list = p->d_vtasks + p->vtask_lo[ti];
        ma.pass[i].count = p->vtask_hi[ti] - p->vtask_lo[ti];
        ma.pass[i].src_space = d.src_space;
        ma.pass[i].dst_space = d.dst_space;
        ma.pass[i].dup_self = d.dup_self;
        if (ma.pass[i].count > most) most = ma.pass[i].count;
        // lanes per task: about the vectors of an average task of this pass
        uint64_t bytes = 0;
        for (size_t t = p->vtask_lo[ti]; t < p->vtask_hi[ti]; t++) bytes += (p->vtasks[t].a >> 48) + 1;
        const uint64_t avg = ma.pass[i].count ? bytes / ma.pass[i].count / (uint64_t)rs.vbytes : 1;
        uint32_t group = 4;
        while (group < 32 && group < avg) group *= 2;
        ma.pass[i].group = group;
    }
    const void* fn = pick_mirror_list(rs.vbytes);
    const size_t smem = (size_t)p->sched.P * p->voff.back();
    int rc = grant_max_smem(p, fn, 16 + vec_slot(rs.vbytes), false);
    if (rc) return rc;
    uint64_t threads = most * 32;  // a warp per task of the largest pass, as far as a CTA goes
    if (threads > 1024) threads = 1024;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    Geom gg = g;
    void* args[] = {&gg, &ma};
    CU(cudaLaunchKernelExC(&cfg, fn, args));
    p->kernel_launches++;
    return SPARBIT_OK;
}

int launch_mirror(sparbit_plan_s* p, const Resolved& rs, const Geom& g, int first, int last, cudaStream_t st) {
    const uint32_t P = p->sched.P;
    const ExecSeq seq = make_seq(p, first, last);
    if (p->variable) return launch_mirror_list(p, rs, g, seq, st);
    MirrorArgs ma;
    memset(&ma, 0, sizeof ma);
    ma.n = seq.count();
    ma.status = p->d_ctl + 1;
    ma.timeout_ns = p->timeout_ns;
    ma.extra_tx = p->mbar_extra_tx;
    uint64_t most = 1;  // vectors of the largest pass
    for (int i = 0; i < ma.n; i++) {
        ma.d[i] = seq.item(i);
        const uint64_t vpc = ma.d[i].copy_bytes / (uint64_t)rs.vbytes;
        const uint64_t v = (uint64_t)P * ma.d[i].copies * vpc;
        if (v > most) most = v;
        ma.magic_vpc[i] = ((1ull << 40) + vpc - 1) / (vpc ? vpc : 1);
        ma.magic_copies[i] = ((1ull << 40) + ma.d[i].copies - 1) / (ma.d[i].copies ? ma.d[i].copies : 1);
    }
    // One CTA while everything fits and is small enough for it (MIRROR_MAX_BYTES, and at most
    // eight times MIRROR_CTA_VECTORS vectors in the largest pass: blocks of a few bytes make many
    // vectors of few bytes); else the smallest cluster that holds it and leaves a CTA at most
    // MIRROR_CTA_VECTORS vectors in the largest pass.
    uint32_t C = 1;
    const unsigned __int128 limit = (unsigned __int128)p->max_smem_optin - 1024;  // as in mirror_possible
    const bool spread = mirror_smem_per_cta(p, 1) > (unsigned __int128)p->tune[SPARBIT_TUNE_MIRROR_MAX_BYTES] ||
                        most > 8 * p->tune[SPARBIT_TUNE_MIRROR_CTA_VECTORS];
    while (C < kMirrorMaxCluster &&
           (mirror_smem_per_cta(p, C) > limit || (C < P && spread && most / C > p->tune[SPARBIT_TUNE_MIRROR_CTA_VECTORS])))
        C *= 2;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    Geom gg = g;
    void* args[] = {&gg, &ma};
    for (;;) {
        const bool work = p->sched.algo == ALGO_BRUCK;  // the only schedule with working buffers
        const void* fn = C == 1 ? pick_mirror_vec(rs.vbytes, work) : pick_cluster_mirror_vec(rs.vbytes);
        const size_t ranks = (P + C - 1) / C;
        size_t smem = ranks * P * p->sched.m;
        ma.work_at = 0;
        if (p->sched.algo == ALGO_BRUCK) {
            ma.work_at = (uint32_t)(smem / (size_t)rs.vbytes);
            smem *= 2;
        }
        // four vectors per thread and pass when there are that many, CTA sizes in steps of two warps
        const uint64_t per_thread = p->tune[SPARBIT_TUNE_MIRROR_THREAD_VECTORS];
        uint64_t threads = (most / C + per_thread - 1) / per_thread;
        threads = (threads + 63) / 64 * 64;
        if (threads > 1024) threads = 1024;
        {
            const int grc = grant_max_smem(p, fn, (C == 1 ? (work ? 32 : 0) : 8) + vec_slot(rs.vbytes), C > 1);
            if (grc) return grc;
        }
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(C);
        cfg.blockDim = dim3((unsigned)threads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (C > 1) {
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = C;
            attr[1].val.clusterDim.y = 1;
            attr[1].val.clusterDim.z = 1;
            cfg.numAttrs = 2;
            // can the device place this cluster at all?  If not, a smaller one that still holds the
            // buffers, else the per-pass kernels
            int fit = 0;
            if (cudaOccupancyMaxActiveClusters(&fit, fn, &cfg) != cudaSuccess || fit < 1) {
                (void)cudaGetLastError();
                if (C > 2 && mirror_smem_per_cta(p, C / 2) <= limit) {
                    C /= 2;
                    continue;
                }
                return launch_stream(p, rs, g, first, last, st);
            }
        }
        CU(cudaLaunchKernelExC(&cfg, fn, args));
        p->kernel_launches++;
        return SPARBIT_OK;
    }
}

// The flow executor's pass table (host only): how each pass is cut into units, where its rank
// enumeration starts, which earlier passes a unit has to wait for, and the counter value that
// says "all units of this launch that write into this rank in this pass are done".  Returns the
// unit count of the largest pass.
uint64_t flow_pass_table(const sparbit_plan_s* p, const ExecSeq& seq, int f, int vbytes, uint64_t max_warps,
                         unsigned epoch, bool never_reached, FlowArgs& fa) {
    const uint32_t P = p->sched.P;
    const int n = seq.count() - f;  // the kernel's passes: positions f.. of the sequence
    fa.n = (uint32_t)n;
    uint64_t most_units = 1;
    uint32_t rot = 0;
    for (int i = 0; i < n; i++) {
        const PhaseDesc& d = seq.item(f + i);
        FlowPass& fp = fa.pass[i];
        const uint64_t vpc = d.copy_bytes / (uint64_t)vbytes;
        const uint64_t span = 32ull * flow_unroll(p, vbytes);
        fp.spc = (uint32_t)((vpc + span - 1) / span);
        const uint64_t spans = (uint64_t)d.copies * fp.spc;  // per source rank
        // Unit size: a small pass is cut into single spans, so that as many warps as possible share
        // it and a hop (copy, release, the next pass's poll) stays short; a pass that keeps every
        // warp busy takes units of up to FLOW_MAX_UNIT_SPANS spans, which spreads
        // the poll and the release over more bytes.
        uint64_t us = (uint64_t)P * spans / (max_warps * p->tune[SPARBIT_TUNE_FLOW_UNITS_PER_WARP]);
        if (us < 1) us = 1;
        if (us > p->tune[SPARBIT_TUNE_FLOW_MAX_UNIT_SPANS]) us = p->tune[SPARBIT_TUNE_FLOW_MAX_UNIT_SPANS];
        if (us > spans) us = spans;
        fp.us = (uint32_t)us;
        fp.upr = (uint32_t)((spans + fp.us - 1) / fp.us);
        fp.rot = rot;
        // units that write into one rank's buffer in this pass: those of its one sender, and in the
        // fused first pass its own as well
        const uint32_t per_rank = fp.upr * (d.dup_self ? 2u : 1u);
        fp.target = epoch * per_rank + (never_reached ? 1u : 0u);  // test hook: a target that is never reached
        fp.dep_mask = 0;  // passes before f are complete when the kernel starts (stream order)
        for (int k = 0; k < i; k++)
            if (seq.item(f + k).dst_space == d.src_space) fp.dep_mask |= 1u << k;
        if (p->tune[SPARBIT_TUNE_FLOW_SKIP_WAITS]) fp.dep_mask = 0;  // measurement hook: wrong results, timing only
        if ((uint64_t)P * fp.upr > most_units) most_units = (uint64_t)P * fp.upr;
        fp.eager = (uint64_t)P * fp.upr <= max_warps ? 1u : 0u;
        // the next pass starts its enumeration where this pass's first receivers are
        if (d.peer_xor == 0 && d.peer_pre == 0) rot = (rot + d.peer_add) % P;
    }
    return most_units;
}

// The collective's small leading passes as chained per-pass kernels, all the others in one
// cooperative kernel without grid barriers (flow_vec_kernel).
// the stream the last flow kernel of this process went to, per device
constexpr int kFlowDevices = 64;
struct FlowStream {
    bool seen = false;
    cudaStream_t stream = nullptr;
};
std::mutex g_flow_mutex;
FlowStream g_flow_last[kFlowDevices];

int launch_flow(sparbit_plan_s* p, const Resolved& rs, const Geom& g, int first, int last, cudaStream_t st) {
    const uint32_t P = p->sched.P;
    const ExecSeq seq = make_seq(p, first, last);
    const int unroll = flow_unroll(p, rs.vbytes);
    const void* fn = pick_flow_vec(rs.vbytes, unroll);
    int per_sm = 0;
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kVecBlock, 0));
    if (per_sm < 1) return cuda_fail(cudaErrorLaunchOutOfResources, "flow kernel does not fit on an SM");
    if (per_sm > 2) per_sm = 2;
    const uint64_t max_warps = (uint64_t)per_sm * p->sm_count * (kVecBlock / 32);
    const int f = flow_first_pass(p, seq, rs.vbytes, max_warps);
    if (f >= seq.count()) return launch_stream(p, rs, g, first, last, st);  // (resolve() rules this out)
    if (f > 0) {
        int rc = launch_stream(p, rs, g, first, last, st, f);
        if (rc) return rc;
    }
    if (!p->d_flow_cnt) {
        CU(cudaMalloc((void**)&p->d_flow_cnt, (size_t)P * kFlowMaxPasses * sizeof(unsigned)));
        p->flow_epoch = 0;
        p->flow_vbytes = 0;
    }
    if (p->flow_vbytes != rs.vbytes * 16 + unroll || p->flow_epoch == 0) {
        // counters count units, and a unit's size follows the vector width and the span: start over
        // (with leading per-pass kernels in front this memset sits between kernels: rare, and correct)
        CU(cudaMemsetAsync(p->d_flow_cnt, 0, (size_t)P * kFlowMaxPasses * sizeof(unsigned), st));
        p->flow_epoch = 0;
        p->flow_vbytes = rs.vbytes * 16 + unroll;
    }
    p->flow_epoch++;
    FlowArgs fa;
    memset(&fa, 0, sizeof fa);
    fa.cnt = p->d_flow_cnt;
    fa.status = p->d_ctl + 1;
    fa.timeout_ns = p->timeout_ns;
    const uint64_t most_units =
        flow_pass_table(p, seq, f, rs.vbytes, max_warps, p->flow_epoch, p->extra_arrivals != 0, fa);
    uint64_t grid = (uint64_t)per_sm * p->sm_count;
    const uint64_t need = (most_units + kVecBlock / 32 - 1) / (kVecBlock / 32);
    if (grid > need) grid = need;
    Geom gg = g;
    const PhaseDesc* descs = p->d_descs;
    int first_idx = (int)seq.table_index(f);
    void* args[] = {&gg, &descs, &first_idx, &fa};
    // The waits inside need all CTAs of the grid resident.  A cooperative launch guarantees that,
    // but cannot start ahead of its predecessor's end as the per-pass kernels do (2-2.5 us per
    // collective).  An ordinary launch of a grid that fits the device is just as safe as long as
    // no other kernel of this kind can hold part of the SMs at the same time: kernels in ONE
    // stream are ordered (the successor's CTAs only wait for the predecessor's end), and every
    // other kernel of this library finishes without waiting for anybody.  So: an ordinary launch
    // when the flow launch before this one (any plan, this device) went to the same stream, a
    // cooperative one otherwise - that one starts only when it fits as a whole, behind or in
    // front of the other stream's kernel, never interleaved with it.
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kVecBlock);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    std::lock_guard<std::mutex> lock(g_flow_mutex);
    FlowStream& prev = g_flow_last[p->device >= 0 && p->device < kFlowDevices ? p->device : 0];
    cfg.numAttrs = (prev.seen && prev.stream == st && !p->tune[SPARBIT_TUNE_FLOW_COOPERATIVE]) ? 1 : 2;
    CU(cudaLaunchKernelExC(&cfg, fn, args));
    prev.seen = true;
    prev.stream = st;
    p->kernel_launches++;
    return SPARBIT_OK;
}

int run_phases(sparbit_plan_s* p, const void* send, void* recv, void* stream, int first, int last) {
    if (!p) return SPARBIT_ERR_ARG;
    const Schedule& s = p->sched;
    if (first < -1 || last > s.last_phase() || first > last) return SPARBIT_ERR_ARG;
    const size_t send_bytes = p->send_bytes();
    const size_t recv_bytes = p->recv_bytes();
    if (send_bytes == 0) return SPARBIT_OK;  // count 0: nothing to do
    if (!send || !recv) return SPARBIT_ERR_ARG;
    if (s.algo == ALGO_BRUCK && (!p->work || p->work_bytes < recv_bytes)) return SPARBIT_ERR_WORKSPACE;
    if (ranges_overlap(send, send_bytes, recv, recv_bytes)) return SPARBIT_ERR_ALIAS;
    if (s.algo == ALGO_BRUCK &&
        (ranges_overlap(send, send_bytes, p->work, recv_bytes) || ranges_overlap(recv, recv_bytes, p->work, recv_bytes)))
        return SPARBIT_ERR_ALIAS;
    int rc = ensure_device(p);
    if (rc) return rc;
    Resolved rs;
    {
        const int vb = pick_vector_bytes(p, send, recv);
        auto& c = p->resolved;
        if (c.valid && c.vbytes == vb && c.first == first && c.last == last && c.version == p->settings_version) {
            rs.vbytes = vb;
            rs.exec = c.exec;
            rs.copy = c.copy;
        } else {
            rs = resolve(p, send, recv, first, last);
            c.valid = true;
            c.vbytes = rs.vbytes;
            c.first = first;
            c.last = last;
            c.version = p->settings_version;
            c.exec = rs.exec;
            c.copy = rs.copy;
        }
    }
    const Geom g = make_geom(p, send, recv);
    cudaStream_t st = (cudaStream_t)stream;
    // On a stream that is being captured the work must be replayable as it stands.  The persistent
    // and the flow kernel take counter values of THIS launch as arguments, and a cached graph
    // would have to be instantiated in the middle of the caller's capture; so there the passes go
    // in as plain chained kernels (the mirror kernel as itself), which replay any number of times.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    CU(cudaStreamIsCapturing(st, &capturing));
    if (capturing != cudaStreamCaptureStatusNone) {
        Resolved rc_rs = rs;
        if (rs.exec != SPARBIT_EXEC_MIRROR) rc_rs.exec = SPARBIT_EXEC_STREAM;
        rc = rc_rs.exec == SPARBIT_EXEC_MIRROR ? launch_mirror(p, rc_rs, g, first, last, st)
                                               : launch_stream(p, rc_rs, g, first, last, st);
        if (rc == SPARBIT_OK) {
            p->copy_last = rc_rs.copy;
            p->exec_last = rc_rs.exec;
            p->last_stream = st;
            p->launched = true;
        }
        return rc;
    }
    switch (rs.exec) {
        case SPARBIT_EXEC_PERSISTENT: rc = launch_persistent(p, rs, g, first, last, st); break;
        case SPARBIT_EXEC_GRAPH: rc = launch_graph(p, rs, g, first, last, st); break;
        case SPARBIT_EXEC_FLOW: rc = launch_flow(p, rs, g, first, last, st); break;
        case SPARBIT_EXEC_MIRROR: rc = launch_mirror(p, rs, g, first, last, st); break;
        default: rc = launch_stream(p, rs, g, first, last, st); break;
    }
    if (rc == SPARBIT_OK) {
        p->copy_last = rs.copy;
        p->exec_last = rs.exec;
        p->last_stream = st;
        p->launched = true;
    }
    return rc;
}

}  // namespace

// What the multi-device entry points (multi.cu) need of a plan and of this file's error record.
namespace spb {
const Schedule* plan_schedule(const sparbit_plan_s* p) { return p ? &p->sched : nullptr; }
bool plan_is_variable(const sparbit_plan_s* p) { return p && p->variable; }
int record_cuda_error(int cuda_error, const char* what) { return cuda_fail((cudaError_t)cuda_error, what); }
}  // namespace spb

extern "C" {

int sparbit_plan_create(int P, size_t block_bytes, int algo, int exec, sparbit_plan_t** out) {
    if (!out) return SPARBIT_ERR_ARG;
    *out = nullptr;
    if (algo < SPARBIT_ALGO_SPARBIT || algo > SPARBIT_ALGO_NEIGHBOR_EXCHANGE) return SPARBIT_ERR_ARG;
    if (exec < SPARBIT_EXEC_AUTO || exec > SPARBIT_EXEC_MIRROR) return SPARBIT_ERR_ARG;
    sparbit_plan_s* p = new (std::nothrow) sparbit_plan_s();
    if (!p) return SPARBIT_ERR_NOMEM;
    int rc;
    try {
        rc = map_sched_err(build_schedule(algo, P, (uint64_t)block_bytes, p->sched));
    } catch (const std::bad_alloc&) {
        rc = SPARBIT_ERR_NOMEM;
    }
    if (rc) {
        delete p;
        return rc;
    }
    p->exec_req = exec == SPARBIT_EXEC_AUTO ? env_exec(SPARBIT_EXEC_AUTO) : exec;
    p->copy_req = env_copy(SPARBIT_COPY_AUTO);
    *out = p;
    return SPARBIT_OK;
}

int sparbit_plan_create_v(int P, const size_t* block_bytes, int algo, int exec, sparbit_plan_t** out) {
    if (!out) return SPARBIT_ERR_ARG;
    *out = nullptr;
    if (!block_bytes || P < 1) return SPARBIT_ERR_ARG;
    if (P > 8192) return SPARBIT_ERR_LIMIT;  // the task lists are built copy by copy: P*(P-1) entries at least
    if (algo < SPARBIT_ALGO_SPARBIT || algo > SPARBIT_ALGO_NEIGHBOR_EXCHANGE) return SPARBIT_ERR_ARG;
    if (algo == SPARBIT_ALGO_BRUCK) return SPARBIT_ERR_UNSUPPORTED;  // rotated workspace: fixed sizes only
    if (exec < SPARBIT_EXEC_AUTO || exec > SPARBIT_EXEC_MIRROR) return SPARBIT_ERR_ARG;
    if (exec == SPARBIT_EXEC_FLOW) return SPARBIT_ERR_UNSUPPORTED;  // lays its work out for equal blocks
    sparbit_plan_s* p = new (std::nothrow) sparbit_plan_s();
    if (!p) return SPARBIT_ERR_NOMEM;
    int rc;
    try {
        rc = map_sched_err(build_schedule(algo, P, 1, p->sched));
        if (rc == SPARBIT_OK) {
            p->variable = true;
            p->voff.assign((size_t)P + 1, 0);
            unsigned __int128 total = 0;
            for (int b = 0; b < P; b++) {
                total += block_bytes[b];
                if (total >> 62) rc = SPARBIT_ERR_OVERFLOW;
                p->voff[(size_t)b + 1] = (uint64_t)total;
                p->voff_bits |= (uintptr_t)p->voff[(size_t)b + 1];
            }
            if ((total * (unsigned)P) >> 62) rc = SPARBIT_ERR_OVERFLOW;
        }
        if (rc == SPARBIT_OK) {
            // the task grid of a phase is laid out for its largest copy
            auto set_max = [&](PhaseDesc& d) {
                uint64_t mx = 0;
                for (uint32_t r = 0; r < p->sched.P; r++)
                    for (uint32_t j = 0; j < d.copies; j++) {
                        const CopyLoc c = locate_copy(d, p->sched.P, r, j);
                        const uint64_t b = p->voff[c.dst_slot + d.run] - p->voff[c.dst_slot];
                        if (b > mx) mx = b;
                    }
                d.copy_bytes = mx;
            };
            for (PhaseDesc& d : p->sched.phases) set_max(d);
            if (p->sched.has_fused_first) set_max(p->sched.fused_first);
            p->sched.m = 0;
            // task lists, indexed like the device descriptor table: every phase, the fused first
            // pass, and (as in that table) phases 1.. once more after it.  A task is a segment of at
            // most kVarSegmentBytes of one copy, with its source and destination byte offsets.
            const uint64_t T = p->voff.back();
            if (((unsigned __int128)T * (unsigned)P) >> 48) rc = SPARBIT_ERR_OVERFLOW;  // offsets are 48-bit fields
            auto add_list = [&](const PhaseDesc& d) {
                p->vtask_lo.push_back(p->vtasks.size());
                for (uint32_t r = 0; r < p->sched.P; r++)
                    for (uint32_t j = 0; j < d.copies; j++) {
                        const CopyLoc c = locate_copy(d, p->sched.P, r, j);
                        const uint64_t b = p->voff[c.dst_slot + d.run] - p->voff[c.dst_slot];
                        // send blocks sit at voff[rank]; every receive buffer holds all blocks
                        const uint64_t soff = d.src_space == SPACE_SEND
                                                  ? p->voff[c.src_rank]
                                                  : (uint64_t)c.src_rank * T + p->voff[c.src_slot];
                        const uint64_t doff = (uint64_t)c.dst_rank * T + p->voff[c.dst_slot];
                        const int delta = (int)r - (int)c.dst_rank;  // |delta| < P <= 8192
                        for (uint64_t at = 0; at < b; at += kVarSegmentBytes) {
                            const uint64_t n = b - at < kVarSegmentBytes ? b - at : kVarSegmentBytes;
                            VarTask t;
                            t.a = (soff + at) | ((n - 1) << 48);
                            t.b = (doff + at) | ((unsigned long long)(unsigned short)(short)delta << 48);
                            p->vtasks.push_back(t);
                        }
                    }
                p->vtask_hi.push_back(p->vtasks.size());
            };
            for (const PhaseDesc& d : p->sched.phases) add_list(d);
            if (p->sched.has_fused_first) {
                add_list(p->sched.fused_first);
                for (size_t i = 2; i < p->sched.phases.size(); i++) {  // same lists as phases 1..
                    p->vtask_lo.push_back(p->vtask_lo[i]);
                    p->vtask_hi.push_back(p->vtask_hi[i]);
                }
            }
            if (p->vtasks.size() >> 27) rc = SPARBIT_ERR_OVERFLOW;  // 2 GiB of task entries: refuse
        }
    } catch (const std::bad_alloc&) {
        rc = SPARBIT_ERR_NOMEM;
    }
    if (rc) {
        delete p;
        return rc;
    }
    p->exec_req = exec;
    if (exec == SPARBIT_EXEC_AUTO) {  // variable-size plans have no flow executor
        const int e = env_exec(SPARBIT_EXEC_AUTO);
        if (e != SPARBIT_EXEC_FLOW) p->exec_req = e;
    }
    p->copy_req = env_copy(SPARBIT_COPY_AUTO);
    *out = p;
    return SPARBIT_OK;
}

sparbit_plan_t* sparbit_plan(int P, size_t block_bytes) {
    sparbit_plan_t* p = nullptr;
    if (sparbit_plan_create(P, block_bytes, SPARBIT_ALGO_SPARBIT, SPARBIT_EXEC_AUTO, &p) != SPARBIT_OK) return nullptr;
    return p;
}

int sparbit_plan_destroy(sparbit_plan_t* p) {
    if (!p) return SPARBIT_OK;
    int rc = SPARBIT_OK;
    if (p->dev_touched || p->stage_send || p->stage_recv || p->stage_work) {
        if (p->launched && cudaDeviceSynchronize() != cudaSuccess) rc = SPARBIT_ERR_CUDA;
        drop_graph(p);
        if (p->capture_stream) cudaStreamDestroy(p->capture_stream);
        cudaFree(p->d_descs);
        cudaFree(p->d_vtasks);
        cudaFree(p->d_vranges);
        cudaFree(p->d_trace);
        cudaFree(p->d_ctl);
        cudaFree(p->d_flow_cnt);
        cudaFree(p->stage_send);
        cudaFree(p->stage_recv);
        cudaFree(p->stage_work);
    }
    delete p;
    return rc;
}

int sparbit_allgather(sparbit_plan_t* p, const void* sendbuf, void* recvbuf, void* stream) {
    if (!p) return SPARBIT_ERR_ARG;
    return run_phases(p, sendbuf, recvbuf, stream, -1, p->sched.last_phase());
}

int sparbit_allgather_steps(sparbit_plan_t* p, const void* sendbuf, void* recvbuf, void* stream, int first,
                            int last) {
    if (!p) return SPARBIT_ERR_ARG;
    if (first > last) return SPARBIT_ERR_ARG;
    return run_phases(p, sendbuf, recvbuf, stream, first, last);
}

int sparbit_allgather_host(sparbit_plan_t* p, const void* host_send, void* host_recv) {
    if (!p) return SPARBIT_ERR_ARG;
    const Schedule& s = p->sched;
    const size_t send_bytes = p->send_bytes();
    const size_t recv_bytes = p->recv_bytes();
    if (send_bytes == 0) return SPARBIT_OK;
    if (!host_send || !host_recv) return SPARBIT_ERR_ARG;
    if (ranges_overlap(host_send, send_bytes, host_recv, recv_bytes)) return SPARBIT_ERR_ALIAS;
    // bind the plan to the current device (or refuse another one) before anything is allocated
    int rc0 = ensure_device(p);
    if (rc0) return rc0;
    if (!p->stage_send) CU(cudaMalloc(&p->stage_send, send_bytes));
    if (!p->stage_recv) CU(cudaMalloc(&p->stage_recv, recv_bytes));
    if (s.algo == ALGO_BRUCK && !p->work) {
        if (!p->stage_work) CU(cudaMalloc(&p->stage_work, recv_bytes));
        p->work = p->stage_work;
        p->work_bytes = recv_bytes;
    }
    cudaStream_t st = nullptr;
    CU(cudaMemcpyAsync(p->stage_send, host_send, send_bytes, cudaMemcpyHostToDevice, st));
    int rc = run_phases(p, p->stage_send, p->stage_recv, st, -1, s.last_phase());
    if (rc) return rc;
    CU(cudaMemcpyAsync(host_recv, p->stage_recv, recv_bytes, cudaMemcpyDeviceToHost, st));
    return sparbit_plan_status(p, nullptr);
}

int sparbit_plan_num_steps(const sparbit_plan_t* p) { return p ? p->sched.K : -1; }
int sparbit_plan_last_phase(const sparbit_plan_t* p) { return p ? p->sched.last_phase() : -2; }

int sparbit_plan_step_info(const sparbit_plan_t* p, int step, int* distance, int* blocks_per_rank, int* ignore) {
    if (!p || step < 0 || step >= p->sched.K) return SPARBIT_ERR_ARG;
    const StepInfo& si = p->sched.steps[(size_t)step];
    if (distance) *distance = si.distance;
    if (blocks_per_rank) *blocks_per_rank = si.blocks;
    if (ignore) *ignore = si.ignore;
    return SPARBIT_OK;
}

int sparbit_plan_messages(const sparbit_plan_t* p, int phase, sparbit_msg* out, size_t cap, size_t* n) {
    if (!p || !n || phase < -1 || phase > p->sched.last_phase()) return SPARBIT_ERR_ARG;
    if (cap > 0 && !out) return SPARBIT_ERR_ARG;
    *n = (size_t)phase_message_count(p->sched, phase);
    if (cap == 0) return SPARBIT_OK;
    static_assert(sizeof(Msg) == sizeof(sparbit_msg), "message layouts must agree");
    try {
        std::vector<Msg> v;
        expand_phase(p->sched, phase, v);
        const size_t k = v.size() < cap ? v.size() : cap;
        memcpy(out, v.data(), k * sizeof(Msg));
    } catch (const std::bad_alloc&) {
        return SPARBIT_ERR_NOMEM;
    }
    return SPARBIT_OK;
}

int sparbit_rank_device(int P, int G, int mapping, int rank) {
    if (P < 1 || G < 1 || rank < 0 || rank >= P) return -1;
    if (mapping != SPARBIT_MAP_SEQUENTIAL && mapping != SPARBIT_MAP_CYCLIC) return -1;
    return (int)rank_device((uint32_t)P, (uint32_t)G, mapping, (uint32_t)rank);
}

int sparbit_plan_partition(const sparbit_plan_t* p, int G, int mapping, int phase, uint64_t* blocks) {
    if (!p || !blocks || G < 1 || G > 4096 || phase < -1 || phase > p->sched.last_phase()) return SPARBIT_ERR_ARG;
    if (mapping != SPARBIT_MAP_SEQUENTIAL && mapping != SPARBIT_MAP_CYCLIC) return SPARBIT_ERR_ARG;
    try {
        std::vector<uint64_t> v;
        partition_counts(p->sched, phase, (uint32_t)G, mapping, v);
        memcpy(blocks, v.data(), v.size() * sizeof(uint64_t));
    } catch (const std::bad_alloc&) {
        return SPARBIT_ERR_NOMEM;
    }
    return SPARBIT_OK;
}

int sparbit_plan_partition_messages(const sparbit_plan_t* p, int G, int mapping, int phase, int src_device,
                                    int dst_device, sparbit_msg* out, size_t cap, size_t* n) {
    if (!p || !n || G < 1 || G > 4096 || phase < -1 || phase > p->sched.last_phase()) return SPARBIT_ERR_ARG;
    if (mapping != SPARBIT_MAP_SEQUENTIAL && mapping != SPARBIT_MAP_CYCLIC) return SPARBIT_ERR_ARG;
    if (src_device < 0 || src_device >= G || dst_device < 0 || dst_device >= G) return SPARBIT_ERR_ARG;
    if (cap > 0 && !out) return SPARBIT_ERR_ARG;
    try {
        std::vector<Msg> v;
        partition_messages(p->sched, phase, (uint32_t)G, mapping, (uint32_t)src_device, (uint32_t)dst_device, v);
        *n = v.size();
        const size_t k = v.size() < cap ? v.size() : cap;
        if (k) memcpy(out, v.data(), k * sizeof(Msg));
    } catch (const std::bad_alloc&) {
        return SPARBIT_ERR_NOMEM;
    }
    return SPARBIT_OK;
}

size_t sparbit_plan_workspace_bytes(const sparbit_plan_t* p) {
    if (!p || p->sched.algo != ALGO_BRUCK) return 0;
    return (size_t)p->sched.P * p->sched.P * p->sched.m;
}

int sparbit_plan_set_workspace(sparbit_plan_t* p, void* dev, size_t bytes) {
    if (!p) return SPARBIT_ERR_ARG;
    if (bytes < sparbit_plan_workspace_bytes(p)) return SPARBIT_ERR_WORKSPACE;
    if (!dev && sparbit_plan_workspace_bytes(p) > 0) return SPARBIT_ERR_WORKSPACE;
    p->work = dev;
    p->settings_version++;
    p->work_bytes = bytes;
    return SPARBIT_OK;
}

int sparbit_plan_set_copy_path(sparbit_plan_t* p, int copy_path) {
    if (!p || copy_path < SPARBIT_COPY_AUTO || copy_path > SPARBIT_COPY_BULK) return SPARBIT_ERR_ARG;
    p->copy_req = copy_path;
    p->settings_version++;
    return SPARBIT_OK;
}

int sparbit_plan_set_tunable(sparbit_plan_t* p, int key, uint64_t value) {
    if (!p || key < 0 || key >= SPARBIT_TUNE_COUNT_) return SPARBIT_ERR_ARG;
    if ((key == SPARBIT_TUNE_MIRROR_CTA_VECTORS || key == SPARBIT_TUNE_MIRROR_THREAD_VECTORS) && value == 0)
        return SPARBIT_ERR_ARG;  // divisors
    if (p->tune[key] == value) return SPARBIT_OK;
    if (p->launched) {
        // cached graphs were cut into launches with the old value
        if (cudaStreamSynchronize(p->last_stream) != cudaSuccess) return SPARBIT_ERR_CUDA;
        drop_graph(p);
    }
    p->tune[key] = value;
    p->settings_version++;
    return SPARBIT_OK;
}

int sparbit_plan_get_tunable(const sparbit_plan_t* p, int key, uint64_t* value) {
    if (!p || !value || key < 0 || key >= SPARBIT_TUNE_COUNT_) return SPARBIT_ERR_ARG;
    *value = p->tune[key];
    return SPARBIT_OK;
}

int sparbit_plan_exec_mode(const sparbit_plan_t* p) {
    if (!p) return -1;
    if (p->exec_last != SPARBIT_EXEC_AUTO) return p->exec_last;  // what the last launch ran on
    if (p->exec_req != SPARBIT_EXEC_AUTO) return p->exec_req;
    // before the first launch neither the buffers nor the device are known: assume 16-byte aligned
    // buffers on a B200
    uintptr_t bits = p->variable ? p->voff_bits : (uintptr_t)p->sched.m;
    int v = 16;
    while (v > 1 && (bits & (uintptr_t)(v - 1))) v >>= 1;
    return auto_exec_before_launch(p, v);
}

int sparbit_plan_copy_path(const sparbit_plan_t* p) { return p ? p->copy_last : -1; }

int sparbit_plan_launch_counts(const sparbit_plan_t* p, uint64_t* kernel_launches, uint64_t* graph_launches) {
    if (!p) return SPARBIT_ERR_ARG;
    if (kernel_launches) *kernel_launches = p->kernel_launches;
    if (graph_launches) *graph_launches = p->graph_launches;
    return SPARBIT_OK;
}

int sparbit_plan_status(sparbit_plan_t* p, int* device_status) {
    if (!p) return SPARBIT_ERR_ARG;
    if (device_status) *device_status = 0;
    if (!p->dev_ready || !p->launched) return SPARBIT_OK;
    CU(cudaStreamSynchronize(p->last_stream));
    unsigned ctl[2] = {0, 0};
    CU(cudaMemcpy(ctl, p->d_ctl, sizeof ctl, cudaMemcpyDeviceToHost));
    if (device_status) *device_status = (int)ctl[1];
    if (ctl[1] != DEV_OK) {
        // a failed launch leaves the arrival counter in an unknown state: start over
        CU(cudaMemset(p->d_ctl, 0, sizeof ctl));
        p->bar_base = 0;
        p->flow_epoch = 0;  // the next flow launch clears its counters
        return SPARBIT_ERR_TIMEOUT;
    }
    return SPARBIT_OK;
}

int sparbit_plan_set_mbarrier_test(sparbit_plan_t* p, uint32_t extra_tx_bytes, uint64_t timeout_ns) {
    if (!p || (extra_tx_bytes & 15u) || extra_tx_bytes > 65536u) return SPARBIT_ERR_ARG;
    p->mbar_extra_tx = extra_tx_bytes;
    p->timeout_ns = timeout_ns ? timeout_ns : kDefaultTimeoutNs;
    return SPARBIT_OK;
}

int sparbit_plan_set_trace(sparbit_plan_t* p, int on) {
    if (!p) return SPARBIT_ERR_ARG;
    p->trace_on = on != 0;
    if (!p->trace_on) p->trace_len = 0;
    return SPARBIT_OK;
}

int sparbit_plan_get_trace(sparbit_plan_t* p, uint64_t* ns, size_t cap, size_t* n) {
    if (!p || !n || (cap > 0 && !ns)) return SPARBIT_ERR_ARG;
    *n = p->trace_len;
    if (p->trace_len == 0 || cap == 0) return SPARBIT_OK;
    CU(cudaStreamSynchronize(p->last_stream));
    static_assert(sizeof(uint64_t) == sizeof(unsigned long long), "time stamps are 64-bit");
    const size_t k = p->trace_len < cap ? p->trace_len : cap;
    CU(cudaMemcpy(ns, p->d_trace, k * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    return SPARBIT_OK;
}

int sparbit_plan_set_barrier_test(sparbit_plan_t* p, int extra_arrivals, uint64_t timeout_ns) {
    if (!p || extra_arrivals < 0) return SPARBIT_ERR_ARG;
    p->extra_arrivals = extra_arrivals;
    p->timeout_ns = timeout_ns ? timeout_ns : kDefaultTimeoutNs;
    return SPARBIT_OK;
}

// Host-side race and bounds check of the descriptors as the kernels will execute them: every
// pass of the full collective (fused first pass included) is expanded through locate_copy; a
// location is (space, rank, slot) and `valid` says whether it already holds its block.
int sparbit_plan_validate(const sparbit_plan_t* p, int* bad_phase) {
    if (!p) return SPARBIT_ERR_ARG;
    if (bad_phase) *bad_phase = -2;
    const Schedule& s = p->sched;
    const uint32_t P = s.P;
    if (P > 8192) return SPARBIT_ERR_LIMIT;
    try {
        const size_t PP = (size_t)P * P;
        // per space (RECV, WORK): 0 = empty, 1 = valid, 2 = written in this pass, 3 = read in this pass
        std::vector<uint8_t> state[2] = {std::vector<uint8_t>(PP, 0), std::vector<uint8_t>(PP, 0)};
        std::vector<uint32_t> writes(PP, 0);
        ExecSeq seq;
        seq.s = &s;
        seq.first = -1;
        seq.last = s.last_phase();
        seq.fused = s.last_phase() >= 0 && s.has_fused_first;
        auto fail = [&](int pass) {
            if (bad_phase) *bad_phase = pass;
            return SPARBIT_ERR_ARG;
        };
        for (int i = 0; i < seq.count(); i++) {
            const PhaseDesc& d = seq.item(i);
            const int pass = seq.fused ? i : i - 1;  // phase number (the fused pass reports 0)
            std::vector<size_t> touched_w, touched_r;
            for (uint32_t r = 0; r < P; r++)
                for (uint32_t j = 0; j < d.copies; j++) {
                    const CopyLoc c = locate_copy(d, P, r, j);
                    if (c.dst_rank >= P || c.src_rank >= P) return fail(pass);
                    for (uint32_t k = 0; k < d.run; k++) {
                        const uint32_t ss = c.src_slot + k, ds = c.dst_slot + k;
                        if (ds >= P || d.dst_space == SPACE_SEND) return fail(pass);
                        if (d.src_space == SPACE_SEND) {
                            if (c.src_slot != 0 || d.run != 1) return fail(pass);  // one block per rank
                        } else {
                            if (ss >= P) return fail(pass);
                            uint8_t& st = state[d.src_space - 1][(size_t)c.src_rank * P + ss];
                            if (st != 1 && st != 3) return fail(pass);  // read before it is valid, or while written
                            if (st == 1) touched_r.push_back((size_t)c.src_rank * P + ss);
                            st = 3;
                        }
                        const int ndst = d.dup_self ? 2 : 1;
                        for (int t = 0; t < ndst; t++) {
                            const uint32_t dr = t == 0 ? c.dst_rank : r;
                            if (t == 1 && dr == c.dst_rank) continue;  // one rank: both destinations coincide
                            const size_t at = (size_t)dr * P + ds;
                            uint8_t& st = state[d.dst_space - 1][at];
                            if (st != 0) return fail(pass);  // written twice, or written while read / valid
                            st = 2;
                            touched_w.push_back(at);
                            if (d.dst_space == SPACE_RECV) writes[at]++;
                        }
                    }
                }
            // the pass boundary: what was written becomes valid, what was read stays valid
            if (d.src_space != SPACE_SEND)
                for (size_t at : touched_r) state[d.src_space - 1][at] = 1;
            for (size_t at : touched_w) state[d.dst_space - 1][at] = 1;
        }
        for (size_t at = 0; at < PP; at++)
            if (state[0][at] != 1 || writes[at] != 1) return fail(s.last_phase() + 1);
    } catch (const std::bad_alloc&) {
        return SPARBIT_ERR_NOMEM;
    }
    return SPARBIT_OK;
}

// Host-side check of the flow executor's bookkeeping for a given vector width and number of
// resident warps: the units of every pass, decoded exactly as the kernel decodes them, must cover
// every span of every rank's copies once; the number of units that write into a rank's buffer
// (through either destination of the fused pass) must be the counter target of that pass; and a
// pass must wait for every earlier pass that writes the space it reads.
int sparbit_plan_validate_flow(const sparbit_plan_t* p, int vector_bytes, int resident_warps, int* first_flow_pass,
                               int* bad_pass) {
    if (!p || resident_warps < 1) return SPARBIT_ERR_ARG;
    if (first_flow_pass) *first_flow_pass = -1;
    if (vector_bytes != 1 && vector_bytes != 2 && vector_bytes != 4 && vector_bytes != 8 && vector_bytes != 16)
        return SPARBIT_ERR_ARG;
    if (bad_pass) *bad_pass = -1;
    if (p->variable) return SPARBIT_ERR_UNSUPPORTED;
    const uint32_t P = p->sched.P;
    const ExecSeq seq = make_seq(p, -1, p->sched.last_phase());
    if (seq.count() < 1) return SPARBIT_ERR_UNSUPPORTED;
    try {
        FlowArgs fa;
        memset(&fa, 0, sizeof fa);
        const unsigned epoch = 3;
        const int f = flow_first_pass(p, seq, vector_bytes, (uint64_t)resident_warps);
        if (f >= seq.count()) return SPARBIT_ERR_UNSUPPORTED;
        flow_pass_table(p, seq, f, vector_bytes, (uint64_t)resident_warps, epoch, false, fa);
        if (first_flow_pass) *first_flow_pass = f;
        for (int i = 0; i < seq.count() - f; i++) {
            const PhaseDesc& d = seq.item(f + i);
            const FlowPass& fp = fa.pass[i];
            auto fail = [&]() {
                if (bad_pass) *bad_pass = i;
                return SPARBIT_ERR_ARG;
            };
            const uint64_t spans_per_rank = (uint64_t)d.copies * fp.spc;
            if (spans_per_rank * P > (1ull << 26)) return SPARBIT_ERR_LIMIT;
            std::vector<uint8_t> covered((size_t)(spans_per_rank * P), 0);
            std::vector<uint32_t> arrivals(P, 0);
            for (uint64_t w = 0; w < (uint64_t)P * fp.upr; w++) {
                const uint32_t x = (uint32_t)(w / fp.upr), k = (uint32_t)(w - (uint64_t)x * fp.upr);
                uint32_t r = x + fp.rot;
                if (r >= P) r -= P;
                const uint64_t s0 = (uint64_t)k * fp.us;
                uint64_t s1 = s0 + fp.us;
                if (s1 > spans_per_rank) s1 = spans_per_rank;
                if (s0 >= s1) return fail();  // an empty unit would still be counted
                uint32_t dst = P;
                for (uint64_t sidx = s0; sidx < s1; sidx++) {
                    uint8_t& c = covered[(size_t)(r * spans_per_rank + sidx)];
                    if (c) return fail();
                    c = 1;
                    const CopyLoc loc = locate_copy(d, P, r, (uint32_t)(sidx / fp.spc));
                    if (dst != P && dst != loc.dst_rank) return fail();  // one destination rank per unit
                    dst = loc.dst_rank;
                }
                arrivals[dst]++;
                if (d.dup_self && dst != r) arrivals[r]++;
            }
            for (uint8_t c : covered)
                if (!c) return fail();
            for (uint32_t q = 0; q < P; q++)
                if (arrivals[q] * epoch != fp.target) return fail();
            uint32_t want_mask = 0;
            for (int k = 0; k < i; k++)
                if (seq.item(f + k).dst_space == d.src_space) want_mask |= 1u << k;
            if (fp.dep_mask != want_mask || (d.src_space == SPACE_SEND && fp.dep_mask)) return fail();
        }
    } catch (const std::bad_alloc&) {
        return SPARBIT_ERR_NOMEM;
    }
    return SPARBIT_OK;
}

const char* sparbit_strerror(int code) {
    switch (code) {
        case SPARBIT_OK: return "success";
        case SPARBIT_ERR_ARG: return "invalid argument";
        case SPARBIT_ERR_OVERFLOW: return "size not representable";
        case SPARBIT_ERR_ALIAS: return "buffers overlap";
        case SPARBIT_ERR_UNSUPPORTED:
            return "unsupported (recursive doubling needs a power-of-two P, neighbor exchange an even P)";
        case SPARBIT_ERR_WORKSPACE: return "workspace missing or too small";
        case SPARBIT_ERR_CUDA: return "CUDA runtime error";
        case SPARBIT_ERR_TIMEOUT: return "device barrier timed out";
        case SPARBIT_ERR_NOMEM: return "out of host memory";
        case SPARBIT_ERR_LIMIT: return "beyond a fixed limit of this entry point (scratch size or rank count)";
        case SPARBIT_ERR_BARRIER: return "the caller's cross-device barrier failed";
        default: return "unknown error";
    }
}

const char* sparbit_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"

// ================================================================================================
// Entry point that allocates no device memory.
//
// Some users of this library run where cudaMalloc is not an option: inside an application whose
// device memory belongs to its own pool, as a plug-in that only receives buffers and a stream,
// or in a loop that must stay clear of the driver's allocation lock.  For them the scratch the
// persistent executor needs (descriptor table, barrier counter, status word) lives in the fixed
// array below, which is part of the library image on every GPU that loads it.
// ================================================================================================
namespace {

constexpr int kNoallocMaxPhases = 28;
constexpr size_t kNoallocCtlBytes = 256;  // [0] barrier counter, [1] status word, rest unused
constexpr size_t kNoallocBytes = kNoallocCtlBytes + kNoallocMaxPhases * sizeof(PhaseDesc);
static_assert(sizeof(PhaseDesc) == 64, "descriptor size is part of the scratch budget");
static_assert(kNoallocBytes == 2048, "the documented size of the fixed scratch");

// Host code must never hand this name to a kernel: on the host it is only a stand-in for the
// symbol.  The device address comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocBytes];

constexpr int kMaxDevices = 64;
struct NoallocDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;  // device address of g_noalloc_scratch on this device
    int sm_count = 0;
    int coop = 0;
};
NoallocDevice g_noalloc_dev[kMaxDevices];
std::mutex g_noalloc_mutex;  // guards the once-per-device set-up only

// once per device, with that device current
int noalloc_setup(int device, NoallocDevice*& out) {
    if (device < 0 || device >= kMaxDevices) return SPARBIT_ERR_ARG;
    NoallocDevice& nd = g_noalloc_dev[device];
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!nd.ready) {
        void* ptr = nullptr;
        CU(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        CU(cudaDeviceGetAttribute(&nd.sm_count, cudaDevAttrMultiProcessorCount, device));
        CU(cudaDeviceGetAttribute(&nd.coop, cudaDevAttrCooperativeLaunch, device));
        nd.scratch = (unsigned char*)ptr;
        // the array is zero when the module is loaded; clear it anyway so that the first call
        // does not depend on that
        CU(cudaMemset(nd.scratch, 0, kNoallocBytes));
        nd.ready = true;
    }
    out = &nd;
    return SPARBIT_OK;
}

}  // namespace

extern "C" {

int sparbit_allgather_noalloc(int P, size_t block_bytes, int algo, const void* sendbuf, void* recvbuf,
                              void* stream) {
    if (algo < SPARBIT_ALGO_SPARBIT || algo > SPARBIT_ALGO_NEIGHBOR_EXCHANGE) return SPARBIT_ERR_ARG;
    if (algo == SPARBIT_ALGO_BRUCK) return SPARBIT_ERR_UNSUPPORTED;  // needs a P*P*m workspace
    Schedule sched;
    int rc;
    try {
        rc = map_sched_err(build_schedule(algo, P, (uint64_t)block_bytes, sched));
    } catch (const std::bad_alloc&) {
        rc = SPARBIT_ERR_NOMEM;
    }
    if (rc) return rc;
    // what is executed, as in sparbit_allgather: the own-block copy and the first step as one fused
    // pass where the schedule has one, then the remaining steps
    std::vector<PhaseDesc> passes;
    try {
        if (sched.has_fused_first) {
            passes.push_back(sched.fused_first);
            passes.insert(passes.end(), sched.phases.begin() + 2, sched.phases.end());
        } else {
            passes = sched.phases;
        }
    } catch (const std::bad_alloc&) {
        return SPARBIT_ERR_NOMEM;
    }
    if (passes.size() > (size_t)kNoallocMaxPhases) return SPARBIT_ERR_LIMIT;
    const size_t send_bytes = (size_t)sched.P * sched.m;
    const size_t recv_bytes = (size_t)sched.P * sched.P * sched.m;
    if (send_bytes == 0) return SPARBIT_OK;
    if (!sendbuf || !recvbuf) return SPARBIT_ERR_ARG;
    if (ranges_overlap(sendbuf, send_bytes, recvbuf, recv_bytes)) return SPARBIT_ERR_ALIAS;

    // this entry point waits for its stream; a capturing stream cannot be waited for
    cudaStream_t st = (cudaStream_t)stream;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    CU(cudaStreamIsCapturing(st, &capturing));
    if (capturing != cudaStreamCaptureStatusNone) return SPARBIT_ERR_UNSUPPORTED;

    int device = -1;
    CU(cudaGetDevice(&device));
    NoallocDevice* nd = nullptr;
    rc = noalloc_setup(device, nd);
    if (rc) return rc;
    if (!nd->coop) return SPARBIT_ERR_UNSUPPORTED;

    // vector width from the alignment of the buffers and m (no workspace here)
    uintptr_t bits = (uintptr_t)sendbuf | (uintptr_t)recvbuf | (uintptr_t)sched.m;
    int vbytes = 16;
    while (vbytes > 1 && (bits & (uintptr_t)(vbytes - 1))) vbytes >>= 1;

    // grid: enough CTAs for the largest phase, at most what is co-resident
    uint64_t need = 1;
    for (const PhaseDesc& d : passes) {
        const uint64_t tasks = vec_tasks(d, sched.P, vbytes);
        if (tasks >> 32) return SPARBIT_ERR_OVERFLOW;
        const uint64_t t = (tasks + kVecBlock / 32 - 1) / (kVecBlock / 32);
        if (t > need) need = t;
    }
    const void* fn = pick_persistent_vec(vbytes);
    int per_sm = 0;
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kVecBlock, 0));
    if (per_sm < 1) return cuda_fail(cudaErrorLaunchOutOfResources, "persistent kernel does not fit on an SM");
    uint64_t grid = (uint64_t)per_sm * nd->sm_count;
    if (grid > need) grid = need;

    unsigned* ctl_words = (unsigned*)nd->scratch;
    PhaseDesc* d_descs = (PhaseDesc*)(nd->scratch + kNoallocCtlBytes);

    // every call starts from a clean scratch: barrier counter and status word at zero, this
    // collective's descriptors in the table (the call waits below, so the host copy outlives it)
    CU(cudaMemsetAsync(ctl_words, 0, kNoallocCtlBytes, st));
    const size_t n = passes.size();
    CU(cudaMemcpyAsync(d_descs, passes.data(), n * sizeof(PhaseDesc), cudaMemcpyHostToDevice, st));

    Geom g;
    memset(&g, 0, sizeof g);
    g.P = sched.P;
    g.m = sched.m;
    g.base[SPACE_SEND] = (char*)const_cast<void*>(sendbuf);
    g.base[SPACE_RECV] = (char*)recvbuf;
    g.base[SPACE_WORK] = nullptr;
    g.rank_pitch[SPACE_SEND] = g.m;
    g.rank_pitch[SPACE_RECV] = (uint64_t)g.P * g.m;
    g.rank_pitch[SPACE_WORK] = (uint64_t)g.P * g.m;
    BarrierCtl ctl;
    ctl.counter = ctl_words;
    ctl.status = ctl_words + 1;
    ctl.base = 0;
    ctl.expected = (unsigned)grid;
    ctl.timeout_ns = kDefaultTimeoutNs;
    ctl.mbar_extra_tx = 0;
    ctl.trace = nullptr;
    int first_idx = 0, last_idx = (int)n - 1;
    const PhaseDesc* descs = d_descs;
    const VarTask* no_tasks = nullptr;
    const VarRange* no_ranges = nullptr;
    void* args[] = {&g, &descs, &first_idx, &last_idx, &ctl, &no_tasks, &no_ranges};
    CU(cudaLaunchCooperativeKernel(fn, dim3((unsigned)grid), dim3(kVecBlock), args, 0, st));
    unsigned words[2] = {0, 0};
    CU(cudaMemcpyAsync(words, ctl_words, sizeof words, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return words[1] == DEV_OK ? SPARBIT_OK : SPARBIT_ERR_TIMEOUT;
}

}  // extern "C"
