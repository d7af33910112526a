// The P ranks of one communicator placed on G devices (Section III-C: process mappings).
//
// Device g holds the send blocks and the receive buffers of the ranks mapped to it, packed in
// increasing rank order.  A step of the schedule is then one kernel PER DEVICE: the device that
// holds the SENDING rank executes the copy, reading the block from its own memory (the sender's
// receive buffer, as the schedule says) and storing it into the receiving rank's buffer - its own
// memory when the receiver is local, the peer's memory through a plain peer pointer when it is
// not.  Nothing here waits on another device inside a kernel: Algorithm 1's Waitall between steps
// is a barrier across the devices that the caller supplies (stream-ordered, e.g. a one-element
// all-reduce of its communication library on the same stream, or a host barrier after a stream
// synchronise).  No bulk-copy engine and no cluster features: peer stores are ordinary 16-byte
// vector stores.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "../../include/sparbit.h"
#include "phase_desc.h"
#include "plan_access.h"

using namespace spb;

namespace {

#define CU(call)                                                      \
    do {                                                              \
        cudaError_t e_ = (call);                                      \
        if (e_ != cudaSuccess) return record_cuda_error((int)e_, #call); \
    } while (0)

constexpr int kMaxDevices = SPARBIT_MULTI_MAX_DEVICES;
constexpr int kBlock = 512;
constexpr int kUnroll = 4;

struct MultiGeom {
    uint32_t P, G, me, cyclic;
    uint32_t n_local;               // ranks held by this device
    uint32_t pad_;
    uint64_t m;                     // bytes per block
    const char* send;               // this device's send blocks, [n_local][m]
    char* recv[kMaxDevices];        // device g's receive buffers, [n_g][P][m]; peer pointers for g != me
    uint32_t first[kMaxDevices + 1];  // sequential mapping: first rank of device g (first[G] = P)
};

__device__ __forceinline__ uint32_t device_of(const MultiGeom& g, uint32_t r) {
    // (r + 1) * G fits 32 bits: P <= 2^24 (schedule limit), G <= 16
    return g.cyclic ? r % g.G : ((r + 1u) * g.G - 1u) / g.P;
}
// rank held at position li of this device
__device__ __forceinline__ uint32_t global_rank(const MultiGeom& g, uint32_t li) {
    return g.cyclic ? g.me + li * g.G : g.first[g.me] + li;
}
// where rank r's receive buffer starts (r on any device)
__device__ __forceinline__ char* recv_of(const MultiGeom& g, uint32_t r) {
    const uint32_t dev = device_of(g, r);
    const uint32_t li = g.cyclic ? r / g.G : r - g.first[dev];
    return g.recv[dev] + (uint64_t)li * g.P * g.m;
}

template <typename V>
__device__ __forceinline__ V ld_stream(const V* p) { return __ldcg(p); }
template <typename V>
__device__ __forceinline__ void st_stream(V* p, V v) { __stcg(p, v); }

// One phase, the copies whose sender lives on this device.  Same decomposition into warp tasks as
// the single-device vector engine: spans of 32 * kUnroll vectors inside a copy, or, for copies
// shorter than a warp row, whole copies side by side in a row.
template <typename V>
__global__ void __launch_bounds__(kBlock, 2) multi_phase_vec_kernel(const __grid_constant__ MultiGeom g,
                                                                    const __grid_constant__ PhaseDesc d) {
    // launched with programmatic stream serialization: nothing is read or written before the
    // kernel ahead on the stream (the step before, or the caller's barrier) has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp_id = blockIdx.x * (kBlock / 32) + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * (kBlock / 32);
    const uint32_t P = g.P;
    const uint64_t vpc64 = d.copy_bytes / sizeof(V);
    const uint32_t n_copies = g.n_local * d.copies;
    const bool from_send = d.src_space == SPACE_SEND;

    if (vpc64 >= 32) {
        const uint32_t span = 32u * kUnroll;
        const uint32_t spc = (uint32_t)((vpc64 + span - 1) / span);
        const uint64_t tasks = (uint64_t)n_copies * spc;
        for (uint64_t w = warp_id; w < tasks; w += n_warps) {
            const uint32_t w32 = (uint32_t)w;
            const uint32_t q = w32 / spc;
            const uint32_t sp = w32 - q * spc;
            const uint32_t li = q / d.copies;
            const uint32_t j = q - li * d.copies;
            const uint32_t r = global_rank(g, li);
            const CopyLoc c = locate_copy(d, P, r, j);
            const char* mine = g.recv[g.me] + (uint64_t)li * P * g.m;
            const V* src = reinterpret_cast<const V*>(from_send ? g.send + (uint64_t)li * g.m
                                                                : mine + (uint64_t)c.src_slot * g.m);
            V* dst = reinterpret_cast<V*>(recv_of(g, c.dst_rank) + (uint64_t)c.dst_slot * g.m);
            V* dst2 = reinterpret_cast<V*>(const_cast<char*>(mine) + (uint64_t)c.dst_slot * g.m);
            const uint64_t v0 = (uint64_t)sp * span + lane;
            V regs[kUnroll];
#pragma unroll
            for (int k = 0; k < kUnroll; k++) {
                const uint64_t v = v0 + 32u * k;
                if (v < vpc64) regs[k] = ld_stream<V>(src + v);
            }
#pragma unroll
            for (int k = 0; k < kUnroll; k++) {
                const uint64_t v = v0 + 32u * k;
                if (v < vpc64) {
                    st_stream<V>(dst + v, regs[k]);
                    if (d.dup_self) st_stream<V>(dst2 + v, regs[k]);
                }
            }
        }
    } else if (vpc64 > 0) {
        const uint32_t vpc = (uint32_t)vpc64;
        const uint32_t cpw = 32u / vpc;       // whole copies per warp row
        const uint32_t sub = lane / vpc;
        const uint32_t v = lane - sub * vpc;
        const bool lane_on = sub < cpw;
        const uint64_t tasks = ((uint64_t)n_copies + cpw - 1) / cpw;
        for (uint64_t w = warp_id; w < tasks; w += n_warps) {
            const uint64_t q64 = w * cpw + sub;
            if (!lane_on || q64 >= n_copies) continue;
            const uint32_t q = (uint32_t)q64;
            const uint32_t li = q / d.copies;
            const uint32_t j = q - li * d.copies;
            const uint32_t r = global_rank(g, li);
            const CopyLoc c = locate_copy(d, P, r, j);
            char* mine = g.recv[g.me] + (uint64_t)li * P * g.m;
            const V* src = reinterpret_cast<const V*>(from_send ? g.send + (uint64_t)li * g.m
                                                                : mine + (uint64_t)c.src_slot * g.m);
            const V x = ld_stream<V>(src + v);
            st_stream<V>(reinterpret_cast<V*>(recv_of(g, c.dst_rank) + (uint64_t)c.dst_slot * g.m) + v, x);
            if (d.dup_self) st_stream<V>(reinterpret_cast<V*>(mine + (uint64_t)c.dst_slot * g.m) + v, x);
        }
    }
    // the next kernel on the stream may be placed on the SMs now; it waits as this one did
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename V>
const void* kernel_fn() { return (const void*)multi_phase_vec_kernel<V>; }
const void* pick_kernel(int vbytes) {
    switch (vbytes) {
        case 16: return kernel_fn<uint4>();
        case 8: return kernel_fn<uint2>();
        case 4: return kernel_fn<unsigned>();
        case 2: return kernel_fn<unsigned short>();
        default: return kernel_fn<unsigned char>();
    }
}

bool mapping_ok(int mapping) { return mapping == SPARBIT_MAP_SEQUENTIAL || mapping == SPARBIT_MAP_CYCLIC; }

uint32_t seq_first(uint32_t P, uint32_t G, uint32_t g) { return (uint32_t)(((uint64_t)g * P) / G); }

uint32_t ranks_on(uint32_t P, uint32_t G, int mapping, uint32_t g) {
    if (mapping == SPARBIT_MAP_CYCLIC) return g < P ? (P - g + G - 1) / G : 0;
    return seq_first(P, G, g + 1) - seq_first(P, G, g);
}

// The passes a whole collective runs, in order: the own-block copy fused with the first step where
// the schedule offers that, else every phase on its own.
struct PassList {
    const PhaseDesc* d[66];
    int phase[66];  // the phase a pass completes (the fused pass: 0)
    int n = 0;
};

int list_passes(const Schedule& sc, int first, int last, PassList& out) {
    if (first < -1 || last > sc.last_phase() || first > last) return SPARBIT_ERR_ARG;
    if (last - first + 1 > 66) return SPARBIT_ERR_LIMIT;
    int ph = first;
    if (first == -1 && last >= 0 && sc.has_fused_first) {
        out.d[out.n] = &sc.fused_first;
        out.phase[out.n++] = 0;
        ph = 1;
    }
    for (; ph <= last; ph++) {
        out.d[out.n] = &sc.phase(ph);
        out.phase[out.n++] = ph;
    }
    return SPARBIT_OK;
}

int check_common(const sparbit_plan_t* plan, int G, int mapping, int device, const Schedule** sc) {
    *sc = plan_schedule(plan);
    if (!*sc || !mapping_ok(mapping) || G < 1 || G > kMaxDevices || device < 0 || device >= G) return SPARBIT_ERR_ARG;
    if (plan_is_variable(plan) || (*sc)->algo == ALGO_BRUCK) return SPARBIT_ERR_UNSUPPORTED;
    return SPARBIT_OK;
}

int launch_pass(const Schedule& sc, const PhaseDesc& d, int G, int mapping, int device, const void* send_local,
                void* const* recv_bases, cudaStream_t stream) {
    MultiGeom g;
    memset(&g, 0, sizeof g);
    g.P = sc.P;
    g.G = (uint32_t)G;
    g.me = (uint32_t)device;
    g.cyclic = mapping == SPARBIT_MAP_CYCLIC;
    g.n_local = ranks_on(sc.P, (uint32_t)G, mapping, (uint32_t)device);
    g.m = sc.m;
    g.send = (const char*)send_local;
    uintptr_t bits = (uintptr_t)send_local | (uintptr_t)sc.m;
    for (int k = 0; k <= G; k++) g.first[k] = seq_first(sc.P, (uint32_t)G, (uint32_t)k);
    for (int k = 0; k < G; k++) {
        g.recv[k] = (char*)recv_bases[k];
        bits |= (uintptr_t)recv_bases[k];
    }
    if (g.n_local == 0 || sc.m == 0 || d.copies == 0) return SPARBIT_OK;
    int vbytes = 16;
    while (vbytes > 1 && (bits & (uintptr_t)(vbytes - 1))) vbytes >>= 1;
    const uint64_t vpc = d.copy_bytes / (uint64_t)vbytes;
    const uint64_t n_copies = (uint64_t)g.n_local * d.copies;
    if (n_copies >> 32) return SPARBIT_ERR_OVERFLOW;
    uint64_t tasks;
    if (vpc >= 32) {
        const uint64_t span = 32ull * kUnroll;
        tasks = n_copies * ((vpc + span - 1) / span);
    } else {
        const uint64_t cpw = 32 / vpc;
        tasks = (n_copies + cpw - 1) / cpw;
    }
    if (tasks >> 32) return SPARBIT_ERR_OVERFLOW;
    int dev = 0, sms = 0;
    CU(cudaGetDevice(&dev));
    CU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const uint64_t wpb = kBlock / 32;
    uint64_t ctas = (tasks + wpb - 1) / wpb;
    if (ctas > (uint64_t)sms * 2) ctas = (uint64_t)sms * 2;
    PhaseDesc dd = d;
    void* args[2] = {&g, &dd};
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(kBlock);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CU(cudaLaunchKernelExC(&cfg, pick_kernel(vbytes), args));
    return SPARBIT_OK;
}

int check_buffers(const Schedule& sc, int G, int mapping, int device, const void* send_local,
                  void* const* recv_bases) {
    if (!recv_bases) return SPARBIT_ERR_ARG;
    if (sc.m == 0) return SPARBIT_OK;
    for (int k = 0; k < G; k++)
        if (!recv_bases[k] && ranks_on(sc.P, (uint32_t)G, mapping, (uint32_t)k)) return SPARBIT_ERR_ARG;
    if (!send_local && ranks_on(sc.P, (uint32_t)G, mapping, (uint32_t)device)) return SPARBIT_ERR_ARG;
    return SPARBIT_OK;
}

}  // namespace

extern "C" {

int sparbit_multi_rank_count(int P, int G, int mapping, int device) {
    if (P < 1 || G < 1 || device < 0 || device >= G || !mapping_ok(mapping)) return -1;
    return (int)ranks_on((uint32_t)P, (uint32_t)G, mapping, (uint32_t)device);
}

int sparbit_multi_local_index(int P, int G, int mapping, int rank) {
    if (P < 1 || G < 1 || rank < 0 || rank >= P || !mapping_ok(mapping)) return -1;
    if (mapping == SPARBIT_MAP_CYCLIC) return rank / G;
    const uint32_t dev = (uint32_t)((((uint64_t)rank + 1) * (uint32_t)G - 1) / (uint32_t)P);
    return rank - (int)seq_first((uint32_t)P, (uint32_t)G, dev);
}

int sparbit_allgather_multi_phases(const sparbit_plan_t* plan, int G, int mapping, int device,
                                   const void* send_local, void* const* recv_bases, void* stream, int first_phase,
                                   int last_phase) {
    const Schedule* sc = nullptr;
    int rc = check_common(plan, G, mapping, device, &sc);
    if (rc != SPARBIT_OK) return rc;
    if ((rc = check_buffers(*sc, G, mapping, device, send_local, recv_bases)) != SPARBIT_OK) return rc;
    PassList pl;
    if ((rc = list_passes(*sc, first_phase, last_phase, pl)) != SPARBIT_OK) return rc;
    for (int i = 0; i < pl.n; i++) {
        rc = launch_pass(*sc, *pl.d[i], G, mapping, device, send_local, recv_bases, (cudaStream_t)stream);
        if (rc != SPARBIT_OK) return rc;
    }
    return SPARBIT_OK;
}

int sparbit_allgather_multi(const sparbit_plan_t* plan, int G, int mapping, int device, const void* send_local,
                            void* const* recv_bases, void* stream, sparbit_device_barrier_fn barrier,
                            void* barrier_ctx) {
    const Schedule* sc = nullptr;
    int rc = check_common(plan, G, mapping, device, &sc);
    if (rc != SPARBIT_OK) return rc;
    if (!barrier && G > 1) return SPARBIT_ERR_ARG;
    if ((rc = check_buffers(*sc, G, mapping, device, send_local, recv_bases)) != SPARBIT_OK) return rc;
    PassList pl;
    if ((rc = list_passes(*sc, -1, sc->last_phase(), pl)) != SPARBIT_OK) return rc;
    // every device has entered the collective: its receive buffers may be written from now on
    if (G > 1 && barrier(barrier_ctx, stream) != 0) return SPARBIT_ERR_BARRIER;
    for (int i = 0; i < pl.n; i++) {
        rc = launch_pass(*sc, *pl.d[i], G, mapping, device, send_local, recv_bases, (cudaStream_t)stream);
        if (rc != SPARBIT_OK) return rc;
        // Algorithm 1's Waitall: what the other devices stored in this step is complete before
        // the next step reads it (after the last step: before the caller reads the result).
        // The own-block copy alone writes local memory only and needs none.
        if (G > 1 && pl.phase[i] >= 0 && barrier(barrier_ctx, stream) != 0) return SPARBIT_ERR_BARRIER;
    }
    return SPARBIT_OK;
}

int sparbit_ipc_export(const void* dev_ptr, void* handle, uint64_t* offset) {
    if (!dev_ptr || !handle || !offset) return SPARBIT_ERR_ARG;
    static_assert(sizeof(cudaIpcMemHandle_t) == SPARBIT_IPC_HANDLE_BYTES, "handle size");
    // the handle names the allocation that contains dev_ptr; find where that allocation starts
    typedef int (*range_fn)(unsigned long long*, size_t*, unsigned long long);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult found;
    CU(cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &found));
    if (!fn || found != cudaDriverEntryPointSuccess) return SPARBIT_ERR_UNSUPPORTED;
    unsigned long long base = 0;
    size_t size = 0;
    if (((range_fn)fn)(&base, &size, (unsigned long long)(uintptr_t)dev_ptr) != 0) return SPARBIT_ERR_ARG;
    cudaIpcMemHandle_t h;
    CU(cudaIpcGetMemHandle(&h, (void*)(uintptr_t)base));
    memcpy(handle, &h, sizeof h);
    *offset = (uint64_t)((uintptr_t)dev_ptr - (uintptr_t)base);
    return SPARBIT_OK;
}

int sparbit_ipc_open(const void* handle, uint64_t offset, void** dev_ptr, void** mapping_base) {
    if (!handle || !dev_ptr || !mapping_base) return SPARBIT_ERR_ARG;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle, sizeof h);
    void* base = nullptr;
    CU(cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess));
    *mapping_base = base;
    *dev_ptr = (char*)base + offset;
    return SPARBIT_OK;
}

int sparbit_ipc_close(void* mapping_base) {
    if (!mapping_base) return SPARBIT_ERR_ARG;
    CU(cudaIpcCloseMemHandle(mapping_base));
    return SPARBIT_OK;
}

}  // extern "C"
