/*
 * sparbit.h - C ABI of the B200 step executor for the Sparbit allgather (Stripe Parallel
 * Binomial Trees) and its comparators.
 *
 * The P ranks of a communicator are P virtual ranks resident in one GPU's memory.  Rank r owns
 * one send block of m bytes and one receive buffer of P slots of m bytes.  A collective runs the
 * chosen algorithm's exchange schedule; each step of the schedule is one data-parallel copy pass
 * over all ranks, a forwarded block being read from the SENDING rank's receive buffer and written
 * into its final slot of the RECEIVING rank's receive buffer, as the algorithm prescribes.  The
 * result is the one MPI_Allgather defines (paper, Section II): slot j of every receive buffer
 * holds the block sent by rank j.
 *
 * Notation: m is the bytes of ONE block (sendcount = recvcount = m).  The paper writes m for the
 * total a process ends up with and m/p for a block.
 *
 * Layout (all device pointers, caller-owned, contiguous):
 *   sendbuf   P * m bytes        rank r's block at byte offset r * m
 *   recvbuf   P * P * m bytes    rank r's buffer at r * P * m, slot b at + b * m
 *   workspace P * P * m bytes    Bruck only (its rotated working buffers), same layout
 *
 * Phases of a collective, in execution order:
 *   -1          local copy of the own block, sendbuf[r] -> recvbuf[r][r] (Bruck: -> workspace[r][0]).
 *               Algorithm 1 sends displacement `rank` at j = 0 as if it were in place already;
 *               Section II's semantics need this copy.  MPI_IN_PLACE is not supported.
 *   0 .. K-1    the algorithm's communication steps (Sparbit: Algorithm 1's loop, K = ceil(log2 P)).
 *   K           Bruck only: the final rotation workspace[r][i] -> recvbuf[r][(r + i) mod P]
 *               (the "memory shifts" of Section II-B).
 * Every phase ends with the equivalent of Algorithm 1's MPI_Waitall: no copy of the next phase
 * starts before all copies of this one are visible.
 *
 * Conventions: every function is extern "C", never throws, never aborts the process.  Functions
 * returning int return SPARBIT_OK (0) or a positive SPARBIT_ERR_* code.  Nothing here
 * synchronises the device unless its comment says so.  All argument errors are found on the
 * host before anything is launched.  A plan may be used by one host thread and on one stream at
 * a time, and belongs to the device that was current at its first launch (later calls with
 * another device current return SPARBIT_ERR_ARG).
 */
#ifndef SPARBIT_H
#define SPARBIT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SPARBIT_OK = 0,
    SPARBIT_ERR_ARG = 1,         /* null handle/buffer, P < 1, phase range or enum out of range */
    SPARBIT_ERR_OVERFLOW = 2,    /* P*P*m (or an internal work count) is not representable */
    SPARBIT_ERR_ALIAS = 3,       /* send / receive / workspace byte ranges overlap */
    SPARBIT_ERR_UNSUPPORTED = 4, /* recursive doubling with P not a power of two; neighbor
                                    exchange with odd P; bad mode combination */
    SPARBIT_ERR_WORKSPACE = 5,   /* Bruck without a workspace, or one that is too small */
    SPARBIT_ERR_CUDA = 6,        /* a CUDA runtime call failed; see sparbit_last_cuda_error() */
    SPARBIT_ERR_TIMEOUT = 7,     /* the device-side grid barrier gave up waiting */
    SPARBIT_ERR_NOMEM = 8,       /* host allocation failed */
    SPARBIT_ERR_LIMIT = 9,       /* beyond a fixed limit of the entry point: the scratch of
                                    sparbit_allgather_noalloc, P of sparbit_plan_create_v / _validate */
    SPARBIT_ERR_BARRIER = 10     /* the caller's cross-device barrier (sparbit_allgather_multi)
                                    returned non-zero */
};

/* Algorithms (paper, Section II-A and Section III).  Only Sparbit is the product's hot path; the
 * other four run on the same executor as comparators. */
enum {
    SPARBIT_ALGO_SPARBIT = 0,
    SPARBIT_ALGO_RING = 1,
    SPARBIT_ALGO_RECURSIVE_DOUBLING = 2, /* powers of two only, as the paper states */
    SPARBIT_ALGO_BRUCK = 3,
    SPARBIT_ALGO_NEIGHBOR_EXCHANGE = 4   /* even P only, as the paper states */
};

/* How the phases are put on the GPU.  When a call runs phases -1 and 0 together they are executed
 * as ONE pass (the own block is read once from sendbuf and written both to its own slot and to
 * the first peer's): same state after phase 0, one pass less. */
enum {
    SPARBIT_EXEC_AUTO = 0,       /* the measured best on B200: MIRROR up to 64 KiB of receive
                                    buffers in all (up to 2 MiB for blocks of 16 B to 4 KiB,
                                    where the chain with a grouped front is not at least as
                                    fast), FLOW for collectives that move 0.4 to 6 GB (unless
                                    COPY_AUTO gives them the bulk engine and m is not a multiple
                                    of 128 B: the vector engine, which FLOW runs on, is 10-30 %
                                    slower on blocks that straddle 128-byte lines), the chain of
                                    per-pass kernels otherwise - as a graph, or kernel by kernel
                                    (STREAM) while it is short (thresholds: SPARBIT_TUNE_*) */
    SPARBIT_EXEC_PERSISTENT = 1, /* one cooperative kernel, bounded-wait grid barrier per pass */
    SPARBIT_EXEC_GRAPH = 2,      /* one kernel per pass, chained by programmatic dependent launch
                                    in a CUDA graph cached per buffer set (4 sets; further sets
                                    re-parameterise the least recently used graph).  Sparbit's
                                    (and recursive doubling's) leading passes share ONE kernel
                                    where the ranks fall into independent groups small enough
                                    for a CTA each (SPARBIT_TUNE_GROUPED_FRONT) */
    SPARBIT_EXEC_STREAM = 3,     /* the same kernels launched one by one on the stream; what AUTO
                                    resolves to for a chain of few kernels
                                    (SPARBIT_TUNE_STREAM_MAX_LAUNCHES) */
    SPARBIT_EXEC_FLOW = 4,       /* one kernel (all CTAs resident) without grid barriers:
                                    Algorithm 1's Waitall is kept per rank (counters of what each
                                    rank has received), so a pass starts where its senders are
                                    ready while the pass before is still finishing elsewhere.
                                    Takes every pass by default (SPARBIT_TUNE_FLOW_MIN_PASS_SPANS
                                    leaves small leading passes to chained per-pass kernels).
                                    Whole collectives of fixed-size blocks of at least 32 vectors
                                    on the vector engine; other calls run as GRAPH */
    SPARBIT_EXEC_MIRROR = 5      /* a whole small collective in ONE CTA: every block written to a
                                    receive buffer is also kept in an on-chip copy of the receive
                                    buffers (shared memory), and every forwarded block is read from
                                    that copy of the sending rank's buffer, so a pass costs a
                                    shared-memory access instead of two trips to global memory.
                                    Same passes, same order, same slots.  When P*P*m (twice that
                                    for Bruck, whose working buffers are kept the same way) does
                                    not fit one SM's shared memory (227 KB on B200), or exceeds
                                    64 KiB, a cluster of up to 16 CTAs shares the work: rank r's
                                    on-chip copy lives in CTA r mod C, a sender stores into the
                                    receiver's CTA through distributed shared memory, and a CTA
                                    starts a pass when the bytes its ranks receive in the passes
                                    before have arrived (one mbarrier per pass counts them; bounded
                                    wait, time-out through sparbit_plan_status).  Needs
                                    ceil(P/16)*P*m to fit one SM, fixed-size blocks, at most 16
                                    passes and a call that starts at the first pass (the on-chip
                                    copy starts empty); other calls run as GRAPH */
};

/* Which copy engine a phase uses. */
enum {
    SPARBIT_COPY_AUTO = 0,   /* BULK for 16-byte aligned buffers, m >= 8 KiB and about 1 GB or more
                                moved by the collective (2*P*(P-1)*m >= 10^9), else VECTOR */
    SPARBIT_COPY_VECTOR = 1, /* warp-cooperative ld/st.global, 16/8/4/2/1-byte vectors */
    SPARBIT_COPY_BULK = 2    /* cp.async.bulk global->shared->global ring (needs 16-byte
                                alignment of buffers and m); falls back to VECTOR otherwise */
};

/* Address spaces a message endpoint can live in. */
enum { SPARBIT_SPACE_SEND = 0, SPARBIT_SPACE_RECV = 1, SPARBIT_SPACE_WORKSPACE = 2 };

typedef struct sparbit_plan_s sparbit_plan_t; /* opaque; owned by the library */

/* One single-block message of a phase, as Algorithm 1 issues them (one MPI_Isend/MPI_Irecv pair
 * per block).  Slots are displacements in blocks inside the rank's buffer of that space. */
typedef struct {
    int32_t phase;
    int32_t src_rank;
    int32_t dst_rank;
    int32_t src_space;
    int32_t src_slot;
    int32_t dst_space;
    int32_t dst_slot;
} sparbit_msg;

/*
 * sparbit_plan - the short form: a Sparbit plan with automatic executor choice for P ranks and
 * blocks of block_bytes.  Returns NULL on any error (use sparbit_plan_create for the code).
 * Host-only: runs Algorithm 1's set-up (lines 1-5) and derives the per-step descriptors; makes
 * no CUDA call.  Device resources (a few hundred bytes plus the descriptor table) are allocated
 * by the first sparbit_allgather on the plan, which should therefore not be inside a stream
 * capture.
 */
sparbit_plan_t* sparbit_plan(int P, size_t block_bytes);

/*
 * sparbit_plan_create - full form.  algo: SPARBIT_ALGO_*; exec: SPARBIT_EXEC_*.  On success
 * *out receives a plan the caller must release with sparbit_plan_destroy.  block_bytes may be 0
 * (the collective is then a no-op, as MPI allows count 0).  Errors: ERR_ARG (P < 1, null out,
 * unknown enum), ERR_OVERFLOW (P*P*block_bytes does not fit in 63 bits, or P > 2^24),
 * ERR_UNSUPPORTED (recursive doubling with P not a power of two, neighbor exchange with odd P:
 * Section II-A defines them for those P only), ERR_NOMEM.  Host-only.
 * Environment: when exec is AUTO, SPARBIT_EXEC=persistent|graph|stream|flow|mirror replaces the
 * automatic choice; SPARBIT_COPY=vector|bulk presets the copy engine (sparbit_plan_set_copy_path
 * still overrides it).  Other values are ignored.
 */
int sparbit_plan_create(int P, size_t block_bytes, int algo, int exec, sparbit_plan_t** out);

/*
 * sparbit_plan_create_v - a plan for blocks of DIFFERENT sizes, i.e. MPI_Allgatherv with
 * contiguous displacements, on the same schedules (the paper's Section VII names Allgatherv as
 * the next target; the schedules themselves never look inside a block, so they carry over
 * unchanged).  block_bytes: host array of P byte counts, block_bytes[j] = what rank j
 * contributes (0 allowed); it is copied.  With T = the sum of the counts and off[j] = the sum
 * of the counts below j:
 *   sendbuf   T bytes       rank r's block at byte offset off[r]
 *   recvbuf   P * T bytes   rank r's buffer at r * T, block j at + off[j]
 * The plan is then used with sparbit_allgather, sparbit_allgather_steps and
 * sparbit_allgather_host exactly like a fixed-size plan (introspection included).  Both copy
 * engines (the bulk engine when all counts and the buffers are multiples of 16 bytes; COPY_AUTO
 * applies its thresholds to the average block) and the GRAPH, STREAM and PERSISTENT executors,
 * and MIRROR in one CTA where P * T fits one SM's shared memory (EXEC_AUTO uses it up to 64 KiB;
 * larger plans run as GRAPH).  FLOW is refused (ERR_UNSUPPORTED: its units assume equal blocks),
 * and so is Bruck (its rotated workspace assumes equal blocks).  P is limited to 8192 here and P * T to 2^48 bytes
 * (ERR_LIMIT, ERR_OVERFLOW beyond: the plan keeps one 16-byte task record per 4 KiB of every
 * copy, with 48-bit offsets).  Other errors as for sparbit_plan_create.  Host-only.
 */
int sparbit_plan_create_v(int P, const size_t* block_bytes, int algo, int exec, sparbit_plan_t** out);

/* Releases the plan and everything it owns (device table, graph).  Synchronises the device if
 * the plan ever launched work.  NULL is allowed. */
int sparbit_plan_destroy(sparbit_plan_t* plan);

/*
 * sparbit_allgather - the collective (paper, Section II; Sparbit: Algorithm 1).  Mirrors
 * MPI_Allgather(sendbuf, m, MPI_BYTE, recvbuf, m, MPI_BYTE, comm) for a communicator of P ranks.
 *   sendbuf  device, P*m bytes, read only          recvbuf  device, P*P*m bytes, fully overwritten
 *   stream   a cudaStream_t passed as void* (NULL = the legacy default stream)
 * Asynchronous: work is enqueued on `stream` and the call returns (in MPI terms this is the
 * non-blocking form; synchronising the stream, or sparbit_plan_status, is the wait).  Any alignment of the
 * pointers and any m >= 1 give the right answer; 16-byte aligned buffers with m % 16 == 0 get
 * the fast paths.  Errors (nothing is launched): ERR_ARG (null plan; null buffer with P*m > 0),
 * ERR_ALIAS (ranges overlap), ERR_WORKSPACE (Bruck without workspace), ERR_CUDA.
 * A device-side barrier time-out is reported later by sparbit_plan_status.
 * On a stream that is being captured (after the plan's first, uncaptured call) the collective
 * goes into the caller's graph as plain chained per-pass kernels - the mirror kernel as itself -
 * whatever executor the plan names: the persistent and the flow kernel take counter values of
 * one particular launch as arguments and would not replay.  The captured graph may be replayed
 * any number of times.
 */
int sparbit_allgather(sparbit_plan_t* plan, const void* sendbuf, void* recvbuf, void* stream);

/*
 * sparbit_allgather_steps - run only phases first..last (inclusive; -1 <= first <= last <=
 * sparbit_plan_last_phase).  For step-by-step comparison with a reference; same contract as
 * sparbit_allgather otherwise.  Phases skipped are the caller's business: the buffers must
 * already hold what the earlier phases would have produced.
 */
int sparbit_allgather_steps(sparbit_plan_t* plan, const void* sendbuf, void* recvbuf, void* stream,
                            int first, int last);

/*
 * sparbit_allgather_host - the same collective for HOST buffers (host_send P*m bytes, host_recv
 * P*P*m bytes; pinned memory makes the copies faster but is not required).  Copies the send
 * blocks to device staging owned by the plan (allocated on first use), runs the collective,
 * copies all P receive buffers back, and SYNCHRONISES before returning.  Errors as for
 * sparbit_allgather, plus ERR_TIMEOUT if the device barrier gave up.
 */
int sparbit_allgather_host(sparbit_plan_t* plan, const void* host_send, void* host_recv);

/* ---- introspection (host-only, no CUDA call) ------------------------------------------------ */

/* K, the number of communication steps: Sparbit and Bruck ceil(log2 P), recursive doubling
 * log2 P, ring P-1, neighbor exchange P/2 (the latency terms of the cost formulae of Sections
 * II-A and III-B). */
int sparbit_plan_num_steps(const sparbit_plan_t* plan);

/* Index of the last phase: K-1, or K for Bruck (rotation).  -1 when P = 1 and not Bruck. */
int sparbit_plan_last_phase(const sparbit_plan_t* plan);

/*
 * Step variables of one communication step (0 <= step < K).  distance: ranks between sender and
 * receiver (Algorithm 1's d).  blocks_per_rank: messages each rank sends in the step
 * (Algorithm 1's data - ignore).  ignore: 1 if the step withholds a block (Sparbit only, else 0).
 * Any out pointer may be NULL.
 */
int sparbit_plan_step_info(const sparbit_plan_t* plan, int step, int* distance, int* blocks_per_rank,
                           int* ignore);

/*
 * Expands the compact descriptor of one phase (-1 .. last phase) into explicit single-block
 * messages, using the same index function the kernels use.  Writes min(cap, *n) entries to out
 * (out may be NULL when cap is 0) and always stores the full count in *n.  Order inside a phase
 * is unspecified.
 */
int sparbit_plan_messages(const sparbit_plan_t* plan, int phase, sparbit_msg* out, size_t cap, size_t* n);

/*
 * Host-side check of what the kernels will execute, in place of a device race detector: every
 * pass of the full collective (the fused first pass included) is expanded through the kernels'
 * own index function and checked for (a) ranks and slots inside their buffers, (b) no location
 * read before an earlier pass has filled it, (c) inside a pass, no location written twice and
 * none both read and written, (d) every receive slot written exactly once over the collective.
 * Section III-B withholds blocks for exactly this purpose: so that no slot is written twice.
 * Returns SPARBIT_OK, or SPARBIT_ERR_ARG with the
 * offending phase in *bad_phase (may be NULL; last phase + 1 = the final count), SPARBIT_ERR_LIMIT
 * for P > 8192 (the check needs P*P bytes of host memory), SPARBIT_ERR_NOMEM.  Host-only.
 */
int sparbit_plan_validate(const sparbit_plan_t* plan, int* bad_phase);

/* ---- placement of the ranks on several devices (host-only, no CUDA call) --------------------
 *
 * Section III-C of the paper discusses how the mapping of processes to machines decides how much
 * of each step's traffic crosses the network: with the sequential mapping neighbouring ranks
 * share a machine, so Sparbit's late steps (small distance, most of the data) stay inside it;
 * with the cyclic mapping they are the ones that leave it.  These calls state the same thing for
 * G devices: they split the messages of a phase into the copies a device performs inside its own
 * memory and the blocks it has to hand to each other device.  They only describe the split; the
 * sparbit_allgather_multi* calls further down execute it.
 */
enum {
    SPARBIT_MAP_SEQUENTIAL = 0, /* device g holds ranks [floor(g*P/G), floor((g+1)*P/G)) */
    SPARBIT_MAP_CYCLIC = 1      /* rank r sits on device r mod G */
};

/* The device that holds `rank` when P ranks are placed on G devices; -1 on a bad argument. */
int sparbit_rank_device(int P, int G, int mapping, int rank);

/*
 * Counts the single-block messages of one phase (-1 .. last phase) by sending and receiving
 * device: blocks[s * G + d] = blocks that ranks on device s send to ranks on device d in that
 * phase (s == d: copies that stay local).  blocks must hold G*G entries; multiply by m for
 * bytes.  1 <= G <= 4096.  Errors: ERR_ARG, ERR_NOMEM.
 */
int sparbit_plan_partition(const sparbit_plan_t* plan, int G, int mapping, int phase, uint64_t* blocks);

/*
 * The messages of one phase that go from device src_device to device dst_device (equal: the
 * local copy list of that device), same record and conventions as sparbit_plan_messages.
 * Over all G*G pairs every message of the phase appears exactly once.
 */
int sparbit_plan_partition_messages(const sparbit_plan_t* plan, int G, int mapping, int phase, int src_device,
                                    int dst_device, sparbit_msg* out, size_t cap, size_t* n);

/*
 * ---- One communicator on G devices (paper, Section III-C; locality argument of Sections II-B, III)
 *
 * The calls above describe the split; these execute it.  Device g holds, packed in increasing
 * rank order, the send blocks ([n_g][m]) and the receive buffers ([n_g][P][m]) of the n_g ranks
 * the mapping gives it.  A step of the schedule is one kernel per device: the device that holds
 * the SENDING rank performs the copy - it reads the block from its own memory (the sender's
 * receive buffer, as in the single-device executor) and stores it into the receiving rank's
 * buffer, which is its own memory or, through a plain peer pointer, another device's.  A kernel
 * never waits for another device.  Algorithm 1's Waitall between steps is a barrier ACROSS the
 * devices, supplied by the caller.  Sparbit, ring, recursive doubling and neighbor exchange with
 * fixed-size blocks; Bruck (working buffers, rotation) and variable sizes: ERR_UNSUPPORTED.
 * The plan is only read: one plan may serve every device of a process, and each process of a
 * multi-process job creates its own with the same (P, m, algorithm).
 *
 * recv_bases: HOST array of G DEVICE pointers, entry g = start of device g's receive buffers as
 * THIS device can address it (its own allocation for g == device, a peer mapping otherwise; an
 * entry may be NULL for a device that holds no rank).  The widest vector (16 B down to 1 B) that
 * divides m and every pointer is used.  Peer access must be enabled by the caller
 * (cudaDeviceEnablePeerAccess, or sparbit_ipc_open between processes).  All buffers stay owned
 * by the caller.  1 <= G <= SPARBIT_MULTI_MAX_DEVICES.
 */
#define SPARBIT_MULTI_MAX_DEVICES 16

/* Ranks held by `device`; -1 on a bad argument.  Sequential: floor((g+1)P/G) - floor(gP/G). */
int sparbit_multi_rank_count(int P, int G, int mapping, int device);
/* Position of `rank` among the ranks of the device that holds it (sparbit_rank_device); -1 on a
 * bad argument. */
int sparbit_multi_local_index(int P, int G, int mapping, int rank);

/*
 * Enqueues on `stream` (of the CURRENT device, which plays `device`) this device's share of the
 * phases first_phase .. last_phase (-1 .. last phase; a call that runs -1 and 0 executes them as
 * one pass where the schedule allows).  No barrier is issued: the caller must separate two steps
 * by a cross-device barrier itself (run one step per call), or be the only "device" that
 * matters - e.g. all G devices emulated on one GPU and one stream, where stream order is the
 * barrier.  Errors: ERR_ARG, ERR_UNSUPPORTED, ERR_OVERFLOW, ERR_LIMIT (more than 66 passes in
 * one call), ERR_CUDA.  Nothing is launched for a device without ranks.
 */
int sparbit_allgather_multi_phases(const sparbit_plan_t* plan, int G, int mapping, int device,
                                   const void* send_local, void* const* recv_bases, void* stream, int first_phase,
                                   int last_phase);

/*
 * The cross-device barrier of sparbit_allgather_multi.  It must arrange that work enqueued on
 * `stream` AFTER it returns starts only when every device's work enqueued BEFORE its own call of
 * the barrier is complete and visible (e.g. a one-element all-reduce of a communication library
 * enqueued on `stream`; or cudaStreamSynchronize followed by a host barrier).  0 = success.
 */
typedef int (*sparbit_device_barrier_fn)(void* ctx, void* stream);

/*
 * The whole collective for this device: barrier (every device has entered, its receive buffers
 * may be written), then pass by pass with a barrier after every communication step - after the
 * last one too, so that the result is complete when work enqueued after this call runs.  Every
 * device of the communicator must make the same call.  barrier may be NULL only for G == 1.
 * Errors as above, and ERR_BARRIER when the barrier returns non-zero (passes already enqueued
 * stay enqueued).
 */
int sparbit_allgather_multi(const sparbit_plan_t* plan, int G, int mapping, int device, const void* send_local,
                            void* const* recv_bases, void* stream, sparbit_device_barrier_fn barrier,
                            void* barrier_ctx);

/*
 * One process per device: how a process lets the others address its receive buffers.  The paper
 * has no counterpart (MPI moves the bytes there).  sparbit_ipc_export writes the 64-byte handle
 * of the device allocation that contains dev_ptr and dev_ptr's offset inside it; the allocation
 * must come from cudaMalloc (not from a pool of mapped virtual memory).  sparbit_ipc_open, in
 * another process, maps that allocation (enabling peer access to its device where needed) and
 * returns the same location as *dev_ptr, plus *mapping_base for sparbit_ipc_close.  A process
 * must not open its own handle; an allocation is opened at most once per process.
 */
#define SPARBIT_IPC_HANDLE_BYTES 64
int sparbit_ipc_export(const void* dev_ptr, void* handle /* 64 bytes, host */, uint64_t* offset);
int sparbit_ipc_open(const void* handle, uint64_t offset, void** dev_ptr, void** mapping_base);
int sparbit_ipc_close(void* mapping_base);

/*
 * The same kind of check for the bookkeeping of the FLOW executor, which replaces the Waitall of
 * Algorithm 1 by per-rank counters: for vector_bytes-wide vectors (1, 2, 4, 8 or 16) and
 * resident_warps warps, the work units of every pass, decoded the way the kernel decodes them,
 * must cover each rank's copies exactly once; the units that write into a rank's buffer must
 * number what the counter of that (rank, pass) is compared with; and a pass must wait for every
 * earlier pass of the kernel that writes the space it reads.  *first_flow_pass (may be NULL)
 * receives the position, in the executed sequence of passes, of the first pass the flow kernel
 * takes (the ones before it run as per-pass kernels).  SPARBIT_OK, SPARBIT_ERR_ARG with the
 * offending pass in *bad_pass (may be NULL), SPARBIT_ERR_UNSUPPORTED if no pass of the plan can
 * run in the flow kernel with that vector width and warp count, SPARBIT_ERR_LIMIT for more than
 * 2^26 spans in a pass.  Host-only.
 */
int sparbit_plan_validate_flow(const sparbit_plan_t* plan, int vector_bytes, int resident_warps,
                               int* first_flow_pass, int* bad_pass);

/* Bytes of workspace the plan needs: 0, or P*P*m for Bruck. */
size_t sparbit_plan_workspace_bytes(const sparbit_plan_t* plan);

/* Gives the plan its workspace (device memory; the caller keeps ownership and must keep it alive
 * while the plan is used).  ERR_WORKSPACE if bytes is too small. */
int sparbit_plan_set_workspace(sparbit_plan_t* plan, void* dev, size_t bytes);

/* Forces the copy engine (SPARBIT_COPY_*).  BULK silently runs as VECTOR for a call whose
 * buffers or m are not 16-byte aligned. */
int sparbit_plan_set_copy_path(sparbit_plan_t* plan, int copy_path);

/*
 * Thresholds behind the automatic choices, per plan.  Defaults come from sweeps on B200; a value
 * set here holds for all later calls on the plan (cached graphs are rebuilt).
 */
enum {
    SPARBIT_TUNE_BULK_MIN_BLOCK_BYTES = 0, /* COPY_AUTO: smallest m that gets the bulk engine (8 KiB) */
    SPARBIT_TUNE_BULK_MIN_MOVED_BYTES = 1, /* COPY_AUTO: and only if 2*P*(P-1)*m reaches this (10^9) */
    SPARBIT_TUNE_FLOW_UNITS_PER_WARP = 2,  /* EXEC_FLOW: a pass is cut into units of 1..4 warp spans
                                              so that every warp gets at least about this many (1) */
    SPARBIT_TUNE_FLOW_MAX_UNIT_SPANS = 3,  /* EXEC_FLOW: largest unit, in warp spans of 1 KiB (8) */
    SPARBIT_TUNE_FLOW_MIN_MOVED_BYTES = 4, /* EXEC_AUTO: FLOW when 2*P*(P-1)*m is at least this (4*10^8) */
    SPARBIT_TUNE_FLOW_MAX_MOVED_BYTES = 5, /* ... and below this (6*10^9); GRAPH otherwise */
    SPARBIT_TUNE_MIRROR_MAX_BYTES = 6,     /* EXEC_AUTO: MIRROR when P*P*m is at most this (64 KiB) */
    SPARBIT_TUNE_FLOW_MIN_PASS_SPANS = 7,  /* EXEC_FLOW: the flow kernel takes the passes at the end of
                                              the collective that have at least this many 1 KiB warp
                                              spans in all (1, the default: every pass - measured equal
                                              or up to 2 % faster than any split; 0: one per resident
                                              warp, 4736 on B200); smaller leading passes run as chained
                                              per-pass kernels in front of it */
    SPARBIT_TUNE_MIRROR_MAX_VECTORS = 8,   /* EXEC_AUTO: MIRROR only when the largest pass moves at most this
                                              many vectors (65536: 2 MiB of receive buffers in 16-byte
                                              vectors) ... */
    SPARBIT_TUNE_MIRROR_CLUSTER_MAX_BLOCK = 9, /* ... and, where P*P*m exceeds MIRROR_MAX_BYTES, m is at most
                                              this (4 KiB) */
    SPARBIT_TUNE_MIRROR_CTA_VECTORS = 10,  /* EXEC_MIRROR: the cluster is doubled while a CTA would get more
                                              vectors than this in the largest pass (256) */
    SPARBIT_TUNE_MIRROR_THREAD_VECTORS = 11, /* EXEC_MIRROR: vectors of the largest pass per thread (4), CTAs
                                              of at most 1024 threads */
    SPARBIT_TUNE_FLOW_COOPERATIVE = 12,    /* EXEC_FLOW: 1 = every launch of the flow kernel is a cooperative
                                              launch; 0 (default) = only the first one and those that go to
                                              another stream than the flow launch before (any plan, same
                                              device): launches that follow one another in ONE stream are
                                              ordered anyway, start ahead of their predecessor's end and save
                                              2-2.5 us each */
    SPARBIT_TUNE_FLOW_SKIP_WAITS = 13,     /* measurement hook, EXEC_FLOW: 1 = no unit waits for its source
                                              rank's counters.  The receive buffers are then WRONG (blocks
                                              are forwarded before they have arrived); the time is what the
                                              kernel would take if waiting cost nothing, the bound on what any
                                              finer readiness tracking could gain (bench.py
                                              --flow-wait-bound).  0 by default */
    SPARBIT_TUNE_GROUPED_FRONT = 14,       /* GRAPH and STREAM executors, Sparbit: 1 (default) = the leading
                                              passes whose distance is a multiple of some G that divides P
                                              run as G independent groups of P/G ranks, one CTA per group
                                              working from an on-chip copy of its part of the receive
                                              buffers (one kernel instead of one per pass), as far as a
                                              group's part stays within MIRROR_MAX_BYTES; 0 = every pass its
                                              own kernel */
    SPARBIT_TUNE_FLOW_WIDE_MAX_MOVED_BYTES = 15, /* EXEC_FLOW: a collective that moves less than this (9*10^8)
                                              in blocks of at least 128 vectors (2 KiB) runs the flow kernel
                                              with four vectors per lane (warp spans of 2 KiB) instead of
                                              two: much of it is served by L2, which takes more loads in
                                              flight than DRAM rewards (P = 256, m = 4 KiB: 85.0 us against
                                              90.3); 0 = never */
    SPARBIT_TUNE_VEC_DENSE_MAX_RECV_BYTES = 16, /* GRAPH and STREAM executors, vector engine: while the receive
                                              buffers total at most this (256 MiB, about twice the L2) a full
                                              per-pass kernel runs three CTAs per SM instead of two (1-5 %:
                                              P = 256, m = 2 KiB 45.4 us against 46.7); 0 = never */
    SPARBIT_TUNE_STREAM_MAX_LAUNCHES = 17, /* EXEC_AUTO: a chain of per-pass kernels on the vector engine that
                                              needs at most this many launches (6; the grouped front counts
                                              as one) is launched kernel by kernel (STREAM) instead of as a
                                              graph: back-to-back graph launches start 1-2 us apart from one
                                              another where plain launches overlap (P = 256, m = 8 B: 9.8 us
                                              of GPU time against 11.8), but each plain launch costs the host
                                              2-3 us where a whole graph costs it 1.8 us, so longer chains
                                              would leave a caller in a tight loop bound by its own
                                              launches; 0 = always GRAPH */
    SPARBIT_TUNE_COUNT_ = 18
};
int sparbit_plan_set_tunable(sparbit_plan_t* plan, int key, uint64_t value);
int sparbit_plan_get_tunable(const sparbit_plan_t* plan, int key, uint64_t* value);

/* What the plan resolved to: executor (SPARBIT_EXEC_*, never AUTO) and the copy engine the last
 * launch used (SPARBIT_COPY_*; AUTO before the first launch). */
int sparbit_plan_exec_mode(const sparbit_plan_t* plan);
int sparbit_plan_copy_path(const sparbit_plan_t* plan);

/* Kernels (and graph launches) the library has enqueued for this plan so far. */
int sparbit_plan_launch_counts(const sparbit_plan_t* plan, uint64_t* kernel_launches, uint64_t* graph_launches);

/*
 * Synchronises the plan's last stream and reports the device status word: SPARBIT_OK, or
 * SPARBIT_ERR_TIMEOUT if a wait inside a kernel gave up (the kernel then returned early and the
 * receive buffers are incomplete).  Clears the condition so the plan can be used again.
 * *device_status (may be NULL) receives the raw word: 0 = none; 1 = a grid barrier of the
 * persistent executor or a wait of the flow executor for a rank's counters; 2 = a wait for bytes
 * on an mbarrier (bulk engine, cluster form of the mirror executor).
 */
int sparbit_plan_status(sparbit_plan_t* plan, int* device_status);

/*
 * Per-pass time stamps of the PERSISTENT executor (off by default; the other executors are timed
 * from outside, kernel by kernel).  With tracing on, CTA 0 stores the GPU's nanosecond timer at
 * kernel start and each time it leaves a pass (for all passes but the last: after the grid
 * barrier that ends it), so entry k+1 minus entry k is pass k as that CTA saw it, Waitall
 * included.  sparbit_plan_get_trace synchronises the plan's last stream and copies the stamps of
 * the last persistent launch: min(cap, *n) entries, *n = passes + 1 (0 if nothing was traced).
 * The first traced call allocates the stamp buffer (not inside a stream capture).
 */
int sparbit_plan_set_trace(sparbit_plan_t* plan, int on);
int sparbit_plan_get_trace(sparbit_plan_t* plan, uint64_t* ns, size_t cap, size_t* n);

/*
 * Test hook for the bounded wait of the grid barrier: the next persistent launches expect
 * `extra_arrivals` more arrivals than there are CTAs and give up after `timeout_ns`
 * nanoseconds (0 restores the defaults: no extra arrivals, 2 s).  With extra_arrivals > 0 the
 * barrier can never complete, so the kernel must return with the time-out status instead of
 * hanging.
 */
int sparbit_plan_set_barrier_test(sparbit_plan_t* plan, int extra_arrivals, uint64_t timeout_ns);

/*
 * sparbit_allgather_noalloc - the collective for callers that must not allocate device memory.
 * (The paper has no counterpart for this entry point; it exists for the library's users.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - an application whose device
 * memory is fully owned by its own pool or framework allocator, a plug-in that is handed
 * buffers and a stream and nothing else, a service that may not take the driver's allocation
 * lock once it is up.  sparbit_allgather keeps a small device-side scratch per plan (the
 * per-phase descriptor table and the grid barrier's counter and status word) and obtains it with
 * cudaMalloc on the plan's first launch; this entry point keeps the same scratch in a fixed
 * 2 KiB array that is part of the library image, so it performs no cudaMalloc, cudaFree or any
 * other allocating CUDA or framework call, at any time.  Every GPU that loads the library
 * carries those 2 KiB until the process exits.  On the host it uses only short-lived ordinary
 * heap memory for the schedule.
 *
 * It runs the persistent executor with the vector copy engine (the same kernel and the same
 * passes sparbit_allgather launches for EXEC_PERSISTENT / COPY_VECTOR, the fused first pass
 * included), for algo = SPARBIT, RING, RECURSIVE_DOUBLING or NEIGHBOR_EXCHANGE; sendbuf / recvbuf /
 * stream as for sparbit_allgather.  Unlike sparbit_allgather it WAITS: the work is enqueued on
 * `stream`, then the call synchronises that stream, on every call, and the return value is
 * final - SPARBIT_OK, or SPARBIT_ERR_TIMEOUT if the grid barrier gave up (recvbuf is then
 * incomplete).  Because it waits it cannot be used on a stream that is being captured: such a
 * call returns SPARBIT_ERR_UNSUPPORTED and enqueues nothing.
 *
 * Limit: the array holds 28 pass descriptors, i.e. any Sparbit or recursive-doubling collective
 * this library accepts (at most 24 passes), rings of at most 29 ranks and neighbor exchanges of
 * at most 56.  Anything larger is refused with SPARBIT_ERR_LIMIT before anything is enqueued.
 * Bruck needs a P*P*m workspace and is refused with SPARBIT_ERR_UNSUPPORTED.
 *
 * The first call on each device looks up the array's device address (once per device, with that
 * device current).  All calls on a
 * device share the one array, and it keeps what the previous call left: each call re-writes the
 * descriptors and clears the barrier words on `stream` before its kernel.  Calls whose GPU work
 * overlaps (two host threads on one device) race on the scratch: serialise them.
 * Other errors: as for sparbit_plan_create and sparbit_allgather.
 */
int sparbit_allgather_noalloc(int P, size_t block_bytes, int algo, const void* sendbuf, void* recvbuf,
                              void* stream);

/*
 * Test hook for the other bounded wait, the bulk engine's wait for a shared-memory stage to
 * fill: the next launches expect `extra_tx_bytes` (a multiple of 16, at most 65536) more bytes
 * per stage than are loaded, so no stage ever reports full; after `timeout_ns` nanoseconds
 * (0 = the default 2 s) the waiting lane must set the time-out status and the kernel must return
 * (every load it issued has long landed by then, so nothing is in flight).  0 bytes switches the
 * hook off.  Shares the time limit with sparbit_plan_set_barrier_test.
 */
int sparbit_plan_set_mbarrier_test(sparbit_plan_t* plan, uint32_t extra_tx_bytes, uint64_t timeout_ns);

const char* sparbit_strerror(int code);

/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* sparbit_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SPARBIT_H */
