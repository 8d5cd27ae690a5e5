/*
 * tfps -- batched critical-path evaluation of one data-flow graph under many
 * candidate partitions (sm_100a CUDA library, C ABI).
 *
 * Problem tuple (paper, Section 2): DAG G=(V,E) with vertex cost c_v and edge
 * size t_e; k devices with speed s_d and capacity C_d; bandwidth matrix B.
 * A partition p: V -> D places every vertex on a device.
 *
 * Cost model in integer ticks (S = `scale` ticks per paper time unit):
 *   rt(v)   = ceil(c_v * S / s_p(v))                       execution time c/s, Section 2
 *   w(u->v) = 0 if p(u)==p(v)                              Section 4.1 (text before Eq. 12)
 *             else ceil(t_uv * S / B[p(u)][p(v)])          B indexed [source device][target device]
 *   tlevel(v) = max over in-edges (u->v) of tlevel(u)+rt(u)+w(u->v); 0 for sources
 *               (earliest start; recursion of Eq. 6 with execution and transfer times)
 *   blevel(v) = rt(v) + max over out-edges (v->x) of w(v->x)+blevel(x); rt(v) for sinks
 *               (path computation time, Eq. 12)
 *   CP        = max_v tlevel(v)+rt(v)                      start of the artificial sink, Section 2 after Eq. 1
 *   load[d]   = sum of rt(v) over vertices on d            the sum inside Eq. 7
 *   memload[d]= sum of mem_v over vertices on d; bit d of viol set iff memload[d] >= C_d
 *               (Eq. 2 is a strict inequality)
 *
 * Conventions common to all calls
 *   - Every function returns TFPS_OK (0) or a negative tfps_status.  Nothing
 *     throws, aborts or traps.  tfps_last_error() gives a thread-local message.
 *   - "dev" pointers are CUDA device pointers on the handle's device, "host"
 *     pointers are ordinary host memory.  The caller owns every buffer it
 *     passes; the handle owns private device copies of graph and tables and
 *     keeps no reference to caller memory after a call returns (asynchronous
 *     calls read/write caller buffers until the stream reaches their end).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Vertex ids are 0..n-1 in any order.  Parallel edges are legal (max
 *     semantics).  A self loop or cycle gives TFPS_ERR_CYCLE.
 *   - Candidate matrices are vertex-major: element (v, j) of a matrix with
 *     leading dimension ldp lives at index v*ldp + j; ldp >= P and ldp % 16 == 0.
 *     Columns P..ldp-1 are padding: read but never written.
 */
#ifndef TFPS_H
#define TFPS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tfps_graph tfps_graph;

typedef enum tfps_status {
    TFPS_OK = 0,
    TFPS_ERR_INVALID_ARG = -1,   /* NULL where data is required, negative size, bad enum, bad ldp */
    TFPS_ERR_BAD_CSR = -2,       /* ptr not monotone / wrong end, index out of range, in/out edge multisets differ, negative c/t/mem */
    TFPS_ERR_CYCLE = -3,         /* graph is not acyclic */
    TFPS_ERR_BAD_DEVICES = -4,   /* k outside 1..TFPS_K_MAX, s_d < 1, off-diagonal B < 1, C_d < 0, scale < 1 */
    TFPS_ERR_BAD_PARTITION = -5, /* a partition id >= k (reported through the status word) */
    TFPS_ERR_OVERFLOW = -6,      /* a path length or load could reach 2^62 ticks */
    TFPS_ERR_WORKSPACE = -7,     /* workspace NULL or too small */
    TFPS_ERR_UNSUPPORTED = -8,   /* size beyond an implementation limit */
    TFPS_ERR_CUDA = -9,          /* a CUDA runtime call failed (message in tfps_last_error) */
    TFPS_ERR_TIMEOUT = -10,      /* a bounded device-side wait ran out */
    TFPS_ERR_STATE = -11         /* call order: devices not set, levels not built */
} tfps_status;

enum { TFPS_K_MAX = 64 };
enum { TFPS_I32 = 0, TFPS_I64 = 1 };          /* dtype selectors for t and mem */
enum { TFPS_HOST = 0, TFPS_DEVICE = 1 };      /* where the arrays given to tfps_graph_create live */

/* flags of tfps_eval_batch / tfps_eval_workspace_bytes */
enum {
    TFPS_EVAL_AUTO = 0,
    TFPS_EVAL_LEVEL_SYNC = 1 << 0,   /* one launch per topological level, thread = (vertex, candidates) */
    TFPS_EVAL_SLICED = 1 << 1,       /* one persistent block per candidate slice walks all levels */
    TFPS_EVAL_NO_VALIDATE = 1 << 4,  /* caller guarantees every id < k; skips the id check */
    TFPS_EVAL_SCRATCH_LEVELS = 1 << 5, /* workspace query: caller will pass tlevel == NULL and blevel == NULL */
    TFPS_EVAL_PROFILE = 1 << 6        /* record CUDA events around the phases, read back with tfps_phase_times */
};

const char* tfps_strerror(int status);
const char* tfps_last_error(void);

/*
 * Tuning and test overrides.  The library chooses kernel family and block shape
 * by itself; the environment variables below override single choices and exist
 * for measurements and tests.  They are read at every call (TFPS_TILE_SPLIT,
 * TFPS_STEP_ORDER, TFPS_LEAN*, TFPS_LEVREC when tfps_devices_set packs its
 * records), change speed only, never results:
 *   TFPS_LEAN=0 / TFPS_LEAN64=0 / TFPS_LEVREC=0   switch a kernel family off
 *   TFPS_LEAN_FORCE_WIDE=1, TFPS_LEAN_ORDER=1|2    64-bit plan; plan in level order | in the caller's numbering
 *   TFPS_LEAN_SLICE, TFPS_LEAN_CPT, TFPS_LEAN_DEPTH, TFPS_SLICED_CPT, TFPS_SLICED_WARPS, TFPS_SLICED_TABLE, TFPS_LEVEL32
 *                                                  candidates per block / per lane, stage depth, warps, cost tables
 *   TFPS_OVERLAP_LOADS=0, TFPS_OVERLAP_PASSES=0    loads kernel / backward pass on the caller's stream only
 *   TFPS_LOADS2=0, TFPS_LOADS_CPT, TFPS_LOADS_BLOCKS_PER_SM   shape of the load kernel
 *   TFPS_TILE_SPLIT                                edges per work item of the record passes (default 8)
 *   TFPS_STEP_ORDER=1|2                            steps = topological levels | runs of the caller's numbering
 *   TFPS_STEP_PERSISTENT=1, TFPS_STEP_GROUPS, TFPS_STEP_TILES, TFPS_STEP_RUN, TFPS_STEP_SHAPE, TFPS_STEP_BLOCKS
 *                                                  persistent record pass and its shape
 *   TFPS_STEP_FLOW=1                               dataflow record pass (ready bits per vertex and tile of 128
 *                                                  candidates instead of grid-wide steps; k <= 16, P <= 4096)
 *   TFPS_WAIT_LIMIT                                polls before a device-side wait gives up (default 2^20;
 *                                                  0 makes every wait run out at once: TFPS_ERR_TIMEOUT)
 */

/*
 * Build a graph handle (Section 2: G, c, t; optional per-vertex memory).
 *   n, m         vertices, edges (n < 2^26, m < 2^31 - 64; larger sizes give TFPS_ERR_UNSUPPORTED)
 *   in_ptr[n+1], in_src[m], in_t[m]     in-edge CSR: row v lists the sources u of edges u->v and their sizes
 *   out_ptr[n+1], out_dst[m], out_t[m]  out-edge CSR; pass all three NULL to have it built by transposing.
 *                                       When given, it must hold the same multiset of (u, v, t) edges.
 *   t_dtype      TFPS_I32 or TFPS_I64 (element type of in_t/out_t), t >= 0
 *   c[n]         int32 vertex cost, c >= 0
 *   mem, mem_dtype  per-vertex memory >= 0, or NULL: mem_v = total size of v's out-edges
 *                (Section 2: data leaving the source vertex of an edge consumes device memory)
 *   ptr_space    TFPS_HOST or TFPS_DEVICE: where all of the above arrays live
 * The arrays are copied; the CSR is validated on the host (device arrays are
 * fetched first).  Synchronises `stream`.  On error *out is NULL.
 */
int tfps_graph_create(tfps_graph** out, int64_t n, int64_t m,
                      const int64_t* in_ptr, const int32_t* in_src, const void* in_t,
                      const int64_t* out_ptr, const int32_t* out_dst, const void* out_t,
                      int t_dtype, const int32_t* c, const void* mem, int mem_dtype,
                      int ptr_space, void* stream);

/* Free the handle and everything it owns (device memory included).  NULL is allowed. */
int tfps_graph_destroy(tfps_graph* g);

/* n, m, number of topological levels (0 until built), k (0 until devices are set). host outputs, any may be NULL */
int tfps_graph_info(const tfps_graph* g, int64_t* n, int64_t* m, int32_t* num_levels, int32_t* k);

/*
 * Set the device tables (Section 2: speeds s, capacities C, bandwidth matrix B).
 *   k            1..TFPS_K_MAX
 *   s[k]         host int32, s_d >= 1
 *   C[k]         host int64, C_d >= 0, INT64_MAX = unbounded
 *   B[k*k]       host int64 row-major [source device][target device]; off-diagonal >= 1 and < 2^62, diagonal ignored
 *   scale        S >= 1, ticks per paper time unit
 * Builds the per-device and per-device-pair exact-division constants and the
 * per-vertex / per-edge scaled numerators.  Requires max c*S and max t*S below
 * 2^62 and the bound  sum_v ceil(c_v S / min s) + sum_e ceil(t_e S / min B)  < 2^62,
 * else TFPS_ERR_OVERFLOW.  Synchronous (default stream).
 */
int tfps_devices_set(tfps_graph* g, int k, const int32_t* s, const int64_t* C, const int64_t* B, int64_t scale);

/*
 * Topological levels by a Kahn frontier on the GPU (a vertex is schedulable
 * once all incoming data is available, Section 2).
 *   level[n]     dev int32 or NULL: 0 for sources, else 1 + max level of a predecessor
 *   order[n]     dev int32 or NULL: vertices grouped by level, ascending id inside a level
 *   level_ptr    host int64[cap] or NULL: level l is order[level_ptr[l] .. level_ptr[l+1])
 *   cap          entries available in level_ptr; TFPS_ERR_INVALID_ARG if cap < num_levels+1
 *   num_levels   host int32 or NULL
 * The structure is built on the first call (also implicitly by tfps_eval_batch)
 * and cached.  Synchronises `stream`.  A cyclic graph gives TFPS_ERR_CYCLE.
 */
int tfps_topo_levels(tfps_graph* g, int32_t* level, int32_t* order,
                     int64_t* level_ptr, int64_t cap, int32_t* num_levels, void* stream);

/*
 * Bytes of caller workspace tfps_eval_batch needs.  0 unless flags contains
 * TFPS_EVAL_SCRATCH_LEVELS (critical-path length wanted without either level
 * matrix), in which case one int64 [n][ldp] matrix is needed.
 */
size_t tfps_eval_workspace_bytes(const tfps_graph* g, int64_t P, int64_t ldp, int flags);

/*
 * Evaluate P candidate partitions.  Asynchronous on `stream`.
 *   part         dev uint8 [n][ldp], part[v*ldp+j] = device of vertex v under candidate j (< k)
 *   tlevel       dev int64 [n][ldp] or NULL
 *   blevel       dev int64 [n][ldp] or NULL     (the PCT priority of Eq. 12)
 *   cp           dev int64 [P] or NULL
 *   load         dev int64 [k][ldp] or NULL
 *   memload      dev int64 [k][ldp] or NULL
 *   viol         dev uint64 [P] or NULL; bit d = capacity of device d violated
 *   workspace    dev, 256-byte aligned, workspace_bytes >= tfps_eval_workspace_bytes(...); may be NULL when that is 0
 *   flags        TFPS_EVAL_* (kernel variant; validation)
 * part and every output that is given must be 16-byte aligned (the kernels move ids
 * and levels as 16-byte vectors; ldp is a multiple of 16, so every row then is):
 * a misaligned pointer gives TFPS_ERR_INVALID_ARG and nothing is launched.
 * The forward pass runs when tlevel is wanted, or when cp is wanted and blevel
 * is not; the backward pass runs when blevel is wanted.  P == 0 or n == 0:
 * TFPS_OK, nothing written.  Host-detectable errors are returned at once and
 * nothing is launched.  An id >= k is found on the device: every later kernel
 * of the call then returns without touching memory, outputs are unspecified,
 * and tfps_get_status reports TFPS_ERR_BAD_PARTITION.  The device status is
 * sticky: until tfps_get_status has read (and cleared) it, the kernels of later
 * calls on the handle return at once as well, although those calls return TFPS_OK.
 */
int tfps_eval_batch(tfps_graph* g, int64_t P, int64_t ldp,
                    const uint8_t* part, int64_t* tlevel, int64_t* blevel,
                    int64_t* cp, int64_t* load, int64_t* memload, uint64_t* viol,
                    void* workspace, size_t workspace_bytes, int flags, void* stream);

/*
 * Same evaluation from HOST buffers: part is host uint8 [n][ldp]; tlevel and
 * blevel (host int64 [n][ldp]), cp[P], load[k*ldp], memload[k*ldp], viol[P] are
 * host outputs, any of which may be NULL.  Copies the ids to the device, runs
 * the load kernel and BOTH passes (the level matrices live in scratch owned by
 * the handle and are copied back only when a host pointer is given), copies
 * the other results back and synchronises `stream`.  Large batches go up in two
 * column chunks on an internal copy stream so that the second half's transfer
 * overlaps the first half's evaluation.  Staging and scratch buffers (and that
 * stream) are created on demand and stay with the handle.  Pinned host memory makes
 * the copies asynchronous and fast; pageable memory works too.  Returns the
 * device status as tfps_get_status would.
 */
int tfps_eval_batch_host(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part,
                         int64_t* tlevel, int64_t* blevel,
                         int64_t* cp, int64_t* load, int64_t* memload, uint64_t* viol,
                         int flags, void* stream);

/*
 * Device time in milliseconds of the phases of the most recent tfps_eval_batch
 * call that carried TFPS_EVAL_PROFILE: ms[0] = load/validate/violation
 * kernels, ms[1] = forward pass, ms[2] = backward pass (0 for a phase that did
 * not run).  Synchronises on the recorded events.
 */
int tfps_phase_times(tfps_graph* g, float ms[3]);

/*
 * Name of the pass kernel family the most recent tfps_eval_batch call on this handle chose ("" before any call):
 *   "pass_lean_kernel"       candidate-sliced, shared-memory window, 32-bit levels inside (k <= 8, paths < 2^31)
 *   "pass_lean64_kernel"     the same with 64-bit levels (k <= 16)
 *   "pass_sliced_kernel"     candidate-sliced without a window (neighbours through L2)
 *   "pass_stepchain_kernel"  step-synchronous on vertex records, one chained launch per step (k <= 64)
 *   "pass_steprec_kernel"    the same as one persistent cooperative launch with bounded barriers (opt-in)
 *   "pass_flow_kernel"       the same records as one persistent launch without steps: an item waits (bounded) for the
 *                            ready bits of exactly the rows it reads (opt-in)
 *   "pass_level_kernel"      step-synchronous with a division per relaxation (any device table)
 * The string is static.
 */
const char* tfps_last_pass_kernel(const tfps_graph* g);

/* Number of kernels this library has launched in the calling process so far. */
int64_t tfps_kernel_launches(void);

/*
 * Diagnostic (no counterpart in the paper): the rate, in GB/s, at which the SMs of
 * the current device gather pseudo-random 1 KiB row segments of a buffer of
 * `working_set_bytes` (16 bytes per lane and load, every warp reads `rows_per_warp`
 * rows).  It is the access pattern of the step-synchronous passes -- a neighbour's
 * levels and ids for one tile of candidates -- without their arithmetic, and so
 * the ceiling those passes can reach.  Allocates and frees its own buffer,
 * synchronises the device.  *gbytes_per_s is a host output.
 */
int tfps_probe_gather_bandwidth(size_t working_set_bytes, int rows_per_warp, double* gbytes_per_s);

/*
 * Diagnostic (no counterpart in the paper): the same with the passes' writes.  A buffer of
 * `total_bytes` is written once, row by row (1 KiB rows in ascending order, dealt to the
 * warps round robin); before a warp writes a row it reads `reads` rows picked pseudo-randomly
 * among the `window_bytes` before it, and what it writes depends on what it read.  Reports
 * (reads + 1) KiB per row over the time of the third launch, in GB/s: what the memory system
 * sustains for a wavefront that reads its recent output out of L2 while the older output is
 * written back to DRAM.  layout 0: every 16-byte load of a warp covers 512 contiguous
 * bytes, read past L1; layout 1: a lane reads 32 contiguous bytes as two loads through L1
 * (the chained record pass' layout).  Allocates and frees its own buffer, synchronises the device.
 */
int tfps_probe_wavefront_bandwidth(size_t total_bytes, size_t window_bytes, int reads, int layout, double* gbytes_per_s);

/*
 * Critical-path lengths without any allocation.  (The paper has no counterpart
 * of this call; it exists for callers of this library that are not allowed to
 * allocate device memory when they evaluate: code running inside a framework's
 * allocator-managed region or under a memory budget that must not move, plug-ins
 * that are handed buffers but no allocator, and real-time loops where a
 * cudaMalloc -- which may synchronise the whole device -- is unacceptable.)
 *
 * Same result as tfps_eval_batch(g, P, ldp, part, NULL, NULL, cp, NULL, NULL,
 * NULL, workspace, ...): cp[j] for the P candidates of `part` (dev uint8
 * [n][ldp]) into `cp` (dev int64 [P]).  The forward pass needs one int64
 * [n][ldp] matrix of scratch; here it lives in a fixed array inside the library
 * (TFPS_NOALLOC_SCRATCH_BYTES, resident on every GPU that loads the library
 * until the process exits) instead of a caller workspace.  The call performs no
 * cudaMalloc/cudaFree and calls no allocating routine.
 *
 *   - n*ldp*8 must not exceed TFPS_NOALLOC_SCRATCH_BYTES, else TFPS_ERR_WORKSPACE.
 *   - tfps_devices_set must have been called (it builds everything the pass
 *     needs), else TFPS_ERR_STATE.
 *   - The device address of the scratch array is looked up once per device by
 *     tfps_devices_set (a synchronous set-up call: make it outside of any stream
 *     capture), so the evaluation call itself finds the address cached.
 *   - All calls on a device share the one array.  It keeps whatever the last call
 *     left in it; nothing in it has to start at zero, because every cell the
 *     pass reads was written earlier in the same call.  Two calls that overlap
 *     on the GPU (different streams, different handles, different host threads)
 *     race on it: serialise them.
 *   - Asynchronous on `stream` like tfps_eval_batch; id errors are reported
 *     through tfps_get_status.
 */
#define TFPS_NOALLOC_SCRATCH_BYTES ((size_t)32 << 20)
int tfps_eval_cp_noalloc(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int64_t* cp,
                         int flags, void* stream);

/*
 * Placement constraints (Section 2).  tfps_constraints_set stores the lists with
 * the handle (host arrays, copied; an earlier set is replaced; synchronous):
 *   pair_a[npairs], pair_b[npairs]      collocation constraints (Eq. 3): vertices pair_a[i] and
 *                                       pair_b[i] must be placed on the same device
 *   dc_vertex[ndev], dc_device[ndev]    device constraints (Eq. 4): vertex dc_vertex[i] must be
 *                                       placed on device dc_device[i] (0 .. TFPS_K_MAX - 1)
 * Every listed pair is one requirement; a vertex index outside 0..n-1 gives
 * TFPS_ERR_INVALID_ARG.  tfps_eval_constraints counts, for each of the P candidates
 * of `part` (dev uint8 [n][ldp], 16-byte aligned), the requirements that do not hold:
 *   coll_viol    dev int32 [P] or NULL: violated collocation pairs
 *   dev_viol     dev int32 [P] or NULL: violated device constraints
 * Asynchronous on `stream`; needs neither the device tables nor the topological
 * levels.  With empty lists the outputs are zero.
 */
int tfps_constraints_set(tfps_graph* g, int64_t npairs, const int32_t* pair_a, const int32_t* pair_b,
                         int64_t ndev, const int32_t* dc_vertex, const int32_t* dc_device);
int tfps_eval_constraints(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part,
                          int32_t* coll_viol, int32_t* dev_viol, void* stream);

/*
 * Critical vertices of evaluated candidates (Section 3.2: the critical path is the
 * longest path from a source to a sink).  mask[v*ldp+j] = 1 where vertex v lies on
 * a longest path of candidate j, i.e. tlevel + blevel == cp, else 0.
 *   tlevel, blevel   dev int64 [n][ldp] as written by tfps_eval_batch
 *   cp               dev int64 [P]
 *   mask             dev uint8 [n][ldp]; padding columns are not written
 * All four 16-byte aligned, ldp a multiple of 16; TFPS_ERR_INVALID_ARG otherwise
 * (nothing is launched).  Asynchronous on `stream`; needs no graph handle.
 */
int tfps_critical_mask(int64_t n, int64_t P, int64_t ldp, const int64_t* tlevel, const int64_t* blevel,
                       const int64_t* cp, uint8_t* mask, void* stream);

/*
 * Vertex ranks (Section 3.2, Eq. 5 and Eq. 6), independent of any partition and of the
 * device tables:
 *   upRank(v)    = c_v + max over successors x of upRank(x)      (a sink: c_v)
 *   downRank(v)  = c_v + max over predecessors u of downRank(u)  (a source: c_v)
 *   totalRank(v) = upRank(v) + downRank(v)                       (Section 3.2.1; c_v is in both)
 *   up, down, total   dev int64 [n] each, any of them NULL when not wanted
 * One launch per topological level and direction.  Asynchronous on `stream`.
 * TFPS_ERR_OVERFLOW if twice the sum of all costs could reach 2^62.
 */
int tfps_ranks(tfps_graph* g, int64_t* up, int64_t* down, int64_t* total, void* stream);

/*
 * The critical path of the Critical Path strategy (Section 3.2.2, steps 1-4): the sink of
 * largest downward rank (equal ranks: the smallest id), then backwards along predecessors
 * of largest downward rank (equal: the smallest id) to a source.
 *   down   dev int64 [n] from tfps_ranks
 *   path   dev int32 [n]; receives the path's vertices from the source to the sink
 *   len    host; number of vertices written
 * Synchronises `stream` (the length comes back to the host).
 */
int tfps_critical_path(tfps_graph* g, const int64_t* down, int32_t* path, int64_t* len, void* stream);

/*
 * Batch Split (Section 3.2.1): vertices in descending order of total rank (equal ranks:
 * ascending id), each assigned to the fastest device (equal speeds: lower index) whose
 * static memory use stays BELOW its capacity with the vertex on it (Eq. 2).  A vertex no
 * device can take goes to the fastest device and is counted.  Uses the device tables of
 * tfps_devices_set (speeds, capacities) and the graph's per-vertex memory.
 *   total      dev int64 [n] from tfps_ranks
 *   part       dev uint8 [n]; receives the device of every vertex
 *   unplaced   host; number of vertices no device could take
 * Synchronises `stream`.  TFPS_ERR_STATE before tfps_devices_set.
 */
int tfps_batch_split(tfps_graph* g, const int64_t* total, uint8_t* part, int64_t* unplaced, void* stream);

/*
 * Critical Path partitioning (Section 3.2.2, Eq. 7).  The path goes to the fastest device
 * that can hold all of it (memory below capacity); if none can, it is walked from its
 * source and every vertex goes to the fastest device that still has room.  Every other
 * vertex, in ascending id, goes to the feasible device d that minimises (execution times
 * already on d) + ceil(c_v * scale / s_d) (equal sums: lower index); without a feasible
 * device the same rule runs over all devices and the vertex is counted.
 *   path, len  dev int32 [len] from tfps_critical_path (len = 0: no path)
 *   part       dev uint8 [n]
 *   unplaced   host
 * Synchronises `stream`.  TFPS_ERR_STATE before tfps_devices_set.
 */
int tfps_cp_partition(tfps_graph* g, const int32_t* path, int64_t len, uint8_t* part, int64_t* unplaced, void* stream);

/*
 * Batched list-scheduling simulation (Section 4, criteria (1)-(6); the event-based
 * simulation of Section 5), every candidate on its own.  A device executes its vertices
 * one at a time without interruption; a vertex is executable once every predecessor has
 * finished and its tensor has arrived (finish + transfer time of the evaluation; transfers
 * do not queue); an idle device with an executable vertex starts one at once:
 *   TFPS_SCHED_FIFO  the vertex that became executable first
 *   TFPS_SCHED_PCT   the vertex with the largest path computation time (Section 4.1,
 *                    Eq. 12): prio = the blevel matrix tfps_eval_batch wrote for `part`
 *   TFPS_SCHED_MSR   the vertex with the largest successor rank (Section 4.2, Eq. 13): the
 *                    sum over its out-edges (v->x) of alpha + beta [x on another device]
 *                    + gamma [x has one in-edge] + delta [x has one in-edge and its device
 *                    executes nothing as the deciding step begins]; weights from
 *                    tfps_msr_weights_set (default 1, 1, 1, 5: Section 5.1)
 * equal keys: the smaller vertex id.  At one time T first the executions that end at T are
 * completed, then the idle devices start; both repeat at T while executions of zero length end.
 *   part       dev uint8 [n][ldp]
 *   prio       dev int64 [n][ldp] (PCT) or NULL (FIFO)
 *   start      dev int64 [n][ldp] or NULL; start time of every vertex (the schedule f of
 *              Section 2); padding columns are not written
 *   makespan   dev int64 [P]; time the last vertex ends (-1 for a candidate with an id >= k,
 *              which also raises TFPS_ERR_BAD_PARTITION in the status word)
 * One warp per candidate; scratch of 16 bytes per vertex and candidate in flight is owned
 * by the handle (allocated on first use).  Asynchronous on `stream`.
 */
enum { TFPS_SCHED_FIFO = 0, TFPS_SCHED_PCT = 1, TFPS_SCHED_MSR = 2 };
/* MSR weights alpha, beta, gamma, delta of Eq. 13, each in 0 .. 2^20 (host call, takes effect at the next tfps_simulate) */
int tfps_msr_weights_set(tfps_graph* g, int64_t alpha, int64_t beta, int64_t gamma, int64_t delta);
int tfps_simulate(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int policy, const int64_t* prio,
                  int64_t* start, int64_t* makespan, void* stream);

/* Synchronise `stream`, return the sticky device-side status of the handle and clear it. */
int tfps_get_status(tfps_graph* g, void* stream);

/*
 * Layout helper: src dev uint8 [P][n] (candidate-major) -> dst dev uint8 [n][ldp]
 * (vertex-major).  Padding columns of dst are not written.  Asynchronous.
 */
int tfps_transpose_u8(const uint8_t* src, uint8_t* dst, int64_t P, int64_t n, int64_t ldp, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TFPS_H */
