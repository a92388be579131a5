/*
 * tangram.h -- C ABI of the batched elastic scheduling round (ARL-Tangram, arxiv 2603.13019)
 * for NVIDIA B200 (sm_100a).
 *
 * One call schedules one round for many independent cluster scenarios at once.  Per
 * scenario it does what the paper's scheduler does when it is invoked (Section 4.2):
 *   - evaluates the action-duration model at every allowed allocation level (Eq. 1),
 *   - takes the longest queue prefix whose least-required units fit every pool, chunk
 *     topology included (Algorithm 1, line 2),
 *   - per pool, either takes all candidates at their only level (Algorithm 1, lines 5-6) or
 *     runs the greedy eviction loop (lines 8-14) whose objective is the optimal discrete
 *     allocation of the kept candidates (DPArrange, Algorithm 3, with the GPU chunk
 *     operator of Algorithm 4) plus the completion-heap estimate of everything that keeps
 *     waiting (Algorithm 2),
 *   - places what it selected: aligned power-of-two GPU chunks, smallest sufficient free
 *     chunk first (Section 5.3); exclusive cores, same NUMA domain first (Section 5.2);
 *     quota or concurrency accounting (Section 5.1),
 *   - reports allocation, placement and predicted action completion time (Eq. 2).
 * tangram_replay_trace repeats this round by round over an arrival trace entirely on the
 * device (the workflow of Section 3: submit, queue, schedule, execute, return).
 *
 * All times are integer microseconds.  Every entry point returns 0 or a negative
 * TANGRAM_E* code; data-dependent problems are reported per scenario in `status`, never
 * by a device trap.  Nothing is allocated after tangram_round_create.
 */
#ifndef TANGRAM_H_
#define TANGRAM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* pool types (Section 5: CPU manager, GPU manager, basic manager) */
#define TANGRAM_POOL_CPU 0
#define TANGRAM_POOL_GPU 1
#define TANGRAM_POOL_API 2

/* bit 7 of an action's `unit` byte: on a GPU pool the g*r GPUs of a level are ONE aligned
 * chunk (a service instance of that degree of parallelism, Section 5.3); without it a
 * level is r separate chunks of g GPUs (replicas). */
#define TANGRAM_UNIT_GANG 0x80

#define TANGRAM_MAX_POOLS 8

/* return codes */
#define TANGRAM_OK 0
#define TANGRAM_EINVAL (-1)   /* null pointer, size out of range, bad pool description */
#define TANGRAM_ENOMEM (-2)   /* device allocation failed in tangram_round_create        */
#define TANGRAM_ECUDA (-3)    /* a CUDA runtime call failed; see tangram_last_cuda_error */
#define TANGRAM_ETOOBIG (-4)  /* tangram_schedule_batch_static: the batch needs more scratch than
                                 the built-in array holds                                    */

/* per-scenario status words */
#define TANGRAM_STATUS_OK 0
#define TANGRAM_STATUS_BAD_ACTION 1   /* a record names no pool, has g = 0, no usable level, or
                                         a GPU chunk size that is no power of two <= node size */
#define TANGRAM_STATUS_UNSORTED 2     /* replay: arrivals not non-decreasing                   */
#define TANGRAM_STATUS_WORKSPACE 4    /* a DP or heap did not fit the workspace; the scenario's
                                         outputs are not valid                                 */

typedef struct tangram_round tangram_round; /* opaque; owns only its device workspace */

typedef struct {
  int32_t type;      /* TANGRAM_POOL_*                                                    */
  int32_t capacity;  /* cores | GPUs | tokens per window (or concurrent calls)            */
  int32_t group;     /* CPU: cores per NUMA domain; GPU: GPUs per node (1,2,4,8);
                        capacity must be a multiple of it; API: ignored                    */
  int32_t window_us; /* API: quota period (usage refills at multiples of it); 0 = the limit
                        is on concurrent usage.  Ignored for CPU and GPU pools.            */
} tangram_pool_desc;

typedef struct {
  int32_t n_scenarios;  /* independent cluster scenarios per call, >= 1                    */
  int32_t max_actions;  /* row stride of every per-action array, >= 1                      */
  int32_t n_pools;      /* 1 .. TANGRAM_MAX_POOLS                                          */
  int32_t depth;        /* levels tried for the first waiting action in the estimate
                           (Algorithm 2); the paper evaluates with 2                       */
  int64_t round_us;     /* replay: round period                                            */
  int32_t max_rounds;   /* replay: rounds per call and rows of `occupancy`; 0 if unused    */
  int32_t host_buffers; /* 0: tangram_actions / tangram_result hold DEVICE pointers;
                           1: they hold HOST pointers and every call copies inputs in and
                           results out (large batches in chunks on internal streams so that
                           copies and kernels overlap; ordered after the work queued on the
                           given stream, which in turn waits for the results; use pinned
                           memory)                                                         */
  int64_t workspace_bytes; /* scratch for the rare large tables (reachable-state DP of fragmented GPU
                              pools with gang requests, simulations beyond shared memory);
                              0 = default (2 GiB): 7/8 of it are up to 48 reusable slots of at
                              least 64 MiB (such a table must fit one), the rest is bump-allocated */
  int64_t slot_wait_us;    /* how long a warp that needs one of those slots waits for another warp to
                              give one back before it gives up (the scenario then gets
                              TANGRAM_STATUS_WORKSPACE); 0 = default (100 ms).  The holders of the
                              slots never wait for anything, so a waiter cannot block them.        */
  int32_t cache_slots;     /* service cache of the GPU pools (Section 5.3, evict on execution): service
                              instances every GPU remembers, 0 .. 4; 0 = no cache (then `service`,
                              `restore_us` and the cache arrays of tangram_actions are ignored).
                              Not available with host_buffers = 1.                                 */
  int32_t side_costs;      /* further entries of an action's cost vector (Section 4.1, vectorized resource
                              cost): 0 .. 2; 0 = the key resource only (then `side_pool` / `side_units`
                              of tangram_actions are ignored).  Not available with host_buffers = 1. */
  const tangram_pool_desc* pools; /* host array of n_pools entries, copied                 */
} tangram_round_desc;

/* Pending actions, structure of arrays, scenario-major: element (sc, i) of a per-action
 * array is at [sc * max_actions + i]; the actions of a scenario are in queue (first-come
 * first-served) order.  Caller-owned; read only. */
typedef struct {
  const uint8_t* pool;        /* index of the pool holding the action's key elastic resource */
  const uint8_t* unit;        /* low 7 bits: g, units per multiplicity step; bit 7: GANG      */
  const uint32_t* level_mask; /* bit r-1 set <=> the action may run with g*r units, r = 1..32 */
  const int64_t* s_us;        /* duration model: T(r) = s + floor(p / r); both clamped to     */
  const int64_t* p_us;        /*   [0, 2^40]                                                  */
  const int64_t* arrival_us;  /* may be null (all 0).  Replay needs it, non-decreasing.       */
  const int32_t* n_actions;   /* per scenario, 0 .. max_actions                               */
  const uint8_t* gpu_busy;    /* may be null.  Per scenario, one byte per node of every GPU
                                 pool (pools in index order, row stride = total nodes): bit b
                                 set <=> GPU b of the node is occupied before the round       */
  /* Service cache (only read when cache_slots > 0; Section 5.3).  An action on a GPU pool asks for a
   * service; the instance it needs is (service, chunk size), different degrees of parallelism of a
   * service being distinct instances.  Among the free chunks of the level that the allocation rule
   * picks, one that caches the instance is preferred; an action one of whose chunks does not cache
   * it runs restore_us longer.  Every GPU remembers cache_slots instances, least recently used out. */
  const uint16_t* service;    /* per action, may be null; 0xffff = no service                    */
  const int64_t* restore_us;  /* per action, may be null (0); clamped to [0, 2^40]               */
  uint32_t* gpu_cache_tag;    /* per scenario [node][8][cache_slots], IN and OUT: instance tag
                                 (service * 8 + log2(chunk size)) + 1, 0 = empty entry           */
  int64_t* gpu_cache_use;     /* same shape, IN and OUT: time of the entry's last use             */
  /* Cost vector (only read when side_costs > 0; Section 4.1).  Beside its key resource, which alone is
   * elastic, an action may ask fixed amounts of up to side_costs further pools (memory beside the cores,
   * the quotas of other sites).  Entry e of action (sc, i) is at [(e * n_scenarios + sc) * max_actions + i].
   * Such a pool is a quota / concurrency pool (TANGRAM_POOL_API) other than the key pool and the amount
   * lies in 1 .. its capacity, else the record is bad (TANGRAM_STATUS_BAD_ACTION).  The candidate prefix
   * (Algorithm 1) ends at the first action whose key request at its least level or one of whose amounts
   * does not fit on top of the actions before it; what the candidates ask of a pool this way is set aside
   * before the pool's own actions share it; a started action consumes its amounts (a quota pool counts them
   * in its window, a concurrency pool holds them until the action ends).                                */
  const uint8_t* side_pool;   /* [side_costs][scenario][action], may be null (none); 0xff = no entry     */
  const uint16_t* side_units; /* same shape; ignored where side_pool is 0xff                             */
} tangram_actions;

/* Results, caller-owned, fully overwritten by a call (rows up to max_actions). */
typedef struct {
  int32_t* alloc_units;   /* units granted; 0 = not scheduled                                 */
  int32_t* place_node;    /* GPU: node of the (first) chunk; CPU: NUMA domain of the lowest
                             core; API: 0; -1 if not scheduled                                */
  int32_t* place_off;     /* GPU: first GPU of the (first) chunk within the node; CPU: lowest
                             core id; API: units of the pool consumed before the grant; -1    */
  int64_t* act_us;        /* predicted completion time (queueing so far + execution), -1 if
                             not scheduled; replay: completion - arrival                      */
  int64_t* total_act_us;  /* per scenario: sum of act_us over scheduled actions               */
  int32_t* n_selected;    /* per scenario                                                     */
  int32_t* status;        /* per scenario, TANGRAM_STATUS_* bits                              */
  int32_t* occupancy;     /* replay only, may be null: [scenario][round][pool] units in use
                             after the round's scheduling; zero once the scenario drained     */
  int32_t* rounds_used;   /* replay only, may be null: rounds until drained, else max_rounds  */
} tangram_result;

/* Validates the description, copies it, allocates all device workspace on the current CUDA
 * device.  *out is set only on success. */
int tangram_round_create(const tangram_round_desc* desc, tangram_round** out);

/* One scheduling round at time now_us for every scenario, all pools empty except for
 * `gpu_busy`, nothing executing (Algorithm 1 with an empty executing queue).
 * Asynchronous on `cuda_stream` (a cudaStream_t, may be null for the default stream). */
int tangram_schedule_batch(tangram_round* round, const tangram_actions* actions, int64_t now_us,
                           tangram_result* result, void* cuda_stream);

/* Replays each scenario's arrival trace: rounds at r * round_us, r = 0 .. max_rounds-1; each
 * round releases finished actions, admits arrived ones, schedules as above with the running
 * actions in the completion heap, and starts what was selected.  The whole loop runs on the
 * device.  Asynchronous on `cuda_stream`. */
int tangram_replay_trace(tangram_round* round, const tangram_actions* actions,
                         tangram_result* result, void* cuda_stream);

/* The same round as tangram_schedule_batch for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside another framework's
 * memory pool whose allocator must see every byte on the device, in a latency-critical loop
 * where an allocation's implicit device synchronisation is not acceptable, or in a process
 * whose device memory is fully reserved up front.  Such a caller has no tangram_round: it
 * passes the description, its own DEVICE input and output buffers (host_buffers must be 0)
 * and a stream, and the library calls neither cudaMalloc nor cudaFree nor any other
 * allocating routine.
 *
 * All scratch lives in one array of TANGRAM_STATIC_SCRATCH_BYTES that is part of the library
 * image: every GPU that loads the library holds those bytes until the process exits, whether
 * or not this entry point is ever called.  A batch whose scratch does not fit is refused with
 * TANGRAM_ETOOBIG and nothing is launched: 12 bytes per action of n_scenarios * max_actions,
 * plus (39 + 16 * depth) * max_actions + 324 KiB for each of 8 to 32 worker warps (as many as
 * fit, at least 8), plus at least 4 MiB for large DP tables must fit.  At most 32 worker warps
 * run, so this call is slower on big batches; results are identical.  A scenario whose DP tables outgrow what is left of the
 * array is marked TANGRAM_STATUS_WORKSPACE in `status`, exactly as with a round whose
 * workspace_bytes is too small; the other scenarios of the batch are unaffected.
 *
 * The first call on each device (with that device current) looks up the array's device
 * address and loads two small constant tables; make that first call outside any stream
 * capture, and from one host thread: the look-up is remembered in plain process-wide
 * variables, so two threads making the FIRST call on a device at the same time race on them
 * (later calls only read them).  Every call uses the same array and leaves its contents behind: two calls whose
 * kernels can overlap on the GPU (different streams, or different host threads on one
 * device) race on it and must be serialised by the caller; calls on one stream are safe.
 * Asynchronous on `cuda_stream`. */
#define TANGRAM_STATIC_SCRATCH_BYTES (32u << 20)
int tangram_schedule_batch_static(const tangram_round_desc* desc, const tangram_actions* actions,
                                  int64_t now_us, tangram_result* result, void* cuda_stream);

/* Frees the workspace.  The caller must have synchronised the streams it used. */
void tangram_round_destroy(tangram_round* round);

/* Launches of this library's kernels since the round was created (for accounting). */
int64_t tangram_kernel_launches(const tangram_round* round);

/* Other queue orders (Section 4.2: first come first served is the paper's choice against starvation, and
 * "the algorithm can work with other ordering algorithms").  policy: 1 = shortest duration at the least
 * level first (Eq. 1), 2 = longest first, 3 = earliest arrival first; equal keys keep their queue order; a
 * record that no pool can serve has key 0.
 *
 * tangram_order_queue writes the permutation: perm[sc * max_actions + k] = index of the action that
 * stands at position k of the sorted queue (positions >= n_actions[sc]: k).  perm: device, caller-owned.
 *
 * tangram_schedule_batch_ordered runs one round (as tangram_schedule_batch) on every queue sorted that way;
 * results are written at the actions' own positions.  policy 0 is tangram_schedule_batch itself.  Its first
 * call allocates 54 B per action of device memory that the round keeps (cudaMalloc; TANGRAM_ENOMEM).
 * Device buffers only; max_actions <= 16384 (TANGRAM_ETOOBIG beyond); not with cache_slots / side_costs
 * (TANGRAM_EINVAL).  Asynchronous on the stream. */
#define TANGRAM_ORDER_FCFS 0
#define TANGRAM_ORDER_SHORTEST 1
#define TANGRAM_ORDER_LONGEST 2
#define TANGRAM_ORDER_ARRIVAL 3
int tangram_order_queue(tangram_round* round, const tangram_actions* actions, int policy, int32_t* perm,
                        void* cuda_stream);
/* tangram_replay_trace with the waiting queue kept in the policy's order: an arrival goes behind the last
 * waiting action whose key is not larger than its own, every round runs Algorithm 1 on the queue as it stands.
 * policy 0 and 3 are tangram_replay_trace itself (a trace is sorted by arrival).  The first call with
 * policy 1 or 2 allocates 8 B per action that the round keeps (TANGRAM_ENOMEM). */
int tangram_replay_trace_ordered(tangram_round* round, const tangram_actions* actions, int policy,
                                 tangram_result* result, void* cuda_stream);
int tangram_schedule_batch_ordered(tangram_round* round, const tangram_actions* actions, int policy,
                                   int64_t now_us, tangram_result* result, void* cuda_stream);

/* Per-node CPU scheduling (Section 5.2, pool in CPU manager): every TANGRAM_POOL_CPU pool of the round is one
 * node with a scheduler of its own (Algorithm 1 treats the pools independently).  In queue order, the first
 * action of a trajectory pins it: among the nodes with at least as many cores as the action's least level
 * (g times its smallest multiplicity) and at least traj_mem free memory, the one with the most free memory
 * (lowest pool index on ties) takes it and sets the memory aside; every action of a pinned trajectory gets
 * that node as its pool.  An action whose trajectory finds no node ends the admitted queue: n_admitted is
 * what to pass as n_actions to the round (first come first served: what stands behind it waits).
 * Actions with trajectory < 0 or >= max_trajectories, and actions whose pool is not a CPU pool, keep their
 * pool.  All pointers device memory, caller-owned; traj_node and node_mem_free are state, in and out (the
 * caller gives memory back when a trajectory ends).  Device buffers only.  Asynchronous on the stream. */
typedef struct {
  const int32_t* trajectory;   /* per action [scenario][action]                                          */
  const uint32_t* traj_mem;    /* per action: memory of the action's whole trajectory                    */
  int32_t max_trajectories;    /* row length of traj_node                                                */
  int32_t* traj_node;          /* [scenario][max_trajectories] pool index of the node, -1 = not pinned   */
  int64_t* node_mem_free;      /* [scenario][n_pools] free memory of every CPU pool (other entries unused) */
  uint8_t* pool_out;           /* [scenario][action] the pool column with the trajectories' nodes        */
  int32_t* n_admitted;         /* [scenario]; not used by tangram_replay_trace_pinned (may be null there) */
  const uint8_t* traj_last;    /* per action, may be null; tangram_replay_trace_pinned only: non-zero marks the
                                  last action of its trajectory                                          */
} tangram_pinning;
int tangram_pin_trajectories(tangram_round* round, const tangram_actions* actions, const tangram_pinning* pin,
                             void* cuda_stream);
/* tangram_replay_trace (policy 0 or 3) / tangram_replay_trace_ordered (policy 1, 2) with the trajectories pinned
 * as their actions arrive: in a round, after the releases, every arrival is pinned by the rule above against the
 * memory free at that moment; the first arrival whose trajectory finds no node waits outside the queue, with
 * everything that arrived after it, and is tried again every round.  When an action marked in traj_last ends,
 * its traj_mem goes back to its trajectory's node and the trajectory is no longer pinned.  pool_out (written
 * by the call) is the pool every action ran or waits on; traj_node / node_mem_free hold the final state.
 * Device buffers only. */
int tangram_replay_trace_pinned(tangram_round* round, const tangram_actions* actions, int policy,
                                const tangram_pinning* pin, tangram_result* result, void* cuda_stream);

/* Measurement aid (no counterpart in the paper).  tangram_set_profiling(round, 1) creates CUDA
 * events once; from then on every call records events around each of its kernels on the
 * call's stream (up to 256 calls between two switches).  After the caller has synchronised,
 * tangram_kernel_time_ms sums device time and launches of kernel index `kernel`
 * (0 .. 7, named by tangram_kernel_name; the launches of one kernel within a call are timed
 * as one interval) since profiling was last switched on;
 * tangram_set_profiling(round, 0) destroys the events. */
int tangram_set_profiling(tangram_round* round, int enable);
int tangram_kernel_time_ms(tangram_round* round, int kernel, double* total_ms, int64_t* launches);
const char* tangram_kernel_name(int kernel);

const char* tangram_strerror(int code);
/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* tangram_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TANGRAM_H_ */
