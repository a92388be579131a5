// Host side of the C ABI declared in include/tangram.h, and the per-pool round kernel.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <limits.h>
#include <new>

#include "../../include/tangram.h"
#include "common.cuh"
#include "prefix_kernel.cuh"
#include "prefix_stream.cuh"
#include "order_pin.cuh"
#include "sims.cuh"
#include "select.cuh"
#include "place.cuh"

#define K2_THREADS 256
#define TG_PROF_CALLS 256   // calls whose kernels can be timed between two queries
#define TG_N_SIM_CLASSES 22
#define TG_FILL_BLOCKS_PER_SM 4   // k_fill is a trickle beside the other kernels, not a flood
#define TG_IO_CHUNKS 16
#define TG_PROF_K 6         // timed intervals per call at most
#define TG_N_KERNELS 8

// ---------------------------------------------------------------------------------------
// Per-(scenario, pool) work of a round, one warp per task.  The pieces are shared by
//   k_select            everything in one kernel (general path: any number of evictions,
//                       running actions in the heap; used by the allocation-free entry point),
//   k_solve / k_finish  the batched path: k_solve computes the optimal allocations of the full
//                       candidate list and of the list without its last candidate; a pool
//                       without elastic candidates, or whose first eviction step cannot pay
//                       (eviction_cannot_pay), is placed and written at once.  For the others
//                       k_sims (sims.cuh) runs the completion-heap simulations one thread
//                       each, and k_finish compares the two objectives (Algorithm 1, lines
//                       8-14), goes on evicting where the first eviction pays, places the
//                       grants and writes the candidates' outputs (Eq. 2).
// ---------------------------------------------------------------------------------------
// Tasks are handed out by a counter so that long tasks do not pile up on the same warps.
__device__ __forceinline__ int next_task(u64* counter, int lane) {
  u64 x = 0;
  if (lane == 0) x = atomicAdd(counter, 1ull);
  return (int)__shfl_sync(TG_FULL, x, 0);
}

struct CandArrays {
  i64* cs; i64* cp; u32* cmask; int* cidx; int* pnode; int* poff; int* rowcand;
  u8* cg; u8* rsel; u8* rkeep;
};

__device__ bool gather_candidates(const Params& P, int sc, int j, const PoolMeta& mt, Slab& slab, int lane,
                                  CandArrays& C) {
  const int m = mt.m;
  const PoolDev& pd = P.pool[j];
  const size_t row = (size_t)sc * P.N;
  // what the sequential loops read over and over goes to the warp's shared-memory window while
  // it lasts (most wanted first), the rest to the warp's slab in global memory
  C.cg = (u8*)slab.take_fast(m);
  C.rkeep = (u8*)slab.take_fast(m);
  C.rsel = (u8*)slab.take_fast(m);
  C.cmask = (u32*)slab.take_fast((u64)m * 4);
  C.rowcand = (int*)slab.take_fast((u64)m * 4);
  C.cp = (i64*)slab.take_fast((u64)m * 8);
  C.cs = (i64*)slab.take_fast((u64)m * 8);
  C.cidx = (int*)slab.take((u64)m * 4);
  C.pnode = (int*)slab.take((u64)m * 4);
  C.poff = (int*)slab.take((u64)m * 4);
  if (!C.cg || !C.rkeep || !C.rsel || !C.cmask || !C.rowcand || !C.cp || !C.cs || !C.cidx || !C.pnode || !C.poff) return false;
  // four candidates per lane at a time: first all their indices, then all their records, so that a
  // pool of up to 128 candidates costs two rounds of loads instead of two per 32 candidates
  for (int i0 = lane; i0 < m; i0 += 128) {
    int idx[4]; u8 un[4]; u32 mk[4]; i64 sv[4], pv[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) idx[x] = i0 + 32 * x < m ? P.order[row + mt.cbase + i0 + 32 * x] : 0;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const bool on = i0 + 32 * x < m;
      un[x] = on ? P.a_unit[row + idx[x]] : 1; mk[x] = on ? P.a_mask[row + idx[x]] : 1;
      sv[x] = on ? P.a_s[row + idx[x]] : 0; pv[x] = on ? P.a_p[row + idx[x]] : 0;
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const int i = i0 + 32 * x;
      if (i >= m) break;
      int g, gang; u32 eff;
      decode_levels(pd, un[x], mk[x], g, gang, eff);
      C.cidx[i] = idx[x]; C.cmask[i] = eff; C.cg[i] = (u8)(g | (gang << 7));
      C.cs[i] = clamp_param(sv[x]); C.cp[i] = clamp_param(pv[x]);
      C.rkeep[i] = (u8)__ffs(eff);
      C.pnode[i] = -1; C.poff[i] = -1;
    }
  }
  __syncwarp();
  return true;
}

// with_waiting = false leaves out the pool's waiting actions (k_solve estimates nothing itself).
__device__ void make_task(const Params& P, int sc, int j, const PoolMeta& mt, const CandArrays& C, int lane,
                          PoolTask& T, bool with_waiting = true) {
  const PoolDev& pd = P.pool[j];
  const size_t row = (size_t)sc * P.N;
  const u8* busy_row = P.gpu_busy ? P.gpu_busy + (size_t)sc * P.n_nodes_total : nullptr;
  T.type = pd.type; T.group = pd.group;
  T.cap[0] = pd.capacity; T.cap[1] = T.cap[2] = T.cap[3] = 0;
  if (pd.type == TG_POOL_GPU) gpu_caps(pd, busy_row, lane, T.cap);
  if (P.n_side > 0 && pd.type == TG_POOL_API) T.cap[0] -= P.side_res[(size_t)sc * P.P + j];   // set aside for the other pools' candidates
  T.m = mt.m; T.cs = C.cs; T.cp = C.cp; T.cmask = C.cmask; T.cg = C.cg;
  T.n_ac = with_waiting ? mt.count - mt.m : 0;
  T.ac_tmin = P.tmin + row + mt.base + mt.m;
  T.ac_first.s = T.ac_first.p = 0; T.ac_first.mask = 1; T.ac_first.g = 1; T.ac_first.gang = 0;
  if (T.n_ac > 0) {
    int idx = mt.first_wait;
    decode_levels(pd, P.a_unit[row + idx], P.a_mask[row + idx], T.ac_first.g, T.ac_first.gang, T.ac_first.mask);
    T.ac_first.s = clamp_param(P.a_s[row + idx]); T.ac_first.p = clamp_param(P.a_p[row + idx]);
  }
  T.seeds = nullptr; T.n_seeds = 0;
  T.depth = P.depth;
  T.rsel = C.rsel; T.rkeep = C.rkeep; T.rowcand = C.rowcand;
  T.sim_base = 0; T.sim_cap = 0;
}

// shared memory of the calling warp for winner trees inside the per-pool kernels
#define WARP_TREE_SLOTS 448
#define WARP_TREE_BYTES (WARP_TREE_SLOTS * 16)
#define WARP_FAST_BYTES 2048
#define WARP_SMEM_BYTES (WARP_TREE_BYTES + WARP_FAST_BYTES)
#define K2_DYN_SMEM ((K2_THREADS / 32) * WARP_SMEM_BYTES + 16)
__device__ __forceinline__ void attach_warp_tree(PoolTask& T) {
  extern __shared__ __align__(16) unsigned char k2_smem[];
  const u32 start = ((u32)__cvta_generic_to_shared(k2_smem) + 15u) & ~15u;
  T.sim_base = start + (threadIdx.x >> 5) * WARP_SMEM_BYTES;
  T.sim_cap = WARP_TREE_SLOTS;
}
// the calling warp's scratch: shared-memory window behind its tree area, then its global slab
__device__ __forceinline__ Slab warp_slab(const Params& P, int gw) {
  extern __shared__ __align__(16) unsigned char k2_smem[];
  Slab s;
  s.base = P.slabs + (u64)gw * P.slab_bytes; s.cap = P.slab_bytes; s.used = 0;
  const u64 start = ((u64)k2_smem + 15u) & ~(u64)15;
  s.fbase = (char*)start + (threadIdx.x >> 5) * WARP_SMEM_BYTES + WARP_TREE_BYTES;
  s.fcap = WARP_FAST_BYTES; s.fused = 0;
  return s;
}

// placement on a fresh copy of the pool's topology state, then the candidates' outputs
__device__ void place_and_write(const Params& P, int sc, int j, const PoolMeta& mt, const CandArrays& C,
                                int keep, Slab slab, int lane, bool defer = false) {
  const int m = mt.m;
  const PoolDev& pd = P.pool[j];
  const size_t row = (size_t)sc * P.N;
  const u8* busy_row = P.gpu_busy ? P.gpu_busy + (size_t)sc * P.n_nodes_total : nullptr;
  const u8* missed = nullptr;                            // candidates whose chunk did not cache their service
  defer = defer && pd.lane_place;
  if (defer) {
    // k_place will place this pool: leave it the kept requests in queue order
    unsigned short* rq = P.preq + row + mt.cbase;
    for (int i = lane; i < keep; i += 32) rq[i] = (unsigned short)(C.cg[i] | ((u32)C.rkeep[i] << 8));
    if (lane == 0) P.keepn[(size_t)sc * P.P + j] = keep;
  } else if (pd.type == TG_POOL_GPU && P.cache_slots > 0) {
    // with a service cache: the chunk that caches the instance first, entries updated, misses noted in C.rsel
    u8* nm = (u8*)slab.take_fast(pd.n_nodes);
    if (!nm) { if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); keep = 0; }
    else {
      for (int v = lane; v < pd.n_nodes; v += 32) nm[v] = busy_row ? busy_row[pd.node0 + v] : 0;
      __syncwarp();
      const size_t cbase = ((size_t)sc * P.n_nodes_total + pd.node0) * 8 * P.cache_slots;
      place_gpu_cache(pd, nm, keep, C.cg, C.rkeep, C.cidx, C.pnode, C.poff, C.rsel,
                      P.a_service ? P.a_service + row : nullptr, P.cache_tag + cbase, P.cache_use + cbase,
                      P.cache_slots, P.now, lane);
      missed = C.rsel;
    }
  } else if (pd.type == TG_POOL_GPU) {
    if (pd.n_nodes <= 128) place_gpu_reg(pd, busy_row ? busy_row + pd.node0 : nullptr, keep, C.cg, C.rkeep, C.pnode, C.poff, lane);
    else {
    u8* nm = (u8*)slab.take_fast(pd.n_nodes);
    if (!nm) { if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); keep = 0; }
    else {
      for (int v = lane; v < pd.n_nodes; v += 32) nm[v] = busy_row ? busy_row[pd.node0 + v] : 0;
      __syncwarp();
      place_gpu(pd, nm, keep, C.cg, C.rkeep, C.pnode, C.poff, lane);
    }
    }
  } else if (pd.type == TG_POOL_CPU && pd.capacity / pd.group <= 128 && pd.group < 65536) {
    place_cpu_fresh_reg(pd, keep, C.cg, C.rkeep, C.pnode, C.poff, lane);
  } else if (pd.type == TG_POOL_CPU) {
    const int D = pd.capacity / pd.group;
    int* dfree = (int*)slab.take_fast((u64)D * 4);
    if (!dfree) { if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); keep = 0; }
    else place_cpu_fresh(pd, dfree, keep, C.cg, C.rkeep, C.pnode, C.poff, lane);
  } else {
    if (lane == 0) {
      int used = 0;
      for (int i = 0; i < keep; ++i) { C.pnode[i] = 0; C.poff[i] = used; used += (C.cg[i] & 0x7f) * C.rkeep[i]; }
    }
    __syncwarp();
  }

  __syncwarp();
  i64 tot = 0; int cnt = 0;
  for (int i = lane; i < m; i += 32) {
    const size_t o = row + C.cidx[i];
    if (i < keep) {
      int r = C.rkeep[i];
      i64 arr = P.a_arrival ? P.a_arrival[o] : 0;
      i64 act = (P.now - arr) + duration(C.cs[i], C.cp[i], r);
      if (missed && missed[i] && P.a_restore) act += clamp_param(P.a_restore[o]);   // restoration precedes execution
      P.o_alloc[o] = (C.cg[i] & 0x7f) * r; P.o_act[o] = act;
      if (!defer) { P.o_node[o] = C.pnode[i]; P.o_off[o] = C.poff[i]; }
      tot += act; ++cnt;
    } else {
      P.o_alloc[o] = 0; P.o_node[o] = -1; P.o_off[o] = -1; P.o_act[o] = -1;
    }
  }
  tot = warp_sum64(tot); cnt = warp_sum32(cnt);
  if (lane == 0 && cnt) {
    atomicAdd((u64*)&P.o_total[sc], (u64)tot);
    atomicAdd(&P.o_nsel[sc], cnt);
  }
}

__device__ void run_pool_task(const Params& P, int sc, int j, Slab slab, int lane) {
  const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
  if (mt.m == 0) return;
  CandArrays C;
  if (!gather_candidates(P, sc, j, mt, slab, lane, C)) {
    if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE);
    return;
  }
  int keep = mt.m;
  if (mt.elastic) {
    PoolTask T;
    make_task(P, sc, j, mt, C, lane, T);
    attach_warp_tree(T);
    keep = evict_loop(P, T, slab, lane);
    if (keep < 0) { if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); keep = 0; }
  }
  place_and_write(P, sc, j, mt, C, keep, slab, lane);
}

__global__ void __launch_bounds__(K2_THREADS) k_select(const __grid_constant__ Params P) {
  const int lane = threadIdx.x & 31;
  const int gw = (blockIdx.x * K2_THREADS + threadIdx.x) >> 5;
  const Slab slab = warp_slab(P, gw);
  const int n_tasks = P.S * P.P;
  for (;;) {
    const int x = next_task(P.arena_top + 3, lane);
    if (x >= n_tasks) break;
    run_pool_task(P, x % P.S, P.pool_order[x / P.S], slab, lane);   // pool-major, heaviest pools first
  }
}

// The pools that the head kernel certified (no elastic candidate, or every candidate's largest level
// fits: then each takes the smallest level that reaches its lowest duration and no eviction can
// pay) need no selection at all.  One warp per such (scenario, pool), nothing but registers: the
// candidates' allocations and predicted completion times (Eq. 2) are written, their requests are
// left for the placement kernel.  Runs beside the streaming kernel, on a stream of its own.
__global__ void __launch_bounds__(256) k_easy(const __grid_constant__ Params P, const HeadState* hst) {
  const int lane = threadIdx.x & 31;
  const long long x = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (x >= (long long)P.S * P.P) return;
  const int sc = (int)(x % P.S), j = P.pool_order[x / P.S], task = sc * P.P + j;
  const PoolDev& pd = P.pool[j];
  if (((hst[sc].need >> j) & 1u) || !pd.lane_place) return;
  const PoolMeta mt = P.meta[task];
  const int m = mt.m;
  if (lane == 0) P.keepn[task] = m;
  if (m == 0) return;
  const size_t row = (size_t)sc * P.N;
  const int* ord = P.order + row + mt.cbase;
  unsigned short* rq = P.preq + row + mt.cbase;
  i64 tot = 0; int cnt = 0;
  for (int i = lane; i < m; i += 32) {
    const size_t o = row + ord[i];
    int g, gang; u32 eff;
    decode_levels(pd, P.a_unit[o], P.a_mask[o], g, gang, eff);
    const i64 s = clamp_param(P.a_s[o]), p = clamp_param(P.a_p[o]);
    const int r = best_level(p, eff);
    const i64 act = (P.now - (P.a_arrival ? P.a_arrival[o] : 0)) + duration(s, p, r);
    P.o_alloc[o] = g * r; P.o_act[o] = act;
    rq[i] = (unsigned short)((u32)g | ((u32)gang << 7) | ((u32)r << 8));
    tot += act; ++cnt;
  }
  tot = warp_sum64(tot); cnt = warp_sum32(cnt);
  if (lane == 0) {
    atomicAdd((u64*)&P.o_total[sc], (u64)tot);
    atomicAdd(&P.o_nsel[sc], cnt);
  }
}

// workspace of the batched path, indexed like the partitioned arrays
struct BatchWs {
  TaskState* ts;   // [S][P]
  i64* seed2;      // [S][cand_stride] durations of the first m-1 candidates under their optimal allocation
  u8* rs1;         // [S][cand_stride] multiplicities of the optimal allocation of all m candidates
  u8* rs2;         // [S][cand_stride] ... of the first m-1
};

__global__ void __launch_bounds__(K2_THREADS, 3) k_solve(const __grid_constant__ Params P, const BatchWs W, const HeadState* hst) {
  const int lane = threadIdx.x & 31;
  const int gw = (blockIdx.x * K2_THREADS + threadIdx.x) >> 5;
  const int n_tasks = P.S * P.P;
  for (;;) {
    const int x = next_task(P.arena_top + 1, lane);
    if (x >= n_tasks) break;
    const int sc = x % P.S, j = P.pool_order[x / P.S], task = sc * P.P + j;
    TaskState* st = W.ts + task;
    if (!((hst[sc].need >> j) & 1u) && P.pool[j].lane_place) {   // certified by the head kernel: k_easy has it
      if (lane == 0) st->flags = TS_DECIDED;
      continue;
    }
    const PoolMeta mt = P.meta[task];
    if (lane == 0) P.keepn[task] = -1;                   // nothing for k_place unless a decision says so
    if (mt.m == 0) { if (lane == 0) st->flags = TS_DECIDED; continue; }
    Slab slab = warp_slab(P, gw);
    CandArrays C;
    if (!gather_candidates(P, sc, j, mt, slab, lane, C)) {
      if (lane == 0) { atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); st->flags = TS_DECIDED; }
      continue;
    }
    // A pool is decided here unless its first eviction step needs the two estimates.
    int keep = mt.m;
    bool decided = true;
    if (mt.elastic) {
      PoolTask T;
      make_task(P, sc, j, mt, C, lane, T, false);
      attach_warp_tree(T);                               // scratch of the small-box DP
      i64 opt0 = 0, opt1 = 0;
      bool all_best;
      bool ok = solve_prefix(P, T, mt.m, slab, lane, &opt0, &all_best);
      if (ok) {
        for (int i = lane; i < mt.m; i += 32) C.rkeep[i] = C.rsel[i];
        __syncwarp();
        if (mt.m >= 2 && !all_best) {                      // all at their best level: eviction_cannot_pay holds
          ok = solve_prefix(P, T, mt.m - 1, slab, lane, &opt1);
          if (ok && !eviction_cannot_pay(T, mt.m - 1, C.rkeep, C.rsel, lane)) {
            decided = false;
            const size_t pos = (size_t)sc * P.N + mt.base, cpos = (size_t)sc * P.N + mt.cbase;
            for (int i = lane; i < mt.m; i += 32) {
              W.rs1[cpos + i] = C.rkeep[i];
              P.tmin[pos + i] = duration(C.cs[i], C.cp[i], C.rkeep[i]);   // heap seeds of the full list
              if (i < mt.m - 1) {
                W.rs2[cpos + i] = C.rsel[i];
                W.seed2[cpos + i] = duration(C.cs[i], C.cp[i], C.rsel[i]);
              }
            }
            if (lane == 0) {
              st->opt[0] = opt0; st->opt[1] = opt1;
              st->est[0] = 0;                              // stays if nothing waits behind the candidates
              st->est[1] = TG_INF;
              st->flags = TS_SOLVED;
            }
          }
        }
      }
      if (!ok) { if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); keep = 0; }
    }
    if (decided) {
      place_and_write(P, sc, j, mt, C, keep, slab, lane, true);
      if (lane == 0) st->flags = TS_DECIDED;
    }
  }
}

// One pool whose first eviction step had to be estimated: compare the two objectives, go on
// evicting where the first eviction pays, hand the result to the placement.
__device__ void finish_task(const Params& P, const BatchWs& W, int x, int gw, int lane) {
  const int sc = x % P.S, j = P.pool_order[x / P.S], task = sc * P.P + j;
  const TaskState st = W.ts[task];
  const PoolMeta mt = P.meta[task];
  Slab slab = warp_slab(P, gw);
  CandArrays C;
  if (!gather_candidates(P, sc, j, mt, slab, lane, C)) {
    if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE);
    return;
  }
  int keep = mt.m;
  if (!(st.flags & TS_SOLVED) || (st.flags & TS_FAILED)) keep = -1;
  else {
    const size_t pos = (size_t)sc * P.N + mt.cbase;
    i64 obj = sat_add(st.opt[0], st.est[0]);
    for (int i = lane; i < mt.m; i += 32) C.rkeep[i] = W.rs1[pos + i];
    i64 nobj = sat_add(st.opt[1], st.est[1]);
    if (nobj < obj) {                                    // the first eviction pays: go on
      for (int i = lane; i < mt.m - 1; i += 32) C.rkeep[i] = W.rs2[pos + i];
      __syncwarp();
      PoolTask T;
      make_task(P, sc, j, mt, C, lane, T);
      attach_warp_tree(T);
      keep = evict_resume(P, T, slab, lane, nobj, mt.m - 1);
    }
    __syncwarp();
  }
  if (keep < 0) { if (lane == 0) atomicOr(&P.o_status[sc], TG_ST_WORKSPACE); keep = 0; }
  place_and_write(P, sc, j, mt, C, keep, slab, lane, true);
}

// Work list of k_finish: the pools that k_solve left undecided, those that go on evicting first.
// Each of the latter is a chain of dependent DPs and simulations, so they must start as early
// as possible.  fl: [0] number of chain tasks, [1] number of other tasks, then the chain tasks
// from the front and the others from the back of an array of S * P entries.
__global__ void k_finish_list(const __grid_constant__ Params P, const BatchWs W, int* fl) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x, lane = threadIdx.x & 31;
  const int n_tasks = P.S * P.P;
  int kind = -1;                                          // 0 chain, 1 other
  if (x < n_tasks) {
    const int sc = x % P.S, j = P.pool_order[x / P.S];
    const TaskState* st = W.ts + (size_t)sc * P.P + j;
    const int flags = st->flags;
    if (!(flags & TS_DECIDED))
      kind = ((flags & TS_SOLVED) && !(flags & TS_FAILED) &&
              sat_add(st->opt[1], st->est[1]) < sat_add(st->opt[0], st->est[0])) ? 0 : 1;
  }
  for (int k = 0; k < 2; ++k) {
    const u32 b = __ballot_sync(TG_FULL, kind == k);
    if (!b) continue;
    int at = 0;
    if (lane == __ffs(b) - 1) at = atomicAdd(&fl[k], __popc(b));
    at = __shfl_sync(TG_FULL, at, __ffs(b) - 1) + __popc(b & ((1u << lane) - 1u));
    if (kind == k) fl[2 + (k == 0 ? at : n_tasks - 1 - at)] = x;
  }
}

__global__ void __launch_bounds__(K2_THREADS) k_finish(const __grid_constant__ Params P, const BatchWs W, const int* fl) {
  const int lane = threadIdx.x & 31;
  const int gw = (blockIdx.x * K2_THREADS + threadIdx.x) >> 5;
  const int n_tasks = P.S * P.P, n_chain = fl[0], n_all = fl[0] + fl[1];
  for (;;) {
    const int y = next_task(P.arena_top + 2, lane);
    if (y >= n_all) break;
    finish_task(P, W, fl[2 + (y < n_chain ? y : n_tasks - 1 - (y - n_chain))], gw, lane);
  }
}

#include "place_lane.cuh"
#include "replay.cuh"

// ---------------------------------------------------------------------------------------
// host
// ---------------------------------------------------------------------------------------
static thread_local char g_cuda_err[256] = "";

static int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
  return TANGRAM_ECUDA;
}
#define CK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail(e_, #call); } while (0)

struct tangram_round {
  tangram_round_desc desc;
  tangram_pool_desc pools[TANGRAM_MAX_POOLS];
  Params P;                 // template: pools, sizes, workspace pointers
  int device;
  int64_t launches;
  // workspace
  void* d_order; void* d_tmin; void* d_meta; void* d_slabs; void* d_arena; void* d_arena_top;
  HeadState* hst; void* d_preq; void* d_keepn; int* d_fl; u32* d_ok_table; int* d_side_bad; int* d_side_res;
  BatchWs W; int sim_blocks; SimLists L; int n_sm;
  ReplayWs R;
  // host-buffer mode: copy-in, kernels and copy-out of successive chunks on streams of their own
  cudaStream_t io_in, io_comp, io_out;
  cudaEvent_t io_begin, io_end, io_in_done[TG_IO_CHUNKS], io_comp_done[TG_IO_CHUNKS];
  // the capacity classes of k_sims are independent: they run on side streams between a fork
  // and a join event so that their partial waves overlap
  cudaStream_t sim_stream[TG_N_SIM_CLASSES + 1];
  cudaEvent_t sim_fork, sim_join[TG_N_SIM_CLASSES + 1];
  // the certified pools (k_easy and their placement) run beside the kernels that follow k_solve
  cudaStream_t side; cudaEvent_t side_fork, side_join;
  // sorted copy of the queue and of its results (tangram_schedule_batch_ordered), allocated at its first call
  char* d_sorted; int* d_perm; u64* d_wkey;
  // staging for host-buffer mode
  char* d_stage; size_t stage_bytes;
  size_t in_off[8], out_off[9];
  // optional per-kernel timing: events recorded around every kernel of a call
  cudaEvent_t* ev; int ev_calls, ev_used; int ev_kernel[TG_PROF_CALLS][TG_PROF_K];
};

static const char* const g_kernel_names[TG_N_KERNELS] = {"k_head", "k_select", "k_replay", "k_solve",
                                                          "k_sims", "k_finish", "k_place", "k_stream"};
// capacity classes (slots per simulation) of the shared-memory simulation kernels
static const int g_sim_caps[TG_N_SIM_CLASSES] = {16, 32, 48, 64, 80, 96, 112, 128, 144, 160, 176, 192, 224, 256,
                                                 320, 384, 448, 512, 576, 608, 640, 672};
#define TG_SMEM_PER_SM 233472   // shared memory an SM can split among resident blocks
#define TG_SMEM_PER_BLOCK 232448

typedef void (*sims_fn)(const Params, TaskState*, const i64*, const SimLists, int);
// levels below the root of the 4-ary tree of a capacity class
static int sim_levels(int cap) {
  long long nodes = tree_nodes(cap), reach = 1, width = 1;
  int d = 0;
  while (reach < nodes) { width *= 4; reach += width; ++d; }
  return d;
}
static sims_fn sim_kernel(int cap) {
  switch (sim_levels(cap)) {
    case 0: case 1: case 2: return k_sims1<2>;
    case 3: return k_sims1<3>;
    case 4: return k_sims1<4>;
    default: return k_sims1<5>;
  }
}
// shared memory of a block (32 trees interleaved by lane) of a capacity class
static int sim_smem_bytes(int cap) { return tree_nodes(cap) * 8 * SIM_PER_WARP; }

static cudaError_t fill_tables() {
  u64 recip[33];
  recip[0] = recip[1] = 0;
  // ceil(2^64 / r) = floor((2^64 - 1) / r) + 1 for every r >= 2
  for (int r = 2; r <= 32; ++r) recip[r] = 0xffffffffffffffffull / (u64)r + 1ull;
  u32 fb[256];
  for (int b = 0; b < 256; ++b) {
    int F[4] = {0, 0, 0, 0};
    // maximal free aligned blocks of an 8-GPU node with busy mask b
    if (b == 0) F[3] = 1;
    else
      for (int h = 0; h < 8; h += 4) {
        if (((b >> h) & 0xf) == 0) { F[2]++; continue; }
        for (int q = h; q < h + 4; q += 2) {
          if (((b >> q) & 0x3) == 0) { F[1]++; continue; }
          for (int s = q; s < q + 2; ++s) if (!((b >> s) & 1)) F[0]++;
        }
      }
    fb[b] = (u32)F[0] | ((u32)F[1] << 8) | ((u32)F[2] << 16) | ((u32)F[3] << 24);
  }
  cudaError_t e = cudaMemcpyToSymbol(c_recip, recip, sizeof(recip));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(c_fblocks, fb, sizeof(fb));
  return e;
}

extern "C" const char* tangram_strerror(int code) {
  switch (code) {
    case TANGRAM_OK: return "ok";
    case TANGRAM_EINVAL: return "invalid argument";
    case TANGRAM_ENOMEM: return "out of device memory";
    case TANGRAM_ECUDA: return "CUDA runtime error";
    case TANGRAM_ETOOBIG: return "problem too large for the static scratch array";
    default: return "unknown error";
  }
}

extern "C" const char* tangram_last_cuda_error(void) { return g_cuda_err; }

extern "C" int64_t tangram_kernel_launches(const tangram_round* r) { return r ? r->launches : 0; }

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// GPU pools first (their tasks may go on evicting), then CPU pools, then API pools
static void fill_pool_order(Params& P) {
  int k = 0;
  const int rank[3] = {TG_POOL_GPU, TG_POOL_CPU, TG_POOL_API};
  for (int r = 0; r < 3; ++r)
    for (int j = 0; j < P.P; ++j)
      if (P.pool[j].type == rank[r]) P.pool_order[k++] = j;
}

// pools that k_place can take: its per-thread state is a few hundred bytes of shared memory
static int lane_place_ok(const PoolDev& d) {
  if (d.type == TG_POOL_API) return 1;
  if (d.type == TG_POOL_CPU) return d.capacity / d.group <= KPL_DOMAINS && d.group <= 255;
  return d.n_nodes <= 64;
}

extern "C" int tangram_round_create(const tangram_round_desc* desc, tangram_round** out) {
  if (!desc || !out || !desc->pools) return TANGRAM_EINVAL;
  if (desc->n_scenarios < 1 || desc->max_actions < 1 || desc->n_pools < 1 ||
      desc->n_pools > TANGRAM_MAX_POOLS || desc->depth < 1 || desc->depth > 32 || desc->max_rounds < 0 ||
      desc->round_us < 0 || desc->workspace_bytes < 0 || desc->slot_wait_us < 0 || desc->cache_slots < 0 ||
      desc->cache_slots > 4 || (desc->cache_slots > 0 && desc->host_buffers) || desc->side_costs < 0 ||
      desc->side_costs > 2 || (desc->side_costs > 0 && desc->host_buffers))
    return TANGRAM_EINVAL;
  if ((int64_t)desc->n_scenarios * desc->max_actions > (int64_t)1 << 31) return TANGRAM_EINVAL;
  tangram_round* r = new (std::nothrow) tangram_round();
  if (!r) return TANGRAM_ENOMEM;
  memset(r, 0, sizeof(*r));
  r->desc = *desc;
  Params& P = r->P;
  P.S = desc->n_scenarios; P.N = desc->max_actions; P.P = desc->n_pools; P.depth = desc->depth;
  P.cache_slots = desc->cache_slots;
  int node0 = 0, slot0 = 0;
  for (int j = 0; j < desc->n_pools; ++j) {
    const tangram_pool_desc& pd = desc->pools[j];
    r->pools[j] = pd;
    bool ok = pd.capacity >= 1 && pd.capacity <= (1 << 20) && pd.window_us >= 0;
    if (pd.type == TANGRAM_POOL_GPU)
      ok = ok && (pd.group == 1 || pd.group == 2 || pd.group == 4 || pd.group == 8) && pd.capacity % pd.group == 0;
    else if (pd.type == TANGRAM_POOL_CPU) ok = ok && pd.group >= 1 && pd.capacity % pd.group == 0;
    else if (pd.type != TANGRAM_POOL_API) ok = false;
    if (!ok) { delete r; return TANGRAM_EINVAL; }
    PoolDev& d = P.pool[j];
    d.type = pd.type; d.capacity = pd.capacity; d.group = pd.type == TANGRAM_POOL_API ? 1 : pd.group;
    d.window_us = pd.type == TANGRAM_POOL_API ? pd.window_us : 0;
    d.node0 = node0; d.n_nodes = pd.type == TANGRAM_POOL_GPU ? pd.capacity / pd.group : 0;
    node0 += d.n_nodes;
    d.slot0 = slot0; d.n_slots = pd.type == TANGRAM_POOL_GPU ? 4 : 1;
    slot0 += d.n_slots;
    d.lane_place = lane_place_ok(d);
    if (desc->cache_slots > 0 && pd.type == TANGRAM_POOL_GPU) d.lane_place = 0;   // placed by the warp that decides the pool
  }
  r->desc.pools = r->pools;
  P.n_nodes_total = node0;
  P.V = slot0 + desc->n_pools;
  fill_pool_order(P);
  P.cand_off[0] = 0;
  for (int j = 0; j < desc->n_pools; ++j)
    P.cand_off[j + 1] = P.cand_off[j] + (int)align_up((size_t)(P.pool[j].capacity < P.N ? P.pool[j].capacity : P.N), 8);
  P.cand_stride = P.cand_off[desc->n_pools];

  cudaError_t e = cudaGetDevice(&r->device);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, r->device);
  if (e == cudaSuccess) e = fill_tables();
  if (e != cudaSuccess) { delete r; return cuda_fail(e, "device set-up"); }

  const size_t SN = (size_t)P.S * P.N, SC = (size_t)P.S * P.cand_stride;
  P.n_workers = prop.multiProcessorCount * 3 * (K2_THREADS / 32);   // what k_solve keeps resident
  if ((int64_t)P.n_workers > (int64_t)P.S * P.P) P.n_workers = (int)align_up((size_t)P.S * P.P, K2_THREADS / 32);
  // every worker warp owns a slab that holds the candidate arrays, heaps and small DP tables of
  // the pool it is working on; larger DP tables come from the shared arena
  size_t per_cand = 8 + 8 + 4 + 4 + 4 + 4 + 4 + 3 + 16 * (size_t)desc->depth;
  size_t slab = align_up((size_t)P.N * per_cand + 64 * 1024 + (1 << 20) / 4 + 4096, 256);
  P.slab_bytes = slab;
  P.arena_bytes = desc->workspace_bytes ? (u64)desc->workspace_bytes : (2ull << 30);
  {
    const int64_t us = desc->slot_wait_us ? desc->slot_wait_us : 100000;
    P.slot_tries = (int)(us / 2 > 0x3fffffff ? 0x3fffffff : (us / 2 < 1 ? 1 : us / 2));
  }
  bool bad = false;
  bad |= cudaMalloc(&r->d_order, SC * sizeof(int)) != cudaSuccess;
  bad |= cudaMalloc(&r->d_tmin, SN * sizeof(i64) * P.P) != cudaSuccess;
  bad |= cudaMalloc(&r->d_meta, (size_t)P.S * P.P * sizeof(PoolMeta)) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->hst, (size_t)P.S * sizeof(HeadState)) != cudaSuccess;
  bad |= cudaMalloc(&r->d_slabs, (size_t)P.n_workers * slab) != cudaSuccess;
  bad |= cudaMalloc(&r->d_arena, P.arena_bytes) != cudaSuccess;
  bad |= cudaMalloc(&r->d_arena_top, 256) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->W.ts, (size_t)P.S * P.P * sizeof(TaskState)) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->W.seed2, SC * sizeof(i64)) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->W.rs1, SC) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->W.rs2, SC) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->d_preq, SC * sizeof(unsigned short)) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->d_keepn, (size_t)P.S * P.P * sizeof(int)) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->d_fl, ((size_t)P.S * P.P + 2) * sizeof(int)) != cudaSuccess;
  if (desc->side_costs > 0) {                              // cost vectors: flags and set-aside amounts
    bad |= cudaMalloc((void**)&r->d_side_bad, (size_t)P.S * sizeof(int)) != cudaSuccess;
    bad |= cudaMalloc((void**)&r->d_side_res, (size_t)P.S * P.P * sizeof(int)) != cudaSuccess;
  }
  const long long n_sims = (long long)P.P * P.S * 2;
  r->sim_blocks = (int)((n_sims + 31) / 32);
  r->n_sm = prop.multiProcessorCount;
  r->L.n_groups = (int)((n_sims + SIM_PER_WARP - 1) / SIM_PER_WARP);
  r->L.n_classes = TG_N_SIM_CLASSES;
  for (int c = 0; c < TG_N_SIM_CLASSES; ++c) r->L.cap[c] = g_sim_caps[c];
  bad |= cudaMalloc((void**)&r->L.count, 2 * 64 * sizeof(int)) != cudaSuccess;
  bad |= cudaMalloc((void**)&r->L.list, (size_t)TG_N_SIM_CLASSES * r->L.n_groups * sizeof(int)) != cudaSuccess;
  r->L.cursor = r->L.count ? r->L.count + 64 : nullptr;
  if (desc->max_rounds > 0) {                              // state of the trace replay
    ReplayWs& R = r->R;
    int u = 0, d = 0;
    for (int j = 0; j < P.P; ++j) {
      R.unit0[j] = u; R.dom0[j] = d;
      if (P.pool[j].type != TG_POOL_API) u += P.pool[j].capacity;
      if (P.pool[j].type == TG_POOL_CPU) d += P.pool[j].capacity / P.pool[j].group;
    }
    R.U = u ? u : 1; R.Dtot = d ? d : 1;
    R.round_us = desc->round_us > 0 ? desc->round_us : 1; R.max_rounds = desc->max_rounds;
    bad |= cudaMalloc((void**)&R.wait, SN * sizeof(int)) != cudaSuccess;
    bad |= cudaMalloc((void**)&R.run, SN * sizeof(int)) != cudaSuccess;
    bad |= cudaMalloc((void**)&R.owner, (size_t)P.S * R.U * sizeof(int)) != cudaSuccess;
    bad |= cudaMalloc((void**)&R.nm, (size_t)P.S * (node0 ? node0 : 1)) != cudaSuccess;
    bad |= cudaMalloc((void**)&R.dfree, (size_t)P.S * R.Dtot * sizeof(int)) != cudaSuccess;
    bad |= cudaMalloc((void**)&R.pst, (size_t)P.S * P.P * 2 * sizeof(int)) != cudaSuccess;
    bad |= cudaMalloc((void**)&R.win, (size_t)P.S * P.P * sizeof(i64)) != cudaSuccess;
  }
  bad |= cudaEventCreateWithFlags(&r->sim_fork, cudaEventDisableTiming) != cudaSuccess;
  for (int c = 0; c <= TG_N_SIM_CLASSES; ++c) {
    if (c == TG_N_SIM_CLASSES) {
      // the fill's stream: highest priority, so that its few blocks get in between those of k_stream
      int lo = 0, hi = 0;
      bad |= cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess;
      bad |= cudaStreamCreateWithPriority(&r->sim_stream[c], cudaStreamNonBlocking, hi) != cudaSuccess;
    } else
      bad |= cudaStreamCreateWithFlags(&r->sim_stream[c], cudaStreamNonBlocking) != cudaSuccess;
    bad |= cudaEventCreateWithFlags(&r->sim_join[c], cudaEventDisableTiming) != cudaSuccess;
  }
  {
    int lo = 0, hi = 0;
    bad |= cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess;
    bad |= cudaStreamCreateWithPriority(&r->side, cudaStreamNonBlocking, lo) != cudaSuccess;
    bad |= cudaEventCreateWithFlags(&r->side_fork, cudaEventDisableTiming) != cudaSuccess;
    bad |= cudaEventCreateWithFlags(&r->side_join, cudaEventDisableTiming) != cudaSuccess;
  }
  if (!bad && desc->host_buffers) {
    bad |= cudaStreamCreateWithFlags(&r->io_in, cudaStreamNonBlocking) != cudaSuccess;
    bad |= cudaStreamCreateWithFlags(&r->io_comp, cudaStreamNonBlocking) != cudaSuccess;
    bad |= cudaStreamCreateWithFlags(&r->io_out, cudaStreamNonBlocking) != cudaSuccess;
    bad |= cudaEventCreateWithFlags(&r->io_begin, cudaEventDisableTiming) != cudaSuccess;
    bad |= cudaEventCreateWithFlags(&r->io_end, cudaEventDisableTiming) != cudaSuccess;
    for (int c = 0; c < TG_IO_CHUNKS; ++c) {
      bad |= cudaEventCreateWithFlags(&r->io_in_done[c], cudaEventDisableTiming) != cudaSuccess;
      bad |= cudaEventCreateWithFlags(&r->io_comp_done[c], cudaEventDisableTiming) != cudaSuccess;
    }
    size_t off = 0;
    size_t in_sz[8] = {SN, SN, SN * 4, SN * 8, SN * 8, SN * 8, (size_t)P.S * 4, (size_t)P.S * (node0 ? node0 : 1)};
    for (int k = 0; k < 8; ++k) { r->in_off[k] = off; off = align_up(off + in_sz[k], 256); }
    size_t occ = (size_t)P.S * (desc->max_rounds > 0 ? desc->max_rounds : 0) * P.P * 4;
    size_t out_sz[9] = {SN * 4, SN * 4, SN * 4, SN * 8, (size_t)P.S * 8, (size_t)P.S * 4, (size_t)P.S * 4,
                        occ ? occ : 4, (size_t)P.S * 4};
    for (int k = 0; k < 9; ++k) { r->out_off[k] = off; off = align_up(off + out_sz[k], 256); }
    r->stage_bytes = off;
    bad |= cudaMalloc((void**)&r->d_stage, off) != cudaSuccess;
  }
  if (bad) { cudaGetLastError(); tangram_round_destroy(r); return TANGRAM_ENOMEM; }
  {
    // usable multiplicities by (pool, unit byte), as decode_levels computes them
    static_assert(sizeof(u32) == 4, "");
    u32* tab = new (std::nothrow) u32[TG_MAX_POOLS * 256]();
    cudaError_t ce = tab ? cudaMalloc((void**)&r->d_ok_table, TG_MAX_POOLS * 256 * sizeof(u32)) : cudaErrorMemoryAllocation;
    if (ce == cudaSuccess) {
      for (int j = 0; j < P.P; ++j)
        for (int un = 0; un < 256; ++un) {
          const int g = un & 0x7f;
          const bool gpu = P.pool[j].type == TG_POOL_GPU, gang = (un >> 7) && gpu;
          u32 ok = g == 0 ? 0u : 0xffffffffu;
          if (g != 0 && gpu) {
            const bool p2 = (g & (g - 1)) == 0;
            if (gang) {
              ok = 0;
              if (p2) {
                if (g <= P.pool[j].group) ok |= 1u;
                if (2 * g <= P.pool[j].group) ok |= 2u;
                if (4 * g <= P.pool[j].group) ok |= 8u;
                if (8 * g <= P.pool[j].group) ok |= 128u;
              }
            } else if (!(p2 && g <= P.pool[j].group)) ok = 0;
          }
          tab[j * 256 + un] = ok;
        }
      ce = cudaMemcpy(r->d_ok_table, tab, TG_MAX_POOLS * 256 * sizeof(u32), cudaMemcpyHostToDevice);
    }
    delete[] tab;
    if (ce != cudaSuccess) { cudaGetLastError(); tangram_round_destroy(r); return TANGRAM_ENOMEM; }
    P.ok_table = r->d_ok_table;
  }
  P.order = (int*)r->d_order; P.tmin = (i64*)r->d_tmin; P.meta = (PoolMeta*)r->d_meta;
  P.preq = (unsigned short*)r->d_preq; P.keepn = (int*)r->d_keepn;
  P.n_side = desc->side_costs; P.side_plane = (u64)P.S * P.N;
  P.side_bad = r->d_side_bad; P.side_res = r->d_side_res;
  P.slabs = (char*)r->d_slabs; P.arena = (char*)r->d_arena; P.arena_top = (u64*)r->d_arena_top;
  e = cudaFuncSetAttribute(k_finish, cudaFuncAttributeMaxDynamicSharedMemorySize, K2_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_solve, cudaFuncAttributeMaxDynamicSharedMemorySize, K2_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_replay<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, KR_DYN_SMEM + (KR_THREADS / 32) * KR_STATE_MAX);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_replay<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, KR_DYN_SMEM + (KR_THREADS / 32) * KR_STATE_MAX);
  for (int c = 0; c < TG_N_SIM_CLASSES && e == cudaSuccess; ++c)
    e = cudaFuncSetAttribute(sim_kernel(g_sim_caps[c]), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TG_SMEM_PER_BLOCK - 1024);
  if (e != cudaSuccess) { tangram_round_destroy(r); return cuda_fail(e, "cudaFuncSetAttribute"); }
  *out = r;
  return TANGRAM_OK;
}

extern "C" int tangram_set_profiling(tangram_round* r, int enable) {
  if (!r) return TANGRAM_EINVAL;
  if (enable && !r->ev) {
    const int n = TG_PROF_CALLS * (TG_PROF_K + 1);
    r->ev = new (std::nothrow) cudaEvent_t[n];
    if (!r->ev) return TANGRAM_ENOMEM;
    for (int i = 0; i < n; ++i) {
      cudaError_t e = cudaEventCreate(&r->ev[i]);
      if (e != cudaSuccess) {
        for (int k = 0; k < i; ++k) cudaEventDestroy(r->ev[k]);
        delete[] r->ev; r->ev = nullptr;
        return cuda_fail(e, "cudaEventCreate");
      }
    }
  }
  if (!enable && r->ev) {
    for (int i = 0; i < TG_PROF_CALLS * (TG_PROF_K + 1); ++i) cudaEventDestroy(r->ev[i]);
    delete[] r->ev; r->ev = nullptr;
  }
  r->ev_used = 0;
  return TANGRAM_OK;
}

extern "C" const char* tangram_kernel_name(int kernel) {
  return kernel >= 0 && kernel < TG_N_KERNELS ? g_kernel_names[kernel] : "";
}

extern "C" int tangram_kernel_time_ms(tangram_round* r, int kernel, double* total_ms, int64_t* launches) {
  if (!r || !total_ms || !launches || kernel < 0 || kernel >= TG_N_KERNELS) return TANGRAM_EINVAL;
  *total_ms = 0.0; *launches = 0;
  if (!r->ev) return TANGRAM_OK;
  for (int c = 0; c < r->ev_used; ++c)
    for (int k = 0; k < TG_PROF_K; ++k) {
      if (r->ev_kernel[c][k] != kernel) continue;
      float ms = 0.f;
      cudaEvent_t* e = r->ev + c * (TG_PROF_K + 1);
      CK(cudaEventElapsedTime(&ms, e[k], e[k + 1]));
      *total_ms += ms; *launches += 1;
    }
  return TANGRAM_OK;
}

// events of the current call, or null when timing is off or the event pool is used up
static cudaEvent_t* prof_begin(tangram_round* r, int k0, int k1, int k2, int k3, int k4 = -1, int k5 = -1) {
  if (!r->ev || r->ev_used >= TG_PROF_CALLS) return nullptr;
  int c = r->ev_used++;
  r->ev_kernel[c][0] = k0; r->ev_kernel[c][1] = k1; r->ev_kernel[c][2] = k2; r->ev_kernel[c][3] = k3;
  r->ev_kernel[c][4] = k4; r->ev_kernel[c][5] = k5;
  return r->ev + c * (TG_PROF_K + 1);
}

extern "C" void tangram_round_destroy(tangram_round* r) {
  if (!r) return;
  if (r->ev) tangram_set_profiling(r, 0);
  cudaFree(r->d_order); cudaFree(r->d_tmin); cudaFree(r->d_meta); cudaFree(r->d_slabs);
  cudaFree(r->d_ok_table); cudaFree(r->d_arena); cudaFree(r->d_arena_top); cudaFree(r->d_stage); cudaFree(r->hst); cudaFree(r->d_preq); cudaFree(r->d_keepn); cudaFree(r->d_fl); cudaFree(r->d_side_bad); cudaFree(r->d_side_res); cudaFree(r->d_sorted); cudaFree(r->d_perm); cudaFree(r->d_wkey);
  cudaFree(r->W.ts); cudaFree(r->W.seed2); cudaFree(r->W.rs1); cudaFree(r->W.rs2);
  cudaFree(r->L.count); cudaFree(r->L.list);
  cudaFree(r->R.wait); cudaFree(r->R.run); cudaFree(r->R.owner); cudaFree(r->R.nm); cudaFree(r->R.dfree);
  cudaFree(r->R.pst); cudaFree(r->R.win);
  if (r->io_in) cudaStreamDestroy(r->io_in);
  if (r->io_comp) cudaStreamDestroy(r->io_comp);
  if (r->io_out) cudaStreamDestroy(r->io_out);
  if (r->io_begin) cudaEventDestroy(r->io_begin);
  if (r->io_end) cudaEventDestroy(r->io_end);
  for (int c = 0; c < TG_IO_CHUNKS; ++c) {
    if (r->io_in_done[c]) cudaEventDestroy(r->io_in_done[c]);
    if (r->io_comp_done[c]) cudaEventDestroy(r->io_comp_done[c]);
  }
  if (r->side) cudaStreamDestroy(r->side);
  if (r->side_fork) cudaEventDestroy(r->side_fork);
  if (r->side_join) cudaEventDestroy(r->side_join);
  if (r->sim_fork) cudaEventDestroy(r->sim_fork);
  for (int c = 0; c <= TG_N_SIM_CLASSES; ++c) {
    if (r->sim_stream[c]) cudaStreamDestroy(r->sim_stream[c]);
    if (r->sim_join[c]) cudaEventDestroy(r->sim_join[c]);
  }
  delete r;
}

// Host-buffer mode: the staging area holds device copies of the caller's arrays.
static void bind_stage(tangram_round* r, const tangram_actions* a, Params& P) {
  char* d = r->d_stage;
  P.a_pool = (const u8*)(d + r->in_off[0]); P.a_unit = (const u8*)(d + r->in_off[1]);
  P.a_mask = (const u32*)(d + r->in_off[2]); P.a_s = (const i64*)(d + r->in_off[3]);
  P.a_p = (const i64*)(d + r->in_off[4]);
  P.a_arrival = a->arrival_us ? (const i64*)(d + r->in_off[5]) : nullptr;
  P.n_actions = (const int*)(d + r->in_off[6]);
  P.gpu_busy = (a->gpu_busy && P.n_nodes_total) ? (const u8*)(d + r->in_off[7]) : nullptr;
  P.o_alloc = (int*)(d + r->out_off[0]); P.o_node = (int*)(d + r->out_off[1]); P.o_off = (int*)(d + r->out_off[2]);
  P.o_act = (i64*)(d + r->out_off[3]); P.o_total = (i64*)(d + r->out_off[4]); P.o_nsel = (int*)(d + r->out_off[5]);
  P.o_status = (int*)(d + r->out_off[6]);
}

// inputs of scenarios [s0, s1) host -> staging
static int copy_in(tangram_round* r, const tangram_actions* a, const Params& P, int s0, int s1, cudaStream_t st) {
  char* d = r->d_stage;
  const void* src[8] = {a->pool, a->unit, a->level_mask, a->s_us, a->p_us, a->arrival_us, a->n_actions, a->gpu_busy};
  const size_t per[8] = {(size_t)P.N, (size_t)P.N, (size_t)P.N * 4, (size_t)P.N * 8, (size_t)P.N * 8, (size_t)P.N * 8,
                         4, (size_t)P.n_nodes_total};
  for (int k = 0; k < 8; ++k)
    if (src[k] && per[k])
      CK(cudaMemcpyAsync(d + r->in_off[k] + per[k] * s0, (const char*)src[k] + per[k] * s0, per[k] * (s1 - s0),
                         cudaMemcpyHostToDevice, st));
  return TANGRAM_OK;
}

// results of scenarios [s0, s1) staging -> host
static int copy_out(tangram_round* r, const tangram_result* res, const Params& P, int s0, int s1, cudaStream_t st) {
  char* d = r->d_stage;
  void* dst[7] = {res->alloc_units, res->place_node, res->place_off, res->act_us, res->total_act_us,
                  res->n_selected, res->status};
  const size_t per[7] = {(size_t)P.N * 4, (size_t)P.N * 4, (size_t)P.N * 4, (size_t)P.N * 8, 8, 4, 4};
  for (int k = 0; k < 7; ++k)
    CK(cudaMemcpyAsync((char*)dst[k] + per[k] * s0, d + r->out_off[k] + per[k] * s0, per[k] * (s1 - s0),
                       cudaMemcpyDeviceToHost, st));
  return TANGRAM_OK;
}

static bool check_io(const tangram_actions* a, const tangram_result* res) {
  return a && res && a->pool && a->unit && a->level_mask && a->s_us && a->p_us && a->n_actions &&
         res->alloc_units && res->place_node && res->place_off && res->act_us && res->total_act_us &&
         res->n_selected && res->status;
}

static void bind_device_io(Params& P, const tangram_actions* a, const tangram_result* res) {
  P.a_pool = a->pool; P.a_unit = a->unit; P.a_mask = a->level_mask;
  P.a_s = (const i64*)a->s_us; P.a_p = (const i64*)a->p_us; P.a_arrival = (const i64*)a->arrival_us;
  P.n_actions = a->n_actions;
  P.gpu_busy = P.n_nodes_total ? a->gpu_busy : nullptr;
  P.a_service = a->service; P.a_restore = (const i64*)a->restore_us;
  P.cache_tag = a->gpu_cache_tag; P.cache_use = (i64*)a->gpu_cache_use;
  P.a_side_pool = a->side_pool; P.a_side_units = a->side_units;
  if (!a->side_pool) P.n_side = 0;                         // no entries handed over: the key resource only
  P.o_alloc = res->alloc_units; P.o_node = res->place_node; P.o_off = res->place_off;
  P.o_act = (i64*)res->act_us; P.o_total = (i64*)res->total_act_us;
  P.o_nsel = res->n_selected; P.o_status = res->status;
}

// The kernels of one round for the scenarios that P describes, on stream st.
static int run_pipeline(tangram_round* r, const Params& P, const BatchWs& W, const SimLists& L, cudaStream_t st,
                        cudaEvent_t* ev) {
  const int wblocks = P.n_workers / (K2_THREADS / 32);
  const long long n_sims = (long long)P.P * P.S * 2;
  CK(cudaMemsetAsync(P.arena_top, 0, 256, st));          // arena top and the task counters
  if (ev) CK(cudaEventRecord(ev[0], st));
  if (P.n_side > 0) {
    CK(cudaMemsetAsync(P.side_bad, 0, (size_t)P.S * sizeof(int), st));
    size_t blocks = ((size_t)P.S * P.N + 255) / 256;
    if (blocks > (size_t)r->n_sm * 16) blocks = (size_t)r->n_sm * 16;
    k_side_check<<<(unsigned)blocks, 256, 0, st>>>(P);
    r->launches += 1;
  }
  if (P.n_side > 0) k_head<true><<<(P.S + 7) / 8, 256, 0, st>>>(P, r->hst);
  else k_head<false><<<(P.S + 7) / 8, 256, 0, st>>>(P, r->hst);
  if (ev) CK(cudaEventRecord(ev[1], st));
  const unsigned place_grid = ((P.S + 31) / 32 * P.P + KPL_WARPS - 1) / KPL_WARPS;
  {                                                        // the output fill runs beside everything that follows
    cudaStream_t fs = r->sim_stream[TG_N_SIM_CLASSES];
    CK(cudaEventRecord(r->sim_fork, st));
    CK(cudaStreamWaitEvent(fs, r->sim_fork, 0));
    size_t blocks = ((size_t)P.S * ((P.N + 3) / 4) + 255) / 256;
    if (blocks > (size_t)r->n_sm * TG_FILL_BLOCKS_PER_SM) blocks = (size_t)r->n_sm * TG_FILL_BLOCKS_PER_SM;
    k_fill<<<(unsigned)blocks, 256, 0, fs>>>(P, r->hst);
    CK(cudaEventRecord(r->sim_join[TG_N_SIM_CLASSES], fs));
  }
  // k_solve needs only what k_head left and could run beside k_stream; measured, the two get in each
  // other's way on the SMs (1.6 ms together against 0.65 + 0.70 one after the other), so they do not
  k_stream<<<P.S, KS_THREADS, 0, st>>>(P, r->hst);
  if (ev) CK(cudaEventRecord(ev[2], st));
  k_solve<<<wblocks, K2_THREADS, K2_DYN_SMEM, st>>>(P, W, r->hst);
  if (ev) CK(cudaEventRecord(ev[3], st));
  CK(cudaMemsetAsync(L.count, 0, 2 * 64 * sizeof(int), st));
  k_sim_classify<<<(L.n_groups + 7) / 8, 256, 0, st>>>(P, W.ts, L);
  CK(cudaEventRecord(r->sim_fork, st));
  for (int c = 0; c < TG_N_SIM_CLASSES; ++c) {
    cudaStream_t ss = r->sim_stream[c];
    CK(cudaStreamWaitEvent(ss, r->sim_fork, 0));
    const int smem = sim_smem_bytes(g_sim_caps[c]);
    int per_sm = TG_SMEM_PER_SM / (smem + 1024);
    if (per_sm > 32) per_sm = 32;
    if (per_sm < 1) per_sm = 1;
    int grid = r->n_sm * per_sm;
    if (grid > L.n_groups) grid = L.n_groups;
    sim_kernel(g_sim_caps[c])<<<grid, 32, smem, ss>>>(P, W.ts, W.seed2, L, c);
    CK(cudaEventRecord(r->sim_join[c], ss));
    CK(cudaStreamWaitEvent(st, r->sim_join[c], 0));
  }
  k_sims_big<<<(int)((n_sims + 31) / 32), 32, 0, st>>>(P, W.ts, W.seed2, g_sim_caps[TG_N_SIM_CLASSES - 1], L.count + 63);
  if (ev) CK(cudaEventRecord(ev[4], st));
  {                                                        // the certified pools: decided and placed beside the continued evictions,
                                                           // which are chains of dependent steps that leave most of the machine idle
    CK(cudaEventRecord(r->side_fork, st));
    CK(cudaStreamWaitEvent(r->side, r->side_fork, 0));
    k_easy<<<(unsigned)(((size_t)P.S * P.P + 7) / 8), 256, 0, r->side>>>(P, r->hst);
    k_place<<<place_grid, KPL_THREADS, 0, r->side>>>(P, r->hst, 0, 0);
    CK(cudaEventRecord(r->side_join, r->side));
  }
  CK(cudaMemsetAsync(r->d_fl, 0, 2 * sizeof(int), st));
  k_finish_list<<<(P.S * P.P + 255) / 256, 256, 0, st>>>(P, W, r->d_fl);
  k_finish<<<wblocks, K2_THREADS, K2_DYN_SMEM, st>>>(P, W, r->d_fl);
  if (ev) CK(cudaEventRecord(ev[5], st));
  // A warp per GPU pool is the shorter chain as long as all those warps are resident at once; beyond
  // that a thread per pool (32 pools per warp instruction) gets through the batch sooner.
  const int gpu_apart = (long long)P.S * P.P <= (long long)r->n_sm * 64 * 2 ? 1 : 0;
  k_place<<<place_grid, KPL_THREADS, 0, st>>>(P, r->hst, 1, gpu_apart);
  if (gpu_apart) k_place_gpu<<<(unsigned)(((size_t)P.S * P.P + 7) / 8), 256, 0, st>>>(P, r->hst);
  CK(cudaStreamWaitEvent(st, r->side_join, 0));
  CK(cudaStreamWaitEvent(st, r->sim_join[TG_N_SIM_CLASSES], 0));   // the fill is part of the round
  if (ev) CK(cudaEventRecord(ev[6], st));
  r->launches += 11 + TG_N_SIM_CLASSES + gpu_apart;
  CK(cudaGetLastError());
  return TANGRAM_OK;
}

extern "C" int tangram_schedule_batch(tangram_round* r, const tangram_actions* a, int64_t now_us,
                                      tangram_result* res, void* cuda_stream) {
  if (!r || !check_io(a, res)) return TANGRAM_EINVAL;
  if (r->desc.cache_slots > 0 && r->P.n_nodes_total > 0 && (!a->gpu_cache_tag || !a->gpu_cache_use)) return TANGRAM_EINVAL;
  if (r->desc.side_costs > 0 && (!a->side_pool) != (!a->side_units)) return TANGRAM_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Params P = r->P;
  P.now = now_us;
  if (!r->desc.host_buffers) {
    bind_device_io(P, a, res);
    return run_pipeline(r, P, r->W, r->L, st, prof_begin(r, 0, 7, 3, 4, 5, 6));
  }
  bind_stage(r, a, P);
  // Host buffers: scenarios go through in chunks, so that the copy-in of a chunk, the kernels
  // of the one before and the copy-out of the one before that overlap (three internal streams).
  const size_t bytes = (size_t)P.S * P.N * 42;
  int C = (int)(bytes >> 26);                              // about 64 MiB of traffic per chunk
  if (C > TG_IO_CHUNKS) C = TG_IO_CHUNKS;
  if (C > P.S) C = P.S;
  if (C <= 1 || r->ev) {                                   // small batch, or per-kernel timing wanted
    int rc = copy_in(r, a, P, 0, P.S, st);
    if (!rc) rc = run_pipeline(r, P, r->W, r->L, st, prof_begin(r, 0, 7, 3, 4, 5, 6));
    if (!rc) rc = copy_out(r, res, P, 0, P.S, st);
    return rc;
  }
  CK(cudaEventRecord(r->io_begin, st));
  CK(cudaStreamWaitEvent(r->io_in, r->io_begin, 0));
  CK(cudaStreamWaitEvent(r->io_comp, r->io_begin, 0));
  CK(cudaStreamWaitEvent(r->io_out, r->io_begin, 0));
  for (int c = 0; c < C; ++c) {
    const int s0 = (int)((long long)P.S * c / C), s1 = (int)((long long)P.S * (c + 1) / C);
    const size_t o = (size_t)s0 * P.N;
    int rc = copy_in(r, a, P, s0, s1, r->io_in);
    if (rc) return rc;
    CK(cudaEventRecord(r->io_in_done[c], r->io_in));
    Params Q = P;                                          // this chunk's view of everything per scenario
    Q.S = s1 - s0;
    Q.a_pool += o; Q.a_unit += o; Q.a_mask += o; Q.a_s += o; Q.a_p += o;
    if (Q.a_arrival) Q.a_arrival += o;
    Q.n_actions += s0;
    if (Q.gpu_busy) Q.gpu_busy += (size_t)s0 * P.n_nodes_total;
    Q.o_alloc += o; Q.o_node += o; Q.o_off += o; Q.o_act += o;
    Q.o_total += s0; Q.o_nsel += s0; Q.o_status += s0;
    if ((int64_t)Q.n_workers > (int64_t)Q.S * P.P) Q.n_workers = (int)align_up((size_t)Q.S * P.P, K2_THREADS / 32);
    SimLists L = r->L;
    L.n_groups = (int)(((long long)P.P * Q.S * 2 + SIM_PER_WARP - 1) / SIM_PER_WARP);
    CK(cudaStreamWaitEvent(r->io_comp, r->io_in_done[c], 0));
    rc = run_pipeline(r, Q, r->W, L, r->io_comp, nullptr);   // the workspace is reused chunk after chunk
    if (rc) return rc;
    CK(cudaEventRecord(r->io_comp_done[c], r->io_comp));
    CK(cudaStreamWaitEvent(r->io_out, r->io_comp_done[c], 0));
    rc = copy_out(r, res, P, s0, s1, r->io_out);
    if (rc) return rc;
  }
  CK(cudaEventRecord(r->io_end, r->io_out));
  CK(cudaStreamWaitEvent(st, r->io_end, 0));
  return TANGRAM_OK;
}

static int replay_impl(tangram_round* r, const tangram_actions* a, tangram_result* res, void* cuda_stream, int policy,
                       const tangram_pinning* pin = nullptr);

extern "C" int tangram_replay_trace(tangram_round* r, const tangram_actions* a, tangram_result* res,
                                    void* cuda_stream) {
  return replay_impl(r, a, res, cuda_stream, 0);
}

extern "C" int tangram_replay_trace_ordered(tangram_round* r, const tangram_actions* a, int policy, tangram_result* res,
                                            void* cuda_stream) {
  if (policy < 0 || policy > 3) return TANGRAM_EINVAL;
  return replay_impl(r, a, res, cuda_stream, policy == 3 ? 0 : policy);   // a trace is sorted by arrival already
}

extern "C" int tangram_replay_trace_pinned(tangram_round* r, const tangram_actions* a, int policy,
                                           const tangram_pinning* pin, tangram_result* res, void* cuda_stream) {
  if (policy < 0 || policy > 3 || !r || !pin || r->desc.host_buffers || !pin->trajectory || !pin->traj_mem ||
      pin->max_trajectories < 1 || !pin->traj_node || !pin->node_mem_free || !pin->pool_out)
    return TANGRAM_EINVAL;
  return replay_impl(r, a, res, cuda_stream, policy == 3 ? 0 : policy, pin);
}

static int replay_impl(tangram_round* r, const tangram_actions* a, tangram_result* res, void* cuda_stream, int policy,
                       const tangram_pinning* pin) {
  if (!r || !check_io(a, res) || r->desc.max_rounds <= 0 || !a->arrival_us) return TANGRAM_EINVAL;
  if (policy && !r->d_wkey) {                              // sort keys of the waiting actions, kept by the round
    if (cudaMalloc((void**)&r->d_wkey, (size_t)r->P.S * r->P.N * sizeof(u64)) != cudaSuccess) {
      cudaGetLastError(); r->d_wkey = nullptr;
      return TANGRAM_ENOMEM;
    }
  }
  if (r->desc.cache_slots > 0 && r->P.n_nodes_total > 0 && (!a->gpu_cache_tag || !a->gpu_cache_use)) return TANGRAM_EINVAL;
  if (r->desc.side_costs > 0 && (!a->side_pool) != (!a->side_units)) return TANGRAM_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Params P = r->P;
  P.now = 0;
  ReplayWs R = r->R;
  R.policy = policy; R.wkey = policy ? r->d_wkey : nullptr;
  R.trajectory = nullptr; R.traj_mem = nullptr; R.traj_last = nullptr; R.max_traj = 0;
  R.traj_node = nullptr; R.mem_free = nullptr; R.pool_rw = nullptr;
  if (r->desc.host_buffers) {
    bind_stage(r, a, P);
    int rc = copy_in(r, a, P, 0, P.S, st);
    if (rc) return rc;
    R.occupancy = res->occupancy ? (int*)(r->d_stage + r->out_off[7]) : nullptr;
    R.rounds_used = res->rounds_used ? (int*)(r->d_stage + r->out_off[8]) : nullptr;
  } else {
    bind_device_io(P, a, res);
    R.occupancy = res->occupancy; R.rounds_used = res->rounds_used;
  }
  CK(cudaMemsetAsync(P.arena_top, 0, 256, st));
  int warps = P.n_workers < P.S ? P.n_workers : (int)align_up((size_t)P.S, K2_THREADS / 32);
  cudaEvent_t* ev = prof_begin(r, 2, -1, -1, -1);
  if (ev) CK(cudaEventRecord(ev[0], st));
  {
    // a scenario's live state (owner of every unit, node masks, free cores per domain, quota counters) goes to
    // shared memory when it is small
    const size_t need = align16((size_t)R.U * 4) + align16((size_t)P.n_nodes_total + 1) + align16((size_t)R.Dtot * 4) +
                        2 * align16((size_t)P.P * 8);
    R.state_bytes = need <= KR_STATE_MAX ? (int)need : 0;
  }
  if (pin) {
    // the kernel reads and rewrites the caller's pool_out: it starts as a copy of the pool column
    CK(cudaMemcpyAsync(pin->pool_out, a->pool, (size_t)P.S * P.N, cudaMemcpyDeviceToDevice, st));
    P.a_pool = pin->pool_out;
    R.trajectory = pin->trajectory; R.traj_mem = pin->traj_mem; R.traj_last = pin->traj_last;
    R.max_traj = pin->max_trajectories; R.traj_node = pin->traj_node; R.mem_free = (i64*)pin->node_mem_free;
    R.pool_rw = pin->pool_out;
  }
  if (policy || pin) k_replay<true><<<warps / (KR_THREADS / 32), KR_THREADS, KR_DYN_SMEM + (KR_THREADS / 32) * R.state_bytes, st>>>(P, R);
  else k_replay<false><<<warps / (KR_THREADS / 32), KR_THREADS, KR_DYN_SMEM + (KR_THREADS / 32) * R.state_bytes, st>>>(P, R);
  if (ev) CK(cudaEventRecord(ev[1], st));
  r->launches += 1;
  CK(cudaGetLastError());
  if (r->desc.host_buffers) {
    int rc = copy_out(r, res, P, 0, P.S, st);
    if (rc) return rc;
    if (res->occupancy)
      CK(cudaMemcpyAsync(res->occupancy, r->d_stage + r->out_off[7],
                         (size_t)P.S * r->desc.max_rounds * P.P * sizeof(int), cudaMemcpyDeviceToHost, st));
    if (res->rounds_used)
      CK(cudaMemcpyAsync(res->rounds_used, r->d_stage + r->out_off[8], (size_t)P.S * sizeof(int), cudaMemcpyDeviceToHost, st));
  }
  return TANGRAM_OK;
}

// ---------------------------------------------------------------------------------------
// Other queue orders (Section 4.2) and trajectories pinned to CPU nodes (Section 5.2)
// ---------------------------------------------------------------------------------------
static int next_pow2(int v) { int p = 1; while (p < v) p <<= 1; return p; }

static int launch_order(tangram_round* r, const Params& P, int policy, int* perm, cudaStream_t st) {
  OrderIo O;
  O.policy = policy; O.n_pad = next_pow2(P.N); O.perm = perm;
  const bool wide = policy == 3;
  if (!wide && O.n_pad >= KO_THREADS) {                  // whole elements per thread: the register version
    const int ept = O.n_pad / KO_THREADS;
    const size_t sm = (size_t)O.n_pad * 8;
    void (*kern)(Params, OrderIo) = ept == 1 ? k_order_regs<1> : ept == 2 ? k_order_regs<2> : ept == 4 ? k_order_regs<4> :
                                    ept == 8 ? k_order_regs<8> : ept == 16 ? k_order_regs<16> : k_order_regs<32>;
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm));
    kern<<<P.S, KO_THREADS, sm, st>>>(P, O);
    r->launches += 1;
    CK(cudaGetLastError());
    return TANGRAM_OK;
  }
  const size_t smem = (size_t)O.n_pad * (wide ? 12 : 8);
  CK(cudaFuncSetAttribute(wide ? k_order<true> : k_order<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  if (wide) k_order<true><<<P.S, KO_THREADS, smem, st>>>(P, O);
  else k_order<false><<<P.S, KO_THREADS, smem, st>>>(P, O);
  r->launches += 1;
  CK(cudaGetLastError());
  return TANGRAM_OK;
}

static bool order_args_ok(const tangram_round* r, const tangram_actions* a, int policy) {
  return r && a && a->pool && a->unit && a->level_mask && a->s_us && a->p_us && a->n_actions &&
         policy >= 1 && policy <= 3 && !r->desc.host_buffers;
}

extern "C" int tangram_order_queue(tangram_round* r, const tangram_actions* a, int policy, int32_t* perm,
                                   void* cuda_stream) {
  if (!order_args_ok(r, a, policy) || !perm) return TANGRAM_EINVAL;
  if (r->P.N > KO_MAX_N) return TANGRAM_ETOOBIG;
  Params P = r->P;
  P.a_pool = a->pool; P.a_unit = a->unit; P.a_mask = a->level_mask;
  P.a_s = (const i64*)a->s_us; P.a_p = (const i64*)a->p_us; P.a_arrival = (const i64*)a->arrival_us;
  P.n_actions = a->n_actions;
  return launch_order(r, P, policy, perm, (cudaStream_t)cuda_stream);
}

extern "C" int tangram_schedule_batch_ordered(tangram_round* r, const tangram_actions* a, int policy, int64_t now_us,
                                              tangram_result* res, void* cuda_stream) {
  if (!r || !check_io(a, res)) return TANGRAM_EINVAL;
  if (policy == 0) return tangram_schedule_batch(r, a, now_us, res, cuda_stream);
  if (!order_args_ok(r, a, policy) || r->desc.cache_slots > 0 || r->desc.side_costs > 0) return TANGRAM_EINVAL;
  if (r->P.N > KO_MAX_N) return TANGRAM_ETOOBIG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Params P = r->P;
  P.now = now_us;
  bind_device_io(P, a, res);
  const size_t SN = (size_t)P.S * P.N;
  // sorted records (pool, unit, mask, s, p, arrival) and sorted results (alloc, node, off, act): 50 B per action
  const size_t off_unit = align_up(SN, 256), off_mask = off_unit + align_up(SN, 256), off_s = off_mask + align_up(SN * 4, 256),
               off_p = off_s + SN * 8, off_arr = off_p + SN * 8, off_alloc = off_arr + SN * 8, off_node = off_alloc + SN * 4,
               off_off = off_node + SN * 4, off_act = align_up(off_off + SN * 4, 256), total = off_act + SN * 8;
  if (!r->d_sorted) {
    if (cudaMalloc((void**)&r->d_sorted, total) != cudaSuccess || cudaMalloc((void**)&r->d_perm, SN * sizeof(int)) != cudaSuccess) {
      cudaGetLastError();
      cudaFree(r->d_sorted); cudaFree(r->d_perm); cudaFree(r->d_wkey); r->d_sorted = nullptr; r->d_perm = nullptr;
      return TANGRAM_ENOMEM;
    }
  }
  char* d = r->d_sorted;
  int rc = launch_order(r, P, policy, r->d_perm, st);
  if (rc) return rc;
  GatherIo G;
  G.perm = r->d_perm; G.pool = (u8*)d; G.unit = (u8*)(d + off_unit); G.mask = (u32*)(d + off_mask);
  G.s = (i64*)(d + off_s); G.p = (i64*)(d + off_p); G.arrival = P.a_arrival ? (i64*)(d + off_arr) : nullptr;
  size_t blocks = (SN + 255) / 256;
  if (blocks > (size_t)r->n_sm * 32) blocks = (size_t)r->n_sm * 32;
  k_gather<<<(unsigned)blocks, 256, 0, st>>>(P, G);
  // the round itself, on the sorted copy; the per-scenario results go straight to the caller
  Params Q = P;
  Q.a_pool = G.pool; Q.a_unit = G.unit; Q.a_mask = G.mask; Q.a_s = G.s; Q.a_p = G.p; Q.a_arrival = G.arrival;
  Q.o_alloc = (int*)(d + off_alloc); Q.o_node = (int*)(d + off_node); Q.o_off = (int*)(d + off_off); Q.o_act = (i64*)(d + off_act);
  rc = run_pipeline(r, Q, r->W, r->L, st, nullptr);
  if (rc) return rc;
  ScatterIo X;
  X.perm = r->d_perm; X.alloc = Q.o_alloc; X.node = Q.o_node; X.off = Q.o_off; X.act = Q.o_act;
  X.o_alloc = P.o_alloc; X.o_node = P.o_node; X.o_off = P.o_off; X.o_act = P.o_act;
  k_scatter<<<(unsigned)blocks, 256, 0, st>>>(P, X);
  r->launches += 2;
  CK(cudaGetLastError());
  return TANGRAM_OK;
}

extern "C" int tangram_pin_trajectories(tangram_round* r, const tangram_actions* a, const tangram_pinning* pin,
                                        void* cuda_stream) {
  if (!r || !a || !pin || !a->pool || !a->unit || !a->level_mask || !a->n_actions || r->desc.host_buffers ||
      !pin->trajectory || !pin->traj_mem || pin->max_trajectories < 1 || !pin->traj_node || !pin->node_mem_free ||
      !pin->pool_out || !pin->n_admitted)
    return TANGRAM_EINVAL;
  Params P = r->P;
  P.a_pool = a->pool; P.a_unit = a->unit; P.a_mask = a->level_mask; P.n_actions = a->n_actions;
  PinIo X;
  X.trajectory = pin->trajectory; X.traj_mem = pin->traj_mem; X.max_traj = pin->max_trajectories;
  X.traj_node = pin->traj_node; X.mem_free = (i64*)pin->node_mem_free; X.pool_out = pin->pool_out;
  X.n_admitted = pin->n_admitted;
  k_pin<<<(P.S + 7) / 8, 256, 0, (cudaStream_t)cuda_stream>>>(P, X);
  r->launches += 1;
  CK(cudaGetLastError());
  return TANGRAM_OK;
}

// ---------------------------------------------------------------------------------------
// tangram_schedule_batch_static: the same round for callers that must not allocate.
// All scratch (partition order, least-level durations, per-pool facts, worker slabs, DP arena)
// is carved out of one file-scope device array that every GPU loading this library holds
// until the process exits.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[TANGRAM_STATIC_SCRATCH_BYTES];

#define TG_MAX_DEVICES 64
static unsigned char* g_static_ptr[TG_MAX_DEVICES];   // device address of the array, per device
static bool g_static_ready[TG_MAX_DEVICES];

// Once per device, with that device current: resolve the array's device address (its name is
// only a host-side handle here and must not be handed to a kernel) and load the constant tables.
static int static_setup(int* dev_out) {
  int dev = -1;
  CK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= TG_MAX_DEVICES) return TANGRAM_EINVAL;
  if (!g_static_ready[dev]) {
    unsigned char* ptr = nullptr;
    CK(cudaGetSymbolAddress((void**)&ptr, g_static_scratch));
    CK(fill_tables());
    g_static_ptr[dev] = ptr;
    g_static_ready[dev] = true;
  }
  *dev_out = dev;
  return TANGRAM_OK;
}

extern "C" int tangram_schedule_batch_static(const tangram_round_desc* desc, const tangram_actions* a,
                                             int64_t now_us, tangram_result* res, void* cuda_stream) {
  if (!desc || !desc->pools || !check_io(a, res)) return TANGRAM_EINVAL;
  if (desc->n_scenarios < 1 || desc->max_actions < 1 || desc->n_pools < 1 ||
      desc->n_pools > TANGRAM_MAX_POOLS || desc->depth < 1 || desc->depth > 32 || desc->host_buffers ||
      desc->cache_slots != 0 || desc->side_costs != 0)
    return TANGRAM_EINVAL;
  if ((int64_t)desc->n_scenarios * desc->max_actions > (int64_t)1 << 31) return TANGRAM_ETOOBIG;
  Params P;
  memset(&P, 0, sizeof(P));
  P.S = desc->n_scenarios; P.N = desc->max_actions; P.P = desc->n_pools; P.depth = desc->depth;
  int node0 = 0, slot0 = 0;
  for (int j = 0; j < desc->n_pools; ++j) {
    const tangram_pool_desc& pd = desc->pools[j];
    bool ok = pd.capacity >= 1 && pd.capacity <= (1 << 20) && pd.window_us >= 0;
    if (pd.type == TANGRAM_POOL_GPU)
      ok = ok && (pd.group == 1 || pd.group == 2 || pd.group == 4 || pd.group == 8) && pd.capacity % pd.group == 0;
    else if (pd.type == TANGRAM_POOL_CPU) ok = ok && pd.group >= 1 && pd.capacity % pd.group == 0;
    else if (pd.type != TANGRAM_POOL_API) ok = false;
    if (!ok) return TANGRAM_EINVAL;
    PoolDev& d = P.pool[j];
    d.type = pd.type; d.capacity = pd.capacity; d.group = pd.type == TANGRAM_POOL_API ? 1 : pd.group;
    d.window_us = pd.type == TANGRAM_POOL_API ? pd.window_us : 0;
    d.node0 = node0; d.n_nodes = pd.type == TANGRAM_POOL_GPU ? pd.capacity / pd.group : 0;
    node0 += d.n_nodes;
    d.slot0 = slot0; d.n_slots = pd.type == TANGRAM_POOL_GPU ? 4 : 1;
    slot0 += d.n_slots;
  }
  P.n_nodes_total = node0;
  P.V = slot0 + desc->n_pools;
  fill_pool_order(P);
  P.now = now_us;

  // carve the array: fixed parts first, then as many worker slabs as fit, the rest is the arena
  const size_t SN = (size_t)P.S * P.N;
  const size_t budget = TANGRAM_STATIC_SCRATCH_BYTES, arena_min = (size_t)4 << 20;
  size_t off = 0;
  const size_t o_top = off;   off = align_up(off + 256, 256);
  const size_t o_meta = off;  off = align_up(off + (size_t)P.S * P.P * sizeof(PoolMeta), 256);
  const size_t o_order = off; off = align_up(off + SN * sizeof(int), 256);
  const size_t o_tmin = off;  off = align_up(off + SN * sizeof(i64), 256);
  size_t per_cand = 8 + 8 + 4 + 4 + 4 + 4 + 4 + 3 + 16 * (size_t)desc->depth;
  size_t slab = align_up((size_t)P.N * per_cand + 64 * 1024 + (1 << 20) / 4 + 4096, 256);
  const int wpb = K2_THREADS / 32;
  if (off + arena_min + slab * wpb > budget) return TANGRAM_ETOOBIG;
  size_t workers = (budget - off - arena_min) / slab / wpb * wpb;
  size_t wanted = align_up((size_t)P.S * P.P, wpb);
  if (workers > wanted) workers = wanted;
  if (workers > 32) workers = 32;                       // keep most of the array for DP tables
  const size_t o_slabs = off; off += workers * slab;
  const size_t o_arena = off;

  int dev = -1;
  int rc = static_setup(&dev);
  if (rc) return rc;
  unsigned char* base = g_static_ptr[dev];
  P.arena_top = (u64*)(base + o_top); P.meta = (PoolMeta*)(base + o_meta);
  P.order = (int*)(base + o_order); P.tmin = (i64*)(base + o_tmin);
  P.slabs = (char*)(base + o_slabs); P.slab_bytes = slab; P.n_workers = (int)workers;
  P.arena = (char*)(base + o_arena); P.arena_bytes = budget - o_arena;
  P.slot_tries = 50000;
  bind_device_io(P, a, res);

  cudaStream_t st = (cudaStream_t)cuda_stream;
  CK(cudaMemsetAsync(P.arena_top, 0, 256, st));           // the only part that must start at zero
  k_prefix<<<P.S, K1_THREADS, P.V * K1_THREADS * sizeof(int), st>>>(P);
  CK(cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, K2_DYN_SMEM));
  k_select<<<P.n_workers / wpb, K2_THREADS, K2_DYN_SMEM, st>>>(P);
  CK(cudaGetLastError());
  return TANGRAM_OK;
}
