// Device-resident trace replay (workflow of Section 3: submit, queue, schedule, execute,
// return), one warp per scenario, no host round trips.  Every round at now = r * round_us
//   1. refills quota pools whose window changed (Section 5.1),
//   2. releases what has finished (cores, chunks, concurrency slots),
//   3. admits the actions that have arrived to the waiting queue,
//   4. runs the scheduler of Algorithm 1 on the queue with the running actions of a pool in
//      its completion heap (Algorithm 2), using the same per-pool routines as a single round,
//   5. starts what was selected and records the occupancy.
// Rounds with an empty queue are skipped ahead to the next arrival or completion (their
// occupancy rows are still written).
#pragma once
#include "common.cuh"
#include "sims.cuh"
#include "select.cuh"
#include "place.cuh"
#include "order_pin.cuh"

struct ReplayWs {
  int* wait;        // [S][N] waiting actions in queue order
  int* run;         // [S][N] running actions
  int* owner;       // [S][U]  action holding each core / GPU (-1 free, -2 occupied beforehand)
  u8* nm;           // [S][nodes] GPU busy masks
  int* dfree;       // [S][Dtot] free cores per NUMA domain
  int* pst;         // [S][P][2] quota used in the window / concurrency slots in use
  i64* win;         // [S][P] current quota window
  int unit0[TG_MAX_POOLS], dom0[TG_MAX_POOLS];   // first unit / domain of every pool in a row
  int U, Dtot;
  i64 round_us; int max_rounds;
  int* occupancy; int* rounds_used;
  int policy;       // 0: first come first served; 1 / 2: the queue is kept in shortest / longest least-level duration order
  u64* wkey;        // [S][N] sort keys of the waiting actions (policy 1 / 2 only)
  // trajectories pinned to CPU nodes as their actions arrive (Section 5.2); trajectory == nullptr: none of it
  const int* trajectory; const u32* traj_mem; const u8* traj_last; int max_traj;
  int* traj_node; i64* mem_free; u8* pool_rw;   // pool_rw: the pool column the kernel reads (P.a_pool) and rewrites
  int state_bytes;  // > 0: a scenario's live state (owner .. win) fits that many bytes of shared memory per warp
};

// Where the live state of the scenario at hand is: the arrays of ReplayWs, or the warp's shared memory (the
// bases are moved back by the scenario's offset, so that the same indexing reaches either).
__host__ __device__ __forceinline__ size_t align16(size_t v) { return (v + 15) & ~(size_t)15; }
struct ReplayState { int* owner; u8* nm; int* dfree; int* pst; i64* win; };

__device__ __forceinline__ int pool_busy_units(const Params& P, const ReplayWs& R, const ReplayState& Z, int sc, int j, int lane) {
  const PoolDev& pd = P.pool[j];
  int b = 0;
  if (pd.type == TG_POOL_API) b = pd.window_us > 0 ? Z.pst[((size_t)sc * P.P + j) * 2] : Z.pst[((size_t)sc * P.P + j) * 2 + 1];
  else {
    const int* ow = Z.owner + (size_t)sc * R.U + R.unit0[j];
    for (int c = lane; c < pd.capacity; c += 32) b += ow[c] != -1;
    b = warp_sum32(b);
  }
  return b;
}

// Candidate prefix of the waiting queue (Algorithm 1, line 2) against the pools' current state.
// dem / cap: 4 ints per pool in the warp's scratch.  Warp-uniform result.
// aside: per pool, what the candidates ask of it beside their key resource (cost vectors);
// ncand: per pool, how many of the candidates have it as their key pool.
__device__ int replay_prefix(const Params& P, const ReplayWs& R, const ReplayState& Z, int sc, const int* wait, int nw,
                             int* dem, int* cap, int* aside, int* ncand, int lane) {
  const size_t row = (size_t)sc * P.N;
  for (int j = 0; j < P.P; ++j) {
    const PoolDev& pd = P.pool[j];
    int c[4] = {0, 0, 0, 0};
    if (pd.type == TG_POOL_GPU) gpu_caps(pd, Z.nm + (size_t)sc * P.n_nodes_total, lane, c);
    else if (pd.type == TG_POOL_CPU) {
      int f = 0;
      for (int d = lane; d < pd.capacity / pd.group; d += 32) f += Z.dfree[(size_t)sc * R.Dtot + R.dom0[j] + d];
      c[0] = warp_sum32(f);
    } else {
      const int* ps = Z.pst + ((size_t)sc * P.P + j) * 2;
      c[0] = pd.capacity - (pd.window_us > 0 ? ps[0] : ps[1]);
    }
    if (lane < 4) { cap[j * 4 + lane] = c[lane]; dem[j * 4 + lane] = 0; }
  }
  if (lane < TG_MAX_POOLS) { aside[lane] = 0; ncand[lane] = 0; }
  __syncwarp();
  int n = 0;
  bool stop = false;
  for (int i0 = 0; i0 < nw && !stop; i0 += 32) {
    // every lane decodes one waiting action, then the 32 are admitted one after the other
    int j = 0, lz = 0, units = 0;
    int k0 = 0xff, u0 = 0, k1 = 0xff, u1 = 0;            // further entries of the cost vector
    if (i0 + lane < nw) {
      const int a = wait[i0 + lane];
      if (P.n_side > 0) {
        k0 = P.a_side_pool[row + a]; u0 = P.a_side_units[row + a];
        if (P.n_side > 1) { k1 = P.a_side_pool[P.side_plane + row + a]; u1 = P.a_side_units[P.side_plane + row + a]; }
      }
      j = P.a_pool[row + a];
      int g, gang; u32 eff;
      decode_levels(P.pool[j], P.a_unit[row + a], P.a_mask[row + a], g, gang, eff);
      const int rmin = __ffs(eff);
      units = g * rmin;
      lz = P.pool[j].type == TG_POOL_GPU ? level_of(g, gang, rmin) : 0;
    }
    const int nb = min(32, nw - i0);
    for (int b = 0; b < nb; ++b) {
      const int bj = __shfl_sync(TG_FULL, j, b), bl = __shfl_sync(TG_FULL, lz, b), bu = __shfl_sync(TG_FULL, units, b);
      bool over = false;
      for (int l = 0; l <= bl; ++l) over |= dem[bj * 4 + l] + bu > cap[bj * 4 + l];
      int a0 = 0xff, c0 = 0, a1 = 0xff, c1 = 0;
      if (P.n_side > 0) {
        a0 = __shfl_sync(TG_FULL, k0, b); c0 = __shfl_sync(TG_FULL, u0, b);
        a1 = __shfl_sync(TG_FULL, k1, b); c1 = __shfl_sync(TG_FULL, u1, b);
        if (a0 != 0xff) over |= dem[a0 * 4] + c0 > cap[a0 * 4];
        if (a1 != 0xff) over |= dem[a1 * 4] + c1 + (a1 == a0 ? c0 : 0) > cap[a1 * 4];
      }
      if (over) { stop = true; break; }
      __syncwarp();
      if (lane <= bl) dem[bj * 4 + lane] += bu;
      if (lane == 0) {
        ncand[bj] += 1;
        if (a0 != 0xff) { dem[a0 * 4] += c0; aside[a0] += c0; }
        if (a1 != 0xff) { dem[a1 * 4] += c1; aside[a1] += c1; }
      }
      __syncwarp();
      ++n;
    }
  }
  return n;
}

// One pool of one replay round: selection among the pool's candidates (the first n waiting
// actions that sit on pool j), placement on the pool's live state, start of what was selected.
// Appends the started actions to run[] (nr updated).  Returns false if the scratch ran out.
__device__ bool replay_pool(const Params& P, const ReplayWs& R, const ReplayState& Z, int sc, int j, const int* wait, int nw, int n,
                            int* run, int& nr, i64 now, Slab slab, int lane, int& busy_units, int aside_j, int m) {
  const size_t row = (size_t)sc * P.N;
  const PoolDev& pd = P.pool[j];
  // m: members of the pool among the candidates (counted by the prefix); n_ac: members behind them, which
  // only an eviction step's estimate looks at (a single candidate is never evicted)
  int n_ac = 0;
  for (int i0 = n & ~31; i0 < nw && m >= 2; i0 += 32) {
    const int i = i0 + lane;
    const bool mine = i < nw && i >= n && P.a_pool[row + wait[i]] == j;
    n_ac += __popc(__ballot_sync(TG_FULL, mine));
  }
  if (m == 0) return true;
  CandArrays C;
  C.cs = (i64*)slab.take((u64)m * 8); C.cp = (i64*)slab.take((u64)m * 8);
  C.cmask = (u32*)slab.take((u64)m * 4); C.cidx = (int*)slab.take((u64)m * 4);
  C.pnode = (int*)slab.take((u64)m * 4); C.poff = (int*)slab.take((u64)m * 4);
  C.rowcand = (int*)slab.take((u64)m * 4);
  C.cg = (u8*)slab.take(m); C.rsel = (u8*)slab.take(m); C.rkeep = (u8*)slab.take(m);
  i64* ac_tmin = (i64*)slab.take((u64)(n_ac + 1) * 8);
  i64* seeds = (i64*)slab.take((u64)(nr + 1) * 8);
  if (!C.cs || !C.cp || !C.cmask || !C.cidx || !C.pnode || !C.poff || !C.rowcand || !C.cg || !C.rsel || !C.rkeep ||
      !ac_tmin || !seeds) return false;
  // fill them in queue order
  int cm = 0, ca = 0, first_ac = -1;
  bool elastic = false;
  for (int i0 = 0; i0 < nw; i0 += 32) {
    const int i = i0 + lane;
    int a = -1; bool mine = false;
    if (i < nw) { a = wait[i]; mine = P.a_pool[row + a] == j; }
    const u32 bc = __ballot_sync(TG_FULL, mine && i < n), ba = __ballot_sync(TG_FULL, mine && i >= n);
    if (mine && (i < n || m >= 2)) {                    // (the waiting actions' durations feed the estimate only)
      int g, gang; u32 eff;
      decode_levels(pd, P.a_unit[row + a], P.a_mask[row + a], g, gang, eff);
      const i64 s = clamp_param(P.a_s[row + a]), p = clamp_param(P.a_p[row + a]);
      if (i < n) {
        const int k = cm + __popc(bc & ((1u << lane) - 1u));
        C.cidx[k] = a; C.cmask[k] = eff; C.cg[k] = (u8)(g | (gang << 7)); C.cs[k] = s; C.cp[k] = p;
        C.rkeep[k] = (u8)__ffs(eff); C.pnode[k] = -1; C.poff[k] = -1;
        elastic |= (eff & (eff - 1)) != 0;
      } else {
        ac_tmin[ca + __popc(ba & ((1u << lane) - 1u))] = duration(s, p, __ffs(eff));
      }
    }
    if (first_ac < 0 && ba) first_ac = __shfl_sync(TG_FULL, a, __ffs(ba) - 1);
    cm += __popc(bc); ca += __popc(ba);
  }
  elastic = __any_sync(TG_FULL, elastic);
  // completion times (relative to now) of what runs on this pool seed the heap
  // (only an eviction step looks at the heap: with one candidate, or none that is elastic, nobody reads it)
  int ns = 0;
  for (int i0 = 0; i0 < nr && elastic && m >= 2; i0 += 32) {
    const int i = i0 + lane;
    int a = -1; bool mine = false;
    if (i < nr) { a = run[i]; mine = P.a_pool[row + a] == j; }
    const u32 b = __ballot_sync(TG_FULL, mine);
    if (mine) {
      const i64 fin = (P.a_arrival ? P.a_arrival[row + a] : 0) + P.o_act[row + a];
      seeds[ns + __popc(b & ((1u << lane) - 1u))] = fin > now ? fin - now : 0;
    }
    ns += __popc(b);
  }
  __syncwarp();
  int keep = m;
  if (elastic) {
    PoolTask T;
    T.type = pd.type; T.group = pd.group;
    T.cap[0] = T.cap[1] = T.cap[2] = T.cap[3] = 0;
    if (pd.type == TG_POOL_GPU) gpu_caps(pd, Z.nm + (size_t)sc * P.n_nodes_total, lane, T.cap);
    else if (pd.type == TG_POOL_CPU) {
      int f = 0;
      for (int d = lane; d < pd.capacity / pd.group; d += 32) f += Z.dfree[(size_t)sc * R.Dtot + R.dom0[j] + d];
      T.cap[0] = warp_sum32(f);
    } else {
      const int* ps = Z.pst + ((size_t)sc * P.P + j) * 2;
      T.cap[0] = pd.capacity - (pd.window_us > 0 ? ps[0] : ps[1]) - aside_j;   // set aside for the other pools' candidates
    }
    T.m = m; T.cs = C.cs; T.cp = C.cp; T.cmask = C.cmask; T.cg = C.cg;
    T.n_ac = n_ac; T.ac_tmin = ac_tmin;
    T.ac_first.s = T.ac_first.p = 0; T.ac_first.mask = 1; T.ac_first.g = 1; T.ac_first.gang = 0;
    if (n_ac > 0) {
      decode_levels(pd, P.a_unit[row + first_ac], P.a_mask[row + first_ac], T.ac_first.g, T.ac_first.gang, T.ac_first.mask);
      T.ac_first.s = clamp_param(P.a_s[row + first_ac]); T.ac_first.p = clamp_param(P.a_p[row + first_ac]);
    }
    T.seeds = seeds; T.n_seeds = ns;
    T.depth = P.depth;
    T.rsel = C.rsel; T.rkeep = C.rkeep; T.rowcand = C.rowcand;
    T.sim_base = 0; T.sim_cap = 0;
    attach_warp_tree(T);
    keep = evict_loop(P, T, slab, lane);
    if (keep < 0) return false;
  }
  // placement on the pool's live state
  const u8* missed = nullptr;                            // candidates whose chunk did not cache their service
  if (pd.type == TG_POOL_GPU && P.cache_slots > 0) {
    const size_t cbase = ((size_t)sc * P.n_nodes_total + pd.node0) * 8 * P.cache_slots;
    place_gpu_cache(pd, Z.nm + (size_t)sc * P.n_nodes_total + pd.node0, keep, C.cg, C.rkeep, C.cidx, C.pnode, C.poff,
                    C.rsel, P.a_service ? P.a_service + row : nullptr, P.cache_tag + cbase, P.cache_use + cbase,
                    P.cache_slots, now, lane, Z.owner + (size_t)sc * R.U + R.unit0[j]);
    missed = C.rsel;
  } else if (pd.type == TG_POOL_GPU) {
    place_gpu(pd, Z.nm + (size_t)sc * P.n_nodes_total + pd.node0, keep, C.cg, C.rkeep, C.pnode, C.poff, lane,
              Z.owner + (size_t)sc * R.U + R.unit0[j], C.cidx);
  } else if (pd.type == TG_POOL_CPU) {
    place_cpu_owner(pd, Z.owner + (size_t)sc * R.U + R.unit0[j], Z.dfree + (size_t)sc * R.Dtot + R.dom0[j],
                    keep, C.cg, C.rkeep, C.cidx, C.pnode, C.poff, lane);
  } else {
    if (lane == 0) {
      int* ps = Z.pst + ((size_t)sc * P.P + j) * 2 + (pd.window_us > 0 ? 0 : 1);
      for (int i = 0; i < keep; ++i) { C.pnode[i] = 0; C.poff[i] = *ps; *ps += (C.cg[i] & 0x7f) * C.rkeep[i]; }
    }
  }
  __syncwarp();
  // start what was selected (Eq. 2: completion - arrival = waited so far + execution)
  i64 tot = 0;
  int started = 0;
  for (int i = lane; i < keep; i += 32) {
    const size_t o = row + C.cidx[i];
    const int r = C.rkeep[i];
    started += (C.cg[i] & 0x7f) * r;
    i64 act = (now - (P.a_arrival ? P.a_arrival[o] : 0)) + duration(C.cs[i], C.cp[i], r);
    if (missed && missed[i] && P.a_restore) act += clamp_param(P.a_restore[o]);   // restoration precedes execution
    P.o_alloc[o] = (C.cg[i] & 0x7f) * r; P.o_node[o] = C.pnode[i]; P.o_off[o] = C.poff[i]; P.o_act[o] = act;
    run[nr + i] = C.cidx[i];
    tot += act;
  }
  tot = warp_sum64(tot);
  busy_units += warp_sum32(started);
  if (lane == 0) { P.o_total[sc] += tot; P.o_nsel[sc] += keep; }
  nr += keep;
  __syncwarp();
  return true;
}

// Blocks of KR_THREADS threads: a scenario is a long chain of dependent steps on one warp, so the warps
// are spread over as many SMs (and schedulers) as possible instead of sharing one.
#define KR_THREADS 64
#define KR_DYN_SMEM ((KR_THREADS / 32) * (WARP_SMEM_BYTES + 320) + 16)
#define KR_STATE_MAX 16384
// ORDERED: the extended instance: the waiting queue may be kept sorted by R.policy's key and the trajectories
// pinned on arrival (R.trajectory); the plain instance keeps its registers.
template <bool ORDERED>
__global__ void __launch_bounds__(KR_THREADS, 1) k_replay(const __grid_constant__ Params P, const ReplayWs R) {
  const int lane = threadIdx.x & 31;
  const int gw = (blockIdx.x * KR_THREADS + threadIdx.x) >> 5;
  const int nw_warps = (gridDim.x * KR_THREADS) >> 5;
  for (int sc = gw; sc < P.S; sc += nw_warps) {
    const size_t row = (size_t)sc * P.N;
    const int n_act = min(max(P.n_actions[sc], 0), P.N);
    int* wait = R.wait + row; int* run = R.run + row;
    ReplayState Z;
    Z.owner = R.owner; Z.nm = R.nm; Z.dfree = R.dfree; Z.pst = R.pst; Z.win = R.win;
    if (R.state_bytes > 0) {
      // the state is small: it lives in this warp's shared memory for the whole trace
      extern __shared__ __align__(16) unsigned char k2_smem[];
      unsigned char* base = k2_smem + (KR_THREADS / 32) * (WARP_SMEM_BYTES + 320) + 16 + (size_t)(threadIdx.x >> 5) * R.state_bytes;
      const size_t o_nm = align16((size_t)R.U * 4), o_df = o_nm + align16((size_t)P.n_nodes_total + 1),
                   o_ps = o_df + align16((size_t)R.Dtot * 4), o_wn = o_ps + align16((size_t)P.P * 8);
      Z.owner = (int*)((size_t)base - (size_t)sc * R.U * 4);
      Z.nm = (u8*)((size_t)(base + o_nm) - (size_t)sc * P.n_nodes_total);
      Z.dfree = (int*)((size_t)(base + o_df) - (size_t)sc * R.Dtot * 4);
      Z.pst = (int*)((size_t)(base + o_ps) - (size_t)sc * P.P * 8);
      Z.win = (i64*)((size_t)(base + o_wn) - (size_t)sc * P.P * 8);
    }
    int* owner = Z.owner + (size_t)sc * R.U;
    u8* nm = Z.nm + (size_t)sc * P.n_nodes_total;
    int* dfree = Z.dfree + (size_t)sc * R.Dtot;
    int* occ = R.occupancy ? R.occupancy + (size_t)sc * R.max_rounds * P.P : nullptr;
    // outputs and state start empty
    for (int i = lane; i < P.N; i += 32) { P.o_alloc[row + i] = 0; P.o_node[row + i] = -1; P.o_off[row + i] = -1; P.o_act[row + i] = -1; }
    int status = 0;
    for (int i = lane; i < n_act; i += 32) {
      const int j = P.a_pool[row + i];
      int g, gang; u32 eff;
      if (j >= P.P || !decode_levels(P.pool[j], P.a_unit[row + i], P.a_mask[row + i], g, gang, eff)) status |= TG_ST_BAD_ACTION;
      for (int e = 0; e < P.n_side; ++e) {                  // further entries: a quota / concurrency pool other than j, 1 .. capacity
        const int k = P.a_side_pool[e * P.side_plane + row + i];
        if (k == 0xff) continue;
        const int c = P.a_side_units[e * P.side_plane + row + i];
        if (k >= P.P || P.pool[k < P.P ? k : 0].type != TG_POOL_API || k == j || c < 1 || c > P.pool[k < P.P ? k : 0].capacity)
          status |= TG_ST_BAD_ACTION;
      }
      if (i > 0 && P.a_arrival && P.a_arrival[row + i - 1] > P.a_arrival[row + i]) status |= TG_ST_UNSORTED;
    }
    for (int o = 16; o; o >>= 1) status |= __shfl_xor_sync(TG_FULL, status, o);
    if (status & TG_ST_BAD_ACTION) status = TG_ST_BAD_ACTION;
    for (int j = 0; j < P.P; ++j) {
      const PoolDev& pd = P.pool[j];
      if (pd.type == TG_POOL_API) { if (lane < 2) Z.pst[((size_t)sc * P.P + j) * 2 + lane] = 0; if (lane == 0) Z.win[(size_t)sc * P.P + j] = 0; continue; }
      for (int c = lane; c < pd.capacity; c += 32) {
        int v = -1;
        if (pd.type == TG_POOL_GPU && P.gpu_busy && (P.gpu_busy[(size_t)sc * P.n_nodes_total + pd.node0 + c / pd.group] >> (c % pd.group) & 1)) v = -2;
        owner[R.unit0[j] + c] = v;
      }
      if (pd.type == TG_POOL_GPU)
        for (int v = lane; v < pd.n_nodes; v += 32)
          nm[pd.node0 + v] = (P.gpu_busy ? P.gpu_busy[(size_t)sc * P.n_nodes_total + pd.node0 + v] : 0) & ((1u << pd.group) - 1u);
      if (pd.type == TG_POOL_CPU)
        for (int d = lane; d < pd.capacity / pd.group; d += 32) dfree[R.dom0[j] + d] = pd.group;
    }
    if (lane == 0) { P.o_total[sc] = 0; P.o_nsel[sc] = 0; P.o_status[sc] = status; }
    if (occ) for (int i = lane; i < R.max_rounds * P.P; i += 32) occ[i] = 0;
    __syncwarp();
    int rounds = 0;
    if (status == 0) {
      extern __shared__ __align__(16) unsigned char k2_smem[];
      int* dem = (int*)(k2_smem + (KR_THREADS / 32) * WARP_SMEM_BYTES + 16) + (threadIdx.x >> 5) * 80;   // 4 ints per pool: demand, capacity
      int* cap = dem + 32;
      int* aside = cap + 32;                              // 1 int per pool
      int* ncand = aside + 8;                             // 1 int per pool
      int next = 0, nw = 0, nr = 0, r = 0;
      bool drained = false;
      // units in use per core / GPU pool, kept up to date by what starts and what is released
      int busy[TG_MAX_POOLS];
      for (int j = 0; j < P.P; ++j) busy[j] = P.pool[j].type == TG_POOL_API ? 0 : pool_busy_units(P, R, Z, sc, j, lane);
      while (r < R.max_rounds) {
        const i64 now = (i64)r * R.round_us;
        // 1. quota refill
        for (int j = 0; j < P.P; ++j) {
          const PoolDev& pd = P.pool[j];
          if (pd.type == TG_POOL_API && pd.window_us > 0 && now / pd.window_us != Z.win[(size_t)sc * P.P + j]) {
            __syncwarp();
            if (lane == 0) { Z.win[(size_t)sc * P.P + j] = now / pd.window_us; Z.pst[((size_t)sc * P.P + j) * 2] = 0; }
            __syncwarp();
          }
        }
        // 2. release what has finished; the running list is compacted in place
        int kept = 0;
        bool gpu_released = false;
        i64 min_fin = TG_INF;                               // earliest completion among what keeps running
        for (int i0 = 0; i0 < nr; i0 += 32) {
          const int i = i0 + lane;
          int a = -1; bool done = false;
          if (i < nr) {
            a = run[i];
            const i64 fin = (P.a_arrival ? P.a_arrival[row + a] : 0) + P.o_act[row + a];
            done = fin <= now;
            if (!done) min_fin = min(min_fin, fin);
          }
          const u32 bd = __ballot_sync(TG_FULL, done), bk = __ballot_sync(TG_FULL, i < nr && !done);
          __syncwarp();
          if (i < nr && !done) run[kept + __popc(bk & ((1u << lane) - 1u))] = a;
          kept += __popc(bk);
          u32 rest = bd;
          while (rest) {
            const int b = __ffs(rest) - 1; rest &= rest - 1;
            const int fa = __shfl_sync(TG_FULL, a, b);
            const int j = P.a_pool[row + fa];
            const PoolDev& pd = P.pool[j];
            if (ORDERED && R.trajectory && R.traj_last && lane == 0 && R.traj_last[row + fa] && pd.type == TG_POOL_CPU) {
              // the trajectory's last action has ended: its memory goes back to its node
              const int t = R.trajectory[row + fa];
              if (t >= 0 && t < R.max_traj) {
                int* tn = R.traj_node + (size_t)sc * R.max_traj;
                if (tn[t] >= 0) { R.mem_free[(size_t)sc * P.P + tn[t]] += (i64)R.traj_mem[row + fa]; tn[t] = -1; }
              }
            }
            if (P.n_side > 0 && lane == 0)                 // a concurrency pool held the action's further amounts until now
              for (int e = 0; e < P.n_side; ++e) {
                const int k = P.a_side_pool[e * P.side_plane + row + fa];
                if (k != 0xff && P.pool[k].window_us == 0) Z.pst[((size_t)sc * P.P + k) * 2 + 1] -= P.a_side_units[e * P.side_plane + row + fa];
              }
            if (pd.type == TG_POOL_API) { if (pd.window_us == 0 && lane == 0) Z.pst[((size_t)sc * P.P + j) * 2 + 1] -= P.o_alloc[row + fa]; }
            else {
              const int freed = P.o_alloc[row + fa];
#pragma unroll
              for (int jj = 0; jj < TG_MAX_POOLS; ++jj) if (jj == j) busy[jj] -= freed;
              for (int c = lane; c < pd.capacity; c += 32) {
                if (owner[R.unit0[j] + c] != fa) continue;
                owner[R.unit0[j] + c] = -1;
                if (pd.type == TG_POOL_CPU) atomicAdd(&dfree[R.dom0[j] + c / pd.group], 1);
                else gpu_released = true;
              }
            }
            __syncwarp();
          }
        }
        nr = kept;
        const int nr_before = nr;
        if (__any_sync(TG_FULL, gpu_released)) {            // node masks follow the owner map
          for (int j = 0; j < P.P; ++j) {
            const PoolDev& pd = P.pool[j];
            if (pd.type != TG_POOL_GPU) continue;
            for (int v = lane; v < pd.n_nodes; v += 32) {
              u32 mk = 0;
              for (int b = 0; b < pd.group; ++b) mk |= (owner[R.unit0[j] + v * pd.group + b] != -1 ? 1u : 0u) << b;
              nm[pd.node0 + v] = (u8)mk;
            }
          }
          __syncwarp();
        }
        // 3. admit arrivals
        const int nw_admitted = nw;
        while (next < n_act) {
          const int i = next + lane;
          const bool in = i < n_act && (P.a_arrival ? P.a_arrival[row + i] : 0) <= now;
          const u32 b = __ballot_sync(TG_FULL, in);
          int cnt = (b == TG_FULL) ? 32 : __ffs(~b) - 1;              // arrivals are sorted: a prefix of the lanes
          if (ORDERED && R.trajectory && cnt > 0) {
            // per-node CPU scheduling: an arrival joins the queue once its trajectory has a node; the first one
            // that finds none waits outside, with everything that arrived after it
            __syncwarp();
            i64 mf = 0; int cores = -1;
            if (lane < P.P && P.pool[lane].type == TG_POOL_CPU) { mf = R.mem_free[(size_t)sc * P.P + lane]; cores = P.pool[lane].capacity; }
            int pool_of = 0xff;
            const int out = pin_chunk(P, R.pool_rw, row + i, lane < cnt, R.trajectory, R.traj_mem, R.max_traj,
                                      R.traj_node + (size_t)sc * R.max_traj, mf, cores, lane, pool_of);
            if (lane < P.P && cores >= 0) R.mem_free[(size_t)sc * P.P + lane] = mf;
            const int adm = min(cnt, out);
            if (lane < adm) R.pool_rw[row + i] = (u8)pool_of;
            __syncwarp();
            if (adm < cnt) {                                  // the gate: nothing behind the action without a node gets in
              if (lane < adm) wait[nw + lane] = i;
              nw += adm; next += adm;
              break;
            }
            cnt = adm;
          }
          if (lane < cnt) wait[nw + lane] = i;
          nw += cnt; next += cnt;
          if (cnt < 32) break;
        }
        __syncwarp();
        if (ORDERED && R.policy && nw > nw_admitted) {
          // Other queue orders (Section 4.2): the queue stays sorted by the policy's key, equal keys in arrival
          // order.  Each new arrival goes behind the last entry whose key is not larger; the tail moves up by one.
          u64* wkey = R.wkey + row;
          for (int x = nw_admitted; x < nw; ++x) {
            const int a = wait[x];
            int g, gang; u32 eff;
            decode_levels(P.pool[P.a_pool[row + a]], P.a_unit[row + a], P.a_mask[row + a], g, gang, eff);
            const i64 T = duration(clamp_param(P.a_s[row + a]), clamp_param(P.a_p[row + a]), __ffs(eff));
            const u64 k = R.policy == 2 ? (u64)((1ll << 42) - T) : (u64)T;
            int p = 0;
            for (int i0 = 0; i0 < x; i0 += 32) {
              const int i = i0 + lane;
              p += __popc(__ballot_sync(TG_FULL, i < x && wkey[i] <= k));
            }
            for (int hi = x; hi > p;) {
              const int lo = max(p, hi - 32), i = lo + lane;
              int va = 0; u64 vk = 0;
              if (i < hi) { va = wait[i]; vk = wkey[i]; }
              __syncwarp();
              if (i < hi) { wait[i + 1] = va; wkey[i + 1] = vk; }
              __syncwarp();
              hi = lo;
            }
            if (lane == 0) { wait[p] = a; wkey[p] = k; }
            __syncwarp();
          }
        }
        // 4. schedule
        int blocked_pool = -1;                              // pool of a head-of-line action that does not fit
        if (nw > 0) {
          const int n = replay_prefix(P, R, Z, sc, wait, nw, dem, cap, aside, ncand, lane);
          if (n == 0 && P.n_side == 0 && !(ORDERED && R.trajectory)) blocked_pool = P.a_pool[row + wait[0]];   // (a pin made later would see other free memory)
          const int nr0 = nr;
          bool ok = true;
          if (n > 0)
            for (int j = 0; j < P.P && ok; ++j) {
              if (ncand[j] == 0) continue;                  // no candidate has this pool as its key pool
              int add = 0;
              ok = replay_pool(P, R, Z, sc, j, wait, nw, n, run, nr, now, warp_slab(P, gw), lane, add, aside[j], ncand[j]);
#pragma unroll
              for (int jj = 0; jj < TG_MAX_POOLS; ++jj) if (jj == j) busy[jj] += add;
            }
          if (!ok) { if (lane == 0) P.o_status[sc] |= TG_ST_WORKSPACE; break; }
          if (P.n_side > 0 && nr > nr0) {                   // the started actions consume their further amounts
            __syncwarp();
            for (int i = nr0 + lane; i < nr; i += 32)
              for (int e = 0; e < P.n_side; ++e) {
                const int k = P.a_side_pool[e * P.side_plane + row + run[i]];
                if (k != 0xff)
                  atomicAdd(&Z.pst[((size_t)sc * P.P + k) * 2 + (P.pool[k].window_us > 0 ? 0 : 1)],
                            (int)P.a_side_units[e * P.side_plane + row + run[i]]);
              }
            __syncwarp();
          }
          if (nr > nr0) {                                   // drop the started actions from the queue
            int kw = 0;
            for (int i0 = 0; i0 < nw; i0 += 32) {
              const int i = i0 + lane;
              int a = -1; bool stay = false;
              u64 kk = 0;
              if (i < nw) { a = wait[i]; stay = P.o_act[row + a] < 0; if (ORDERED && R.policy) kk = R.wkey[row + i]; }
              const u32 b = __ballot_sync(TG_FULL, stay);
              __syncwarp();
              if (stay) { wait[kw + __popc(b & ((1u << lane) - 1u))] = a; if (ORDERED && R.policy) R.wkey[row + kw + __popc(b & ((1u << lane) - 1u))] = kk; }
              kw += __popc(b);
            }
            nw = kw;
            __syncwarp();
          }
        }
        // 5. occupancy of this round
        for (int j = 0; j < P.P; ++j) if (P.pool[j].type == TG_POOL_API) busy[j] = pool_busy_units(P, R, Z, sc, j, lane);
        if (occ && lane == 0) for (int j = 0; j < P.P; ++j) occ[(size_t)r * P.P + j] = busy[j];
        ++r;
        if (next == n_act && nw == 0 && nr == 0) { drained = true; break; }
        // with an empty queue nothing happens before the next arrival or completion: jump there
        if (nw == 0) {
          // (what was running before this round: the release scan's minimum; what started in it: the tail of the list)
          i64 t_next = next < n_act ? (P.a_arrival ? P.a_arrival[row + next] : 0) : TG_INF;
          t_next = min(t_next, min_fin);
          for (int i = nr_before + lane; i < nr; i += 32) {
            const int a = run[i];
            t_next = min(t_next, (P.a_arrival ? P.a_arrival[row + a] : 0) + P.o_act[row + a]);
          }
          t_next = warp_min64(t_next);
          i64 r_next = (t_next + R.round_us - 1) / R.round_us;
          if (r_next > R.max_rounds) r_next = R.max_rounds;
          // skipped rounds repeat this occupancy, except that quota usage restarts with its window
          for (i64 rr = r + lane; rr < r_next; rr += 32)
            for (int j = 0; j < P.P; ++j) {
              const PoolDev& pd = P.pool[j];
              int v = busy[j];
              if (pd.type == TG_POOL_API && pd.window_us > 0 && (rr * R.round_us) / pd.window_us != Z.win[(size_t)sc * P.P + j]) v = 0;
              if (occ) occ[(size_t)rr * P.P + j] = v;
            }
          if (r_next > r) r = (int)r_next;
        } else if (blocked_pool >= 0) {
          // The action at the head of the queue does not fit its pool, so nothing can start (the prefix is
          // empty) until that pool changes: an action running on it ends, or its quota window turns.  The
          // rounds up to then only admit arrivals behind the head and release what ends on other pools;
          // their occupancy rows follow from the completion times.
          const PoolDev& hp = P.pool[blocked_pool];
          i64 t_next = TG_INF;
          if (hp.type == TG_POOL_API && hp.window_us > 0) t_next = (Z.win[(size_t)sc * P.P + blocked_pool] + 1) * (i64)hp.window_us;
          // (in a sorted queue an arrival with a smaller key becomes the head)
          if (ORDERED && next < n_act) t_next = min(t_next, P.a_arrival ? P.a_arrival[row + next] : 0);
          for (int i = lane; i < nr; i += 32) {
            const int a = run[i];
            if (P.a_pool[row + a] == blocked_pool) t_next = min(t_next, (P.a_arrival ? P.a_arrival[row + a] : 0) + P.o_act[row + a]);
          }
          t_next = warp_min64(t_next);
          i64 r_next = t_next == TG_INF ? (i64)R.max_rounds : (t_next + R.round_us - 1) / R.round_us;
          if (r_next > R.max_rounds) r_next = R.max_rounds;
          if (r_next > r) {
            if (occ) {
              for (i64 rr = r + lane; rr < r_next; rr += 32)
                for (int j = 0; j < P.P; ++j) {
                  const PoolDev& pd = P.pool[j];
                  int v = busy[j];
                  if (pd.type == TG_POOL_API && pd.window_us > 0 && (rr * R.round_us) / pd.window_us != Z.win[(size_t)sc * P.P + j]) v = 0;
                  occ[(size_t)rr * P.P + j] = v;
                }
              __syncwarp();
              // what ends on the other pools inside the jump leaves the rows from its round on
              for (int i = lane; i < nr; i += 32) {
                const int a = run[i];
                const int j = P.a_pool[row + a];
                const PoolDev& pd = P.pool[j];
                if (pd.type == TG_POOL_API && pd.window_us > 0) continue;      // used quota is not given back
                const i64 fin = (P.a_arrival ? P.a_arrival[row + a] : 0) + P.o_act[row + a];
                i64 fr = (fin + R.round_us - 1) / R.round_us;
                if (fr < r) fr = r;
                for (i64 rr = fr; rr < r_next; ++rr) atomicSub(&occ[(size_t)rr * P.P + j], P.o_alloc[row + a]);
              }
              __syncwarp();
            }
            r = (int)r_next;
          }
        }
      }
      rounds = drained ? r : R.max_rounds;
      if (!drained && r < R.max_rounds) rounds = r;
    }
    if (R.rounds_used && lane == 0) R.rounds_used[sc] = rounds;
    __syncwarp();
  }
}
