// Completion-heap simulations of Algorithm 2 (estimate).
//
// A round needs, per elastic (scenario, pool), the objective of the full candidate list and of
// the list without its last candidate (the first eviction step), each at `depth` levels of the
// first waiting action: 2 * depth independent sequential simulations of |waiting| "pop the
// earliest completion, push completion + duration" steps.
//
// The priority queue of a simulation is a winner tree over its H slots: slot values val[0..H)
// and, for every internal node n = 1..H-1 of the implicit tree (leaf i = node H+i), the slot
// holding the subtree's minimum.  Replacing the minimum only touches the path from its leaf to
// the root, and the siblings on that path are known from the leaf alone.  FOUR LANES share one
// simulation: each lane loads the siblings of its 2-3 levels, a two-step prefix-minimum over
// the four lanes yields the winner entering every level, each lane stores its levels' winners.
// A warp thus runs 8 simulations with a short dependent chain per step, and four times as
// many warps are resident for the same shared memory as with one lane per simulation (the
// trees' shared-memory footprint, not registers, limits residency).
//
// Work distribution: k_sim_classify sorts groups of 8 consecutive simulations (same pool,
// neighbouring scenarios, hence similar H) into capacity classes; one persistent kernel per
// class, sized to fill the GPU at that class's shared-memory footprint, pulls groups from its
// list.  Classes run concurrently on side streams.  Trees too large for shared memory are
// simulated one lane each in the arena (k_sims_big).
#pragma once
#include "common.cuh"

#define SIM_G 4                 // lanes per simulation
#define SIM_PER_WARP 8          // simulations per warp (32 / SIM_G)
#define SIM_SLOT_BYTES 10       // shared memory per slot: i64 value + u16 node
typedef unsigned short u16;

// per (scenario, pool) state handed from the solve kernel to the simulations and the finish kernel
struct TaskState {
  i64 opt[2];     // optimal duration sum of all m candidates / of the first m-1
  i64 est[2];     // estimate of the rest for those two prefixes: min over depths (atomicMin)
  int flags;      // TS_* bits
  int pad;
};
#define TS_SOLVED 1   // both prefixes solved, heap seeds written
#define TS_FAILED 2   // workspace too small

__device__ __forceinline__ int nth_level_of(u32 mask, int d) {
  for (int k = 0; k < d; ++k) mask &= mask - 1;
  return __ffs(mask);
}

struct SimJob {
  bool active;
  int H, n_list, e;
  const i64* seeds; const i64* lst;
  i64 first_dur;
  TaskState* st;
};

// number of slots of simulation `sim` (0 if it does not exist); cheap, for classification
__device__ __forceinline__ int sim_slots(const Params& P, const TaskState* ts, long long sim) {
  const long long n_sims = (long long)P.P * P.S * 2 * P.depth;
  if (sim >= n_sims) return 0;
  long long x = sim / P.depth;
  const int e = (int)(x & 1); x >>= 1;
  const int sc = (int)(x % P.S), j = (int)(x / P.S);
  const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
  if (!(mt.elastic && mt.m >= 1 + e && (e + mt.count - mt.m) > 0)) return 0;
  if (!(ts[(size_t)sc * P.P + j].flags & TS_SOLVED)) return 0;
  return mt.m - e;
}

__device__ __forceinline__ SimJob sim_job(const Params& P, TaskState* ts, const i64* seed2, long long sim) {
  SimJob J;
  J.active = false; J.H = 0; J.n_list = 0; J.e = 0; J.seeds = nullptr; J.lst = nullptr; J.first_dur = 0; J.st = nullptr;
  const long long n_sims = (long long)P.P * P.S * 2 * P.depth;
  if (sim >= n_sims) return J;
  const int d = (int)(sim % P.depth);
  long long x = sim / P.depth;
  const int e = (int)(x & 1); x >>= 1;
  const int sc = (int)(x % P.S), j = (int)(x / P.S);
  const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
  J.st = ts + (size_t)sc * P.P + j;
  J.e = e;
  const int n_ac = mt.count - mt.m;
  if (!(mt.elastic && mt.m >= 1 + e && (e + n_ac) > 0 && (J.st->flags & TS_SOLVED))) return J;
  const size_t row = (size_t)sc * P.N;
  const PoolDev& pd = P.pool[j];
  // first remaining action: the evicted last candidate (e = 1) or the first waiting one
  const int idx = P.order[row + mt.base + mt.m - e];
  int g, gang; u32 fm;
  decode_levels(pd, P.a_unit[row + idx], P.a_mask[row + idx], g, gang, fm);
  if (d >= min(P.depth, __popc(fm))) return J;
  J.active = true;
  J.first_dur = duration(clamp_param(P.a_s[row + idx]), clamp_param(P.a_p[row + idx]), nth_level_of(fm, d));
  J.H = mt.m - e;
  J.seeds = (e ? seed2 : P.tmin) + row + mt.base;
  J.lst = P.tmin + row + mt.base + mt.m + (1 - e);
  J.n_list = n_ac - (1 - e);
  return J;
}

// work lists of the capacity classes
struct SimLists {
  int* count;      // [n_classes] groups appended
  int* cursor;     // [n_classes] groups taken
  int* list;       // [n_classes][n_groups]
  int n_groups, n_classes;
  int cap[32];     // capacity (slots) of every class, ascending; a group goes to the first that fits
};

__global__ void k_sim_classify(const __grid_constant__ Params P, const TaskState* ts, const SimLists L) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= L.n_groups) return;
  int hmax = 0;
  for (int s = 0; s < SIM_PER_WARP; ++s) hmax = max(hmax, sim_slots(P, ts, (long long)g * SIM_PER_WARP + s));
  if (hmax == 0) return;
  int c = 0;
  while (c < L.n_classes && hmax > L.cap[c]) ++c;
  if (c == L.n_classes) { L.count[63] = 1; return; }  // beyond shared memory: k_sims_big takes it
  const int pos = atomicAdd(&L.count[c], 1);
  L.list[(size_t)c * L.n_groups + pos] = g;
}

struct Key { i64 v; int i; };
__device__ __forceinline__ Key key_min(Key a, Key b) { return b.v < a.v ? b : a; }

// position of element e of simulation s inside a warp's arrays (swizzled against bank conflicts)
__device__ __forceinline__ int sim_at(int e, int s) { return e * SIM_PER_WARP + ((s + e) & (SIM_PER_WARP - 1)); }

// One persistent warp per block; LPL = tree levels per lane (4 * LPL >= path length of the class).
template <int LPL>
__global__ void __launch_bounds__(32) k_sims4(const __grid_constant__ Params P, TaskState* ts, const i64* seed2,
                                              const SimLists L, int cls) {
  extern __shared__ __align__(16) unsigned char sim_smem[];
  const int hcap = L.cap[cls];
  i64* val = (i64*)sim_smem;
  u16* tree = (u16*)(sim_smem + (size_t)hcap * SIM_PER_WARP * sizeof(i64));
  const int lane = threadIdx.x, q = lane & (SIM_G - 1), s = lane >> 2;
  const int count = L.count[cls];
  for (;;) {
    int gi = 0;
    if (lane == 0) gi = atomicAdd(&L.cursor[cls], 1);
    gi = __shfl_sync(TG_FULL, gi, 0);
    if (gi >= count) break;
    const int grp = L.list[(size_t)cls * L.n_groups + gi];
    const SimJob J = sim_job(P, ts, seed2, (long long)grp * SIM_PER_WARP + s);
    const int H = J.H;
    __syncwarp();
    if (J.active) {
      for (int i = q; i < H; i += SIM_G) val[sim_at(i, s)] = J.seeds[i];
    }
    __syncwarp();
    if (J.active && q == 0) {
      for (int n = H - 1; n >= 1; --n) {
        int ca = 2 * n, cb = 2 * n + 1;
        int a = ca >= H ? ca - H : (int)tree[sim_at(ca, s)];
        int b = cb >= H ? cb - H : (int)tree[sim_at(cb, s)];
        tree[sim_at(n, s)] = (u16)(val[sim_at(b, s)] < val[sim_at(a, s)] ? b : a);
      }
    }
    __syncwarp();
    int w = 0; i64 wv = 0;
    if (J.active) { w = H > 1 ? (int)tree[sim_at(1, s)] : 0; wv = val[sim_at(w, s)]; }
    const int steps = J.active ? J.n_list + 1 : 0;
    const int kmax = warp_max32(steps);
    i64 tmp = 0;
    i64 d0 = J.first_dur;
    i64 d1 = J.n_list > 0 ? J.lst[0] : 0, d2 = J.n_list > 1 ? J.lst[1] : 0;
    for (int k = 0; k < kmax; ++k) {
      const bool live = k < steps;
      i64 d3 = (live && k + 2 < J.n_list) ? J.lst[k + 2] : 0;       // durations fetched three steps ahead
      const i64 v = wv + d0;                                         // pop earliest completion, push ts + T
      if (live) tmp = sat_add(tmp, v);
      const int n0 = H + w;
      if (live && q == 0) val[sim_at(w, s)] = v;
      // siblings of this lane's levels
      Key sk[LPL]; int par[LPL];
#pragma unroll
      for (int x = 0; x < LPL; ++x) {
        const int n = n0 >> (q * LPL + x);
        par[x] = (live && n >= 2) ? (n >> 1) : 0;
        sk[x].v = TG_INF; sk[x].i = 0;
        if (par[x]) {
          const int sb = n ^ 1;
          sk[x].i = sb >= H ? sb - H : (int)tree[sim_at(sb, s)];
        }
      }
#pragma unroll
      for (int x = 0; x < LPL; ++x) if (par[x]) sk[x].v = val[sim_at(sk[x].i, s)];
      // minimum over this lane's levels, then exclusive prefix-minimum over the lanes below it
      Key lm = sk[0];
#pragma unroll
      for (int x = 1; x < LPL; ++x) lm = key_min(lm, sk[x]);
      Key pm = lm;
#pragma unroll
      for (int off = 1; off < SIM_G; off <<= 1) {
        Key o;
        o.v = __shfl_up_sync(TG_FULL, pm.v, off, SIM_G);
        o.i = __shfl_up_sync(TG_FULL, pm.i, off, SIM_G);
        if (q >= off) pm = key_min(pm, o);
      }
      Key ex;
      ex.v = __shfl_up_sync(TG_FULL, pm.v, 1, SIM_G);
      ex.i = __shfl_up_sync(TG_FULL, pm.i, 1, SIM_G);
      Key c; c.v = v; c.i = w;
      if (q > 0) c = key_min(c, ex);
      // winners of this lane's levels, bottom up
#pragma unroll
      for (int x = 0; x < LPL; ++x) {
        if (par[x]) {
          c = key_min(c, sk[x]);
          tree[sim_at(par[x], s)] = (u16)c.i;
        }
      }
      // the top lane holds the new overall winner
      const i64 nv = __shfl_sync(TG_FULL, c.v, SIM_G - 1, SIM_G);
      const int ni = __shfl_sync(TG_FULL, c.i, SIM_G - 1, SIM_G);
      if (live) { wv = nv; w = ni; }
      d0 = d1; d1 = d2; d2 = d3;
      __syncwarp();
    }
    if (J.active && q == 0) atomicMin((u64*)&J.st->est[J.e], (u64)tmp);
  }
}

// One lane per simulation, trees in the arena: for H beyond the largest shared-memory class.
__global__ void __launch_bounds__(32) k_sims_big(const __grid_constant__ Params P, TaskState* ts,
                                                 const i64* seed2, int hcap_lo, const int* any_big) {
  if (*any_big == 0) return;
  const int t = threadIdx.x;
  const SimJob J = sim_job(P, ts, seed2, (long long)blockIdx.x * 32 + t);
  const int hmax = warp_max32(J.active ? J.H : 0);
  if (hmax <= hcap_lo) return;
  u64 off = 0;
  const u64 bytes = ((u64)hmax * 32 * (sizeof(i64) + 2 * sizeof(u32)) + 255) & ~(u64)255;
  if (t == 0) off = atomicAdd(P.arena_top, bytes);
  off = __shfl_sync(TG_FULL, off, 0);
  if (off + bytes > P.arena_bytes) { if (J.active) atomicOr(&J.st->flags, TS_FAILED); return; }
  if (!J.active || J.H <= hcap_lo) return;
  i64* val = (i64*)(P.arena + off);
  u32* tree = (u32*)(P.arena + off + (u64)hmax * 32 * sizeof(i64));
  const int H = J.H;
  for (int i = 0; i < H; ++i) {
    val[(size_t)i * 32 + t] = J.seeds[i];
    tree[(size_t)(H + i) * 32 + t] = (u32)i;
  }
  for (int n = H - 1; n >= 1; --n) {
    u32 a = tree[(size_t)(2 * n) * 32 + t], b = tree[(size_t)(2 * n + 1) * 32 + t];
    tree[(size_t)n * 32 + t] = val[(size_t)b * 32 + t] < val[(size_t)a * 32 + t] ? b : a;
  }
  int w = H > 1 ? (int)tree[32 + t] : 0;
  i64 wv = val[(size_t)w * 32 + t];
  i64 tmp = 0;
  i64 dur = J.first_dur;
  for (int k = 0; k <= J.n_list; ++k) {
    i64 nxt = k < J.n_list ? J.lst[k] : 0;
    i64 v = wv + dur;
    tmp = sat_add(tmp, v);
    val[(size_t)w * 32 + t] = v;
    int ci = w; i64 cv = v;
    for (int n = H + w; n >= 2; n >>= 1) {
      int sb = (int)tree[(size_t)(n ^ 1) * 32 + t];
      i64 x = val[(size_t)sb * 32 + t];
      if (x < cv) { cv = x; ci = sb; }
      tree[(size_t)(n >> 1) * 32 + t] = (u32)ci;
    }
    w = ci; wv = cv;
    dur = nxt;
  }
  atomicMin((u64*)&J.st->est[J.e], (u64)tmp);
}
