// Completion-heap simulations of Algorithm 2 (estimate).
//
// A round needs, per elastic (scenario, pool), the objective of the full candidate list and of
// the list without its last candidate (the first eviction step).  Each is a sequential
// simulation of |waiting| "pop the earliest completion ts, push ts + T" steps.
//
// One simulation per prefix is enough although Algorithm 2 tries `depth` levels of the first
// waiting action and keeps the best: if one multiset of completion times is elementwise <=
// another, it stays so after a step with the same T and every popped time is <=, so the
// estimate is non-decreasing in the first action's duration; durations do not grow with the
// level, hence the best depth is always the largest level tried.
//
// The priority queue is a winner tree of packed keys: every node of an implicit tree over H slots
// (4-ary, see tree_sim) holds the smallest key of its subtree, key = completion << 12 | slot.
// Replacing the minimum only touches the path from its leaf to the root, and the siblings on
// that path are known from the leaf alone, so their loads are all issued at once and only a
// chain of integer minima remains sequential (an fp64 fmin on the same bits was measured
// slower on this part).
// One lane runs one simulation; a warp's 32 trees live in shared memory interleaved by lane
// (node n of lane t at n * 32 + t, conflict free).  Shared memory bounds how many simulations
// are resident, so what matters is the latency of a step, not the number of warps.
// A completion time that would not fit 49 value bits sends the simulation to the exact
// 64-bit kernel below.
//
// Work distribution: k_sim_classify sorts groups of 32 consecutive simulations (same pool,
// neighbouring scenarios, hence similar H) into capacity classes; one persistent kernel per
// class, sized to fill the GPU at that class's shared-memory footprint, pulls groups from its
// list.  Classes run concurrently on side streams.  k_sims_big (trees in the arena) takes what
// is too large for shared memory or overflowed the packing.
#pragma once
#include "common.cuh"

#define SIM_PER_WARP 32         // simulations per warp
#define SIM_SLOT_BITS 12
#define SIM_VALUE_LIMIT (1LL << 49)

// per (scenario, pool) state handed from the solve kernel to the simulations and the finish kernel
struct TaskState {
  i64 opt[2];     // optimal duration sum of all m candidates / of the first m-1
  i64 est[2];     // estimate of the rest for those two prefixes
  int flags;      // TS_* bits
  int pad;
};
#define TS_SOLVED 1   // both prefixes solved, heap seeds written
#define TS_FAILED 2   // workspace too small
#define TS_REDO0 4    // simulation of prefix e overflowed the packed keys: bit TS_REDO0 << e
#define TS_DECIDED 16 // placed and written by the solve kernel: no estimate needed

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

// simulation index = (pool * S + scenario) * 2 + e
__device__ __forceinline__ int sim_slots(const Params& P, const TaskState* ts, long long sim) {
  if (sim >= (long long)P.P * P.S * 2) return 0;
  const int e = (int)(sim & 1);
  const long long x = sim >> 1;
  const int sc = (int)(x % P.S), j = (int)(x / P.S);
  const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
  if (!(mt.elastic && mt.m >= 1 + e && (e + mt.count - mt.m) > 0)) return 0;
  if (!(ts[(size_t)sc * P.P + j].flags & TS_SOLVED)) return 0;
  return mt.m - e;
}

__device__ __forceinline__ SimJob sim_job(const Params& P, TaskState* ts, const i64* seed2, long long sim) {
  SimJob J;
  J.active = false; J.H = 0; J.n_list = 0; J.e = 0; J.seeds = nullptr; J.lst = nullptr; J.first_dur = 0; J.st = nullptr;
  if (sim >= (long long)P.P * P.S * 2) return J;
  const int e = (int)(sim & 1);
  const long long x = sim >> 1;
  const int sc = (int)(x % P.S), j = (int)(x / P.S);
  const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
  J.st = ts + (size_t)sc * P.P + j;
  J.e = e;
  const int n_ac = mt.count - mt.m;
  if (!(mt.elastic && mt.m >= 1 + e && (e + n_ac) > 0 && (J.st->flags & TS_SOLVED))) return J;
  const size_t row = (size_t)sc * P.N;
  const PoolDev& pd = P.pool[j];
  // first remaining action: the evicted last candidate (e = 1) or the first waiting one; it takes
  // the largest of its first `depth` levels (see the header for why that depth is the best)
  const int idx = e ? P.order[row + mt.cbase + mt.m - 1] : mt.first_wait;
  int g, gang; u32 fm;
  decode_levels(pd, P.a_unit[row + idx], P.a_mask[row + idx], g, gang, fm);
  const int d = min(P.depth, __popc(fm)) - 1;
  J.active = true;
  J.first_dur = duration(clamp_param(P.a_s[row + idx]), clamp_param(P.a_p[row + idx]), nth_level_of(fm, d));
  J.H = mt.m - e;
  J.seeds = e ? seed2 + row + mt.cbase : P.tmin + row + mt.base;
  J.lst = P.tmin + row + mt.base + mt.m + (1 - e);
  J.n_list = n_ac - (1 - e);
  return J;
}

// work lists of the capacity classes
struct SimLists {
  int* count;      // [n_classes] groups appended; count[63]: something is left for k_sims_big
  int* cursor;     // [n_classes] groups taken
  int* list;       // [n_classes][n_groups]
  int n_groups, n_classes;
  int cap[32];     // capacity (slots) of every class, ascending; a group goes to the first that fits
};

// one warp per group, one lane per simulation
__global__ void k_sim_classify(const __grid_constant__ Params P, const TaskState* ts, const SimLists L) {
  const long long sim = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int g = (int)(sim / SIM_PER_WARP);
  if (g >= L.n_groups) return;
  const int hmax = warp_max32(sim_slots(P, ts, sim));
  if (hmax == 0 || (threadIdx.x & 31) != 0) return;
  int c = 0;
  while (c < L.n_classes && hmax > L.cap[c]) ++c;
  if (c == L.n_classes) { L.count[63] = 1; return; }  // beyond shared memory: k_sims_big takes it
  const int pos = atomicAdd(&L.count[c], 1);
  L.list[(size_t)c * L.n_groups + pos] = g;
}

__device__ __forceinline__ i64 key_min(i64 a, i64 b) { return b < a ? b : a; }

__device__ __forceinline__ i64 lds64(u32 addr) {
  i64 v;
  asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts64(u32 addr, i64 v) {
  asm volatile("st.shared.b64 [%0], %1;" :: "r"(addr), "l"(v) : "memory");
}

// nodes of the 4-ary winner tree over H slots: I internal nodes (every one with four children),
// then 3 I + 1 leaves of which the first H are the slots and the rest hold +inf
__host__ __device__ __forceinline__ int tree_internal(int H) { return (H + 1) / 3; }
__host__ __device__ __forceinline__ int tree_nodes(int H) { return 4 * tree_internal(H) + 1; }

// One whole simulation on a 4-ary winner tree in shared memory, run by the calling lane alone.
// Node n (root 0, children of n: 4n+1 .. 4n+4, slot s = node I + s) is at shared address
// base + (n << SS).  MAXD bounds the number of levels below the root.  seed(i) gives slot i's
// first completion, dur(k) the duration of the k-th remaining action, k = 0 .. steps-1.
// Replacing the minimum walks from its leaf to the root; the node indices of that path follow
// from the leaf alone, so the three siblings of every level are loaded at once, their minimum
// is taken off the critical path, and one minimum per level remains sequential.
// Returns the estimate (saturating sum of completions); *overflow tells that a completion
// reached 2^49 and the packed keys cannot be trusted.
template <int MAXD, int SS, class SeedFn, class DurFn>
__device__ __forceinline__ i64 tree_sim(u32 base, int H, int steps, SeedFn seed, DurFn dur, bool* overflow) {
  const int I = tree_internal(H), T = 4 * I + 1;
  for (int i = 0; i < T - I; ++i) sts64(base + ((u32)(I + i) << SS), i < H ? ((seed(i) << SIM_SLOT_BITS) | i) : TG_INF);
  for (int n = I - 1; n >= 0; --n) {
    const u32 c0 = base + ((u32)(4 * n + 1) << SS);
    sts64(base + ((u32)n << SS), key_min(key_min(lds64(c0), lds64(c0 + (1u << SS))),
                                         key_min(lds64(c0 + (2u << SS)), lds64(c0 + (3u << SS)))));
  }
  i64 top = lds64(base);                               // key of the earliest completion
  i64 tmp = 0;
  u32 ovf = 0;
  // durations are fetched a chunk of four ahead
  i64 cur[4], nxt[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) cur[x] = x < steps ? dur(x) : 0;
  for (int k0 = 0; k0 < steps; k0 += 4) {
#pragma unroll
    for (int x = 0; x < 4; ++x) nxt[x] = (k0 + 4 + x < steps) ? dur(k0 + 4 + x) : 0;
    i64 chunk = 0;                                     // four completions < 2^51: no overflow here
#pragma unroll
    for (int x4 = 0; x4 < 4; ++x4) {
      if (k0 + x4 < steps) {
        const u32 w = (u32)top & ((1u << SIM_SLOT_BITS) - 1u);
        i64 c = top + (cur[x4] << SIM_SLOT_BITS);      // pop earliest completion ts, push ts + T (same slot)
        chunk += c >> SIM_SLOT_BITS;
        ovf |= (u32)(c >> 32);
        int n = I + (int)w;
        sts64(base + ((u32)n << SS), c);
        // siblings' minimum and parent of every level of the path
        i64 sm[MAXD]; u32 pa[MAXD]; bool on[MAXD];
#pragma unroll
        for (int x = 0; x < MAXD; ++x) {
          on[x] = n > 0;
          const int nn = on[x] ? n : 1;                // beyond the root: a harmless read of node 1's group
          const int g = ((nn - 1) & ~3) + 1, k = (nn - 1) & 3;
          const i64 s1 = lds64(base + ((u32)(g + ((k + 1) & 3)) << SS));
          const i64 s2 = lds64(base + ((u32)(g + ((k + 2) & 3)) << SS));
          const i64 s3 = lds64(base + ((u32)(g + ((k + 3) & 3)) << SS));
          sm[x] = key_min(s1, key_min(s2, s3));
          n = (nn - 1) >> 2;
          pa[x] = base + ((u32)n << SS);
        }
#pragma unroll
        for (int x = 0; x < MAXD; ++x) {
          if (on[x]) { c = key_min(c, sm[x]); sts64(pa[x], c); }
        }
        top = c;
      }
    }
    tmp = sat_add(tmp, chunk);
#pragma unroll
    for (int x = 0; x < 4; ++x) cur[x] = nxt[x];
  }
  *overflow = (ovf >> 29) != 0;                        // a completion >= 2^49
  return tmp;
}

// The same simulation on a binary winner tree (more shared memory, fewer instructions per
// step): for the single simulations of continued evictions, where latency is all that counts.
// Node n is at shared address base + (n << SS); base must be a multiple of 2 << SS plus an offset
// below 1 << SS, so that with o = n << SS the sibling of a node is at (base + o) ^ (1 << SS) and
// the node offsets of a leaf-to-root path are (leaf offset >> level) & ~((1 << SS) - 1).
// MAXD bounds the path length (2 * H <= 2^(MAXD+1)).  seed(i) gives slot i's first completion,
// dur(k) the duration of the k-th remaining action, k = 0 .. steps-1.  Returns the estimate
// (saturating sum of completions); *overflow tells that a completion reached 2^49 and the
// packed keys cannot be trusted.
template <int MAXD, int SS, class SeedFn, class DurFn>
__device__ __forceinline__ i64 tree_sim2(u32 base, int H, int steps, SeedFn seed, DurFn dur, bool* overflow) {
  const u32 NM = ~((1u << SS) - 1u);
  for (int i = 0; i < H; ++i) sts64(base + ((u32)(H + i) << SS), (seed(i) << SIM_SLOT_BITS) | i);
  for (int n = H - 1; n >= 1; --n)
    sts64(base + ((u32)n << SS), key_min(lds64(base + ((u32)(2 * n) << SS)), lds64(base + ((u32)(2 * n + 1) << SS))));
  i64 top = lds64(base + ((u32)(H > 1 ? 1 : H) << SS));   // key of the earliest completion
  i64 tmp = 0;
  u32 ovf = 0;
  // durations are fetched a chunk of four ahead
  i64 cur[4], nxt[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) cur[x] = x < steps ? dur(x) : 0;
  for (int k0 = 0; k0 < steps; k0 += 4) {
#pragma unroll
    for (int x = 0; x < 4; ++x) nxt[x] = (k0 + 4 + x < steps) ? dur(k0 + 4 + x) : 0;
    i64 chunk = 0;                                     // four completions < 2^51: no overflow here
#pragma unroll
    for (int x4 = 0; x4 < 4; ++x4) {
      if (k0 + x4 < steps) {
        const u32 w = (u32)top & ((1u << SIM_SLOT_BITS) - 1u);
        const i64 v = (top >> SIM_SLOT_BITS) + cur[x4];       // pop earliest, push ts + T
        chunk += v;
        ovf |= (u32)(v >> 32);
        i64 c = (v << SIM_SLOT_BITS) | (i64)w;
        const u32 o0 = ((u32)H + w) << SS;             // byte offset of the leaf
        sts64(base + o0, c);
        i64 sk[MAXD]; u32 pa[MAXD];
#pragma unroll
        for (int x = 0; x < MAXD; ++x) {
          pa[x] = base + ((o0 >> (x + 1)) & NM);       // parent of the level-x node
          const u32 cu = base + ((o0 >> x) & NM);      // the level-x node itself
          sk[x] = lds64(cu ^ (1u << SS));              // its sibling (a harmless read beyond the root)
        }
#pragma unroll
        for (int x = 0; x < MAXD; ++x) {
          if ((o0 >> (x + SS + 1)) != 0) {             // level-x node is not the root: n >= 2
            c = key_min(c, sk[x]);
            sts64(pa[x], c);
          }
        }
        top = c;
      }
    }
    tmp = sat_add(tmp, chunk);
#pragma unroll
    for (int x = 0; x < 4; ++x) cur[x] = nxt[x];
  }
  *overflow = (ovf >> 17) != 0;                        // a completion >= 2^49
  return tmp;
}

// One simulation run by a whole warp: for the single simulations of continued evictions, where
// the latency of a step is all that counts.  Slot i lives in lane i & 31, register i >> 5
// (H <= 32 * NS).  A step takes the minimum of the packed keys with two 32-bit warp reductions
// (high words, then low words among the lanes that tie on the high word); the lane that owns
// the winning slot replaces it.  Durations are loaded 32 steps at a time, one per lane.
// Same result and overflow rule as tree_sim2.
template <int NS, class SeedFn, class DurFn>
__device__ __forceinline__ i64 warp_sim(int H, int steps, SeedFn seed, DurFn dur, int lane, bool* overflow) {
  u64 key[NS];
#pragma unroll
  for (int j = 0; j < NS; ++j) {
    const int i = j * 32 + lane;
    key[j] = i < H ? (((u64)seed(i) << SIM_SLOT_BITS) | (u64)i) : ~0ull;
  }
  i64 total = 0;
  u32 ovf = 0;
  for (int k0 = 0; k0 < steps; k0 += 32) {
    const i64 mine = k0 + lane < steps ? dur(k0 + lane) : 0;
    const int nb = min(32, steps - k0);
    i64 chunk = 0;                                       // 32 completions < 2^49 each
    for (int b = 0; b < nb; ++b) {
      const i64 d = __shfl_sync(TG_FULL, mine, b);
      u64 lm = key[0];
#pragma unroll
      for (int j = 1; j < NS; ++j) lm = key[j] < lm ? key[j] : lm;
      const u32 hi = (u32)(lm >> 32);
      const u32 mhi = __reduce_min_sync(TG_FULL, hi);
      const u32 mlo = __reduce_min_sync(TG_FULL, hi == mhi ? (u32)lm : 0xffffffffu);
      const u64 top = ((u64)mhi << 32) | mlo;            // earliest completion and its slot
      const u64 c = top + ((u64)d << SIM_SLOT_BITS);     // pop it, push ts + T into the same slot
      chunk += (i64)(c >> SIM_SLOT_BITS);
      ovf |= (u32)(c >> (32 + SIM_SLOT_BITS));
      const u32 slot = mlo & ((1u << SIM_SLOT_BITS) - 1u);
      if (lane == (int)(slot & 31u)) {
#pragma unroll
        for (int j = 0; j < NS; ++j) if (j == (int)(slot >> 5)) key[j] = c;
      }
    }
    total = sat_add(total, chunk);
  }
  *overflow = (ovf >> 17) != 0;                          // a completion >= 2^49
  return total;
}

// One simulation run by a whole warp on a SORTED array of completion times spread over the lanes:
// position i lives in lane i & 31, register i >> 5 (H <= 32 * NS), unused positions hold
// 0xffffffff.  "Pop the earliest, push earliest + T" removes position 0 and inserts the new time
// where it belongs: every lane compares its elements with it, one vote per register counts the
// smaller ones, and the elements in front of that place move down one position (a rotation by one
// lane per register, which does not depend on the new time and is issued ahead).  The two earliest
// times are also kept in every lane, so that the next completion is known a few instructions after
// the step starts; no reduction sits on the path from step to step.
// Keys are 32-bit completion times saturated at SORTED_SAT (about 71 minutes); the sum of
// completions is exact: the popped keys are exact as long as none of them is saturated, and the
// durations are summed apart, 32 at a time.  A saturated key that gets popped sets *overflow: the
// caller then uses an exact 64-bit simulation.
#define SORTED_SAT 0xfffffffeu
template <int NS>
__device__ __forceinline__ void sorted_replace_min(u32 (&key)[NS], u32 c, int lane) {
  int lt = 0;
#pragma unroll
  for (int r = 0; r < NS; ++r) lt += __popc(__ballot_sync(TG_FULL, key[r] < c));
  const int cnt = max(lt - 1, 0);                        // where c goes once position 0 is gone
  u32 rot[NS + 1];
#pragma unroll
  for (int r = 0; r < NS; ++r) rot[r] = __shfl_sync(TG_FULL, key[r], (lane + 1) & 31);
  rot[NS] = 0xffffffffu;
#pragma unroll
  for (int r = 0; r < NS; ++r) {
    const int pos = r * 32 + lane;
    const u32 next = lane < 31 ? rot[r] : rot[r + 1];    // the element one position behind
    key[r] = pos < cnt ? next : (pos == cnt ? c : key[r]);
  }
}
__device__ __forceinline__ u32 sorted_key(i64 v) { return v >= (i64)SORTED_SAT ? SORTED_SAT : (u32)v; }

template <int NS, class SeedFn, class DurFn>
__device__ __forceinline__ i64 sorted_sim(int H, int steps, SeedFn seed, DurFn dur, int lane, bool* overflow) {
  u32 key[NS];
  // start from H zeros (no seed is smaller) and replace them by the seeds one by one
#pragma unroll
  for (int r = 0; r < NS; ++r) key[r] = r * 32 + lane < H ? 0u : 0xffffffffu;
  for (int i0 = 0; i0 < H; i0 += 32) {
    const u32 mine = i0 + lane < H ? sorted_key(seed(i0 + lane)) : 0u;
    const int nb = min(32, H - i0);
    for (int b = 0; b < nb; ++b) sorted_replace_min<NS>(key, __shfl_sync(TG_FULL, mine, b), lane);
  }
  u32 t0 = __shfl_sync(TG_FULL, key[0], 0), t1 = __shfl_sync(TG_FULL, key[0], 1);
  i64 total = 0;
  bool ovf = false;
  for (int k0 = 0; k0 < steps; k0 += 32) {
    const i64 mine = k0 + lane < steps ? dur(k0 + lane) : 0;
    const u32 mine32 = sorted_key(mine);
    const int nb = min(32, steps - k0);
    u64 pops = 0;                                        // 32 popped keys below 2^32 each
    for (int b = 0; b < nb; ++b) {
      const u32 d = __shfl_sync(TG_FULL, mine32, b);
      const u32 b2 = __shfl_sync(TG_FULL, key[0], 2);    // the third earliest time
      ovf |= t0 >= SORTED_SAT;                           // the popped key is not an exact time any more
      pops += t0;
      const u64 c64 = (u64)t0 + d;                       // pop the earliest completion ts, push ts + T
      const u32 c = c64 >= SORTED_SAT ? SORTED_SAT : (u32)c64;
      sorted_replace_min<NS>(key, c, lane);
      const bool lt1 = t1 < c, lt2 = b2 < c;
      t0 = lt1 ? t1 : c;
      t1 = lt1 ? (lt2 ? b2 : c) : t1;
    }
    total = sat_add(total, (i64)pops + warp_sum64(mine));  // completions = popped times + durations
  }
  *overflow = ovf;
  return total;
}

// One persistent warp per block, one lane per simulation (trees interleaved by lane: SS = 8).
template <int MAXD>
__global__ void __launch_bounds__(32) k_sims1(const __grid_constant__ Params P, TaskState* ts, const i64* seed2,
                                              const SimLists L, int cls) {
  extern __shared__ __align__(16) unsigned char sim_smem[];
  const int lane = threadIdx.x;
  const u32 base = (u32)__cvta_generic_to_shared(sim_smem) + (u32)lane * 8u;   // 16-byte aligned, no padding: it would cost a resident block
  const int count = L.count[cls];
  for (;;) {
    int gi = 0;
    if (lane == 0) gi = atomicAdd(&L.cursor[cls], 1);
    gi = __shfl_sync(TG_FULL, gi, 0);
    if (gi >= count) break;
    const int grp = L.list[(size_t)cls * L.n_groups + gi];
    const SimJob J = sim_job(P, ts, seed2, (long long)grp * SIM_PER_WARP + lane);
    if (!J.active) continue;                           // lanes are independent: no warp-wide step below
    bool overflow;
    const i64 tmp = tree_sim<MAXD, 8>(
        base, J.H, J.n_list + 1, [&](int i) { return J.seeds[i]; },
        [&](int k) { return k == 0 ? J.first_dur : J.lst[k - 1]; }, &overflow);
    if (overflow) { atomicOr(&J.st->flags, TS_REDO0 << J.e); L.count[63] = 1; }
    else J.st->est[J.e] = tmp;
  }
}

// One lane per simulation, exact 64-bit values, trees in the arena: for H beyond the largest
// shared-memory class and for simulations whose packed keys overflowed.
__global__ void __launch_bounds__(32) k_sims_big(const __grid_constant__ Params P, TaskState* ts,
                                                 const i64* seed2, int hcap_lo, const int* any_big) {
  if (*any_big == 0) return;
  const int t = threadIdx.x;
  SimJob J = sim_job(P, ts, seed2, (long long)blockIdx.x * 32 + t);
  if (J.active && !(J.H > hcap_lo || (J.st->flags & (TS_REDO0 << J.e)))) J.active = false;
  const int hmax = warp_max32(J.active ? J.H : 0);
  if (hmax == 0) return;
  u64 off = 0;
  const u64 bytes = ((u64)hmax * 32 * (sizeof(i64) + 2 * sizeof(u32)) + 255) & ~(u64)255;
  if (t == 0) off = atomicAdd(P.arena_top, bytes);
  off = __shfl_sync(TG_FULL, off, 0) + arena_bump_base(P);                   // bump part of the arena
  if (off + bytes > P.arena_bytes) { if (J.active) atomicOr(&J.st->flags, TS_FAILED); return; }
  if (!J.active) return;
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
  J.st->est[J.e] = tmp;
}
