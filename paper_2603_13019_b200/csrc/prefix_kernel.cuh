// Kernel 1 of a round: one CTA per scenario.
//   - evaluates the duration model at each action's least level (Eq. 1),
//   - finds the candidate prefix: the longest queue prefix whose least-required units fit
//     every pool, nested chunk capacities included (Algorithm 1, line 2),
//   - splits the queue by pool (Algorithm 1, line 4): a stable partition whose positions are
//     written to the workspace, candidates of a pool first,
//   - writes the "not scheduled" outputs of everything behind the prefix.
//
// A thread owns 16 consecutive actions of a tile of 4096 (128-bit loads of the structure-of-
// arrays records, 128-bit stores of the outputs).  Per pool it counts actions and sums the
// least-level demand per chunk level in its own shared-memory column; an exclusive scan of
// every column over the CTA (shuffles within a warp, warp totals through shared memory)
// turns these into running totals, which the thread then advances action by action: the first
// action whose pool overflows a level ends the prefix, the running count is the action's
// position inside its pool.
#pragma once
#include "common.cuh"

#define K1_THREADS 256
#define K1_ITEMS 16
#define K1_TILE (K1_THREADS * K1_ITEMS)
#define K1_MAXV (5 * TG_MAX_POOLS)

// exclusive scan over the CTA of every column sm[v][thread], continuing from carry[v];
// afterwards carry[v] holds the total including this tile.  wsum: [8][K1_MAXV] scratch.
__device__ __forceinline__ void k1_scan_columns(int* sm, int* carry, int* wsum, int V, int t) {
  const int lane = t & 31, warp = t >> 5;
  for (int v = 0; v < V; ++v) {
    int x = sm[v * K1_THREADS + t], incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(TG_FULL, incl, o); if (lane >= o) incl += y; }
    if (lane == 31) wsum[warp * K1_MAXV + v] = incl;
    sm[v * K1_THREADS + t] = incl - x;                 // exclusive within the warp
  }
  __syncthreads();
  if (t < V) {                                         // warp totals -> offsets of the warps, new carry
    int acc = carry[t];
    for (int w = 0; w < K1_THREADS / 32; ++w) { int x = wsum[w * K1_MAXV + t]; wsum[w * K1_MAXV + t] = acc; acc += x; }
    carry[t] = acc;
  }
  __syncthreads();
  for (int v = 0; v < V; ++v) sm[v * K1_THREADS + t] += wsum[warp * K1_MAXV + v];
}

__global__ void __launch_bounds__(K1_THREADS) k_prefix(const __grid_constant__ Params P) {
  extern __shared__ int sm[];                       // [V][K1_THREADS] scan columns
  __shared__ int s_cap[4 * TG_MAX_POOLS];           // capacity of every demand slot
  __shared__ int s_carry[K1_MAXV];
  __shared__ int s_wsum[(K1_THREADS / 32) * K1_MAXV];
  __shared__ int s_tot[TG_MAX_POOLS], s_base[TG_MAX_POOLS], s_m[TG_MAX_POOLS];
  __shared__ int s_n, s_bad, s_el;
  __shared__ u32 s_pinfo[TG_MAX_POOLS];             // type | GPUs per node << 4 | slot0 << 8

  const int sc = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const size_t row = (size_t)sc * P.N;
  const int n_act = min(max(P.n_actions[sc], 0), P.N);
  const int D = P.V - P.P;                          // demand slots come first, then one count slot per pool
  const bool one_tile = n_act <= K1_TILE;
  // 128-bit accesses need 16-byte aligned rows
  const bool vec = (P.N % 16 == 0) &&
                   ((((size_t)P.a_pool | (size_t)P.a_unit | (size_t)P.a_mask | (size_t)P.a_s | (size_t)P.a_p |
                      (size_t)P.o_alloc | (size_t)P.o_node | (size_t)P.o_off | (size_t)P.o_act) & 15) == 0);

  if (t < TG_MAX_POOLS) {
    s_tot[t] = 0; s_m[t] = 0; s_base[t] = 0;
    s_pinfo[t] = t < P.P ? (u32)P.pool[t].type | ((u32)(P.pool[t].type == TG_POOL_GPU ? P.pool[t].group : 0) << 4) |
                                ((u32)P.pool[t].slot0 << 8) : 0u;
  }
  if (t < K1_MAXV) s_carry[t] = 0;
  if (t == 0) { s_n = INT_MAX; s_bad = 0; s_el = 0; }
  if (warp < P.P) {                                 // free capacity of every demand slot
    const PoolDev& pd = P.pool[warp];
    if (pd.type == TG_POOL_GPU) {
      int cap[4];
      gpu_caps(pd, P.gpu_busy ? P.gpu_busy + (size_t)sc * P.n_nodes_total : nullptr, lane, cap);
      if (lane < 4) s_cap[pd.slot0 + lane] = cap[lane];
    } else if (lane == 0) s_cap[pd.slot0] = pd.capacity;
  }
  __syncthreads();

  // queues longer than a tile: count the actions per pool first (gives the partition bases)
  if (!one_tile) {
    for (int i0 = warp * 32; i0 < n_act; i0 += K1_THREADS) {
      int i = i0 + lane;
      int pj = i < n_act ? (int)P.a_pool[row + i] : 255;
      for (int j = 0; j < P.P; ++j) {
        u32 b = __ballot_sync(TG_FULL, pj == j);
        if (lane == 0 && b) atomicAdd(&s_tot[j], __popc(b));
      }
    }
    __syncthreads();
    if (t == 0) { int acc = 0; for (int j = 0; j < P.P; ++j) { s_base[j] = acc; acc += s_tot[j]; } }
    __syncthreads();
  }

  for (int tile0 = 0; tile0 < n_act; tile0 += K1_TILE) {
    for (int v = 0; v < P.V; ++v) sm[v * K1_THREADS + t] = 0;
    const bool found_before = s_n != INT_MAX;
    // info: bits 0-3 pool, 4 present, 5 elastic, 6-7 chunk level, 8-20 least units
    u32 info[K1_ITEMS];
    i64 tm[K1_ITEMS];
    const int i_first = tile0 + t * K1_ITEMS;
    const bool full = vec && i_first + K1_ITEMS <= n_act;
    u8 rp[K1_ITEMS], ru[K1_ITEMS];
    u32 rm[K1_ITEMS];
    if (full) {
      *(uint4*)rp = *(const uint4*)(P.a_pool + row + i_first);
      *(uint4*)ru = *(const uint4*)(P.a_unit + row + i_first);
#pragma unroll
      for (int k = 0; k < K1_ITEMS; k += 4) *(uint4*)(rm + k) = *(const uint4*)(P.a_mask + row + i_first + k);
    } else {
#pragma unroll
      for (int k = 0; k < K1_ITEMS; ++k) {
        const int i = i_first + k;
        rp[k] = i < n_act ? P.a_pool[row + i] : 0;
        ru[k] = i < n_act ? P.a_unit[row + i] : 0;
        rm[k] = i < n_act ? P.a_mask[row + i] : 0;
      }
    }
    bool bad = false;
#pragma unroll
    for (int k = 0; k < K1_ITEMS; k += 2) {
      i64 sv[2], pv[2];
      if (full) {
        *(longlong2*)sv = *(const longlong2*)(P.a_s + row + i_first + k);
        *(longlong2*)pv = *(const longlong2*)(P.a_p + row + i_first + k);
      } else {
        for (int h = 0; h < 2; ++h) {
          const int i = i_first + k + h;
          sv[h] = i < n_act ? P.a_s[row + i] : 0;
          pv[h] = i < n_act ? P.a_p[row + i] : 0;
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int kk = k + h, i = i_first + kk;
        info[kk] = 0; tm[kk] = 0;
        if (i < n_act) {
          const int j = rp[kk];
          if (j >= P.P) { bad = true; continue; }
          const u32 pi = s_pinfo[j];
          PoolDev pd;
          pd.type = pi & 15; pd.group = (pi >> 4) & 15;
          const int slot0 = pi >> 8;
          int g, gang; u32 eff;
          if (!decode_levels(pd, ru[kk], rm[kk], g, gang, eff)) { bad = true; continue; }
          const int rmin = __ffs(eff);
          const int units = g * rmin;
          const int lz = pd.type == TG_POOL_GPU ? level_of(g, gang, rmin) : 0;
          info[kk] = (u32)j | 16u | ((eff & (eff - 1)) ? 32u : 0u) | ((u32)lz << 6) | ((u32)units << 8);
          tm[kk] = duration(clamp_param(sv[h]), clamp_param(pv[h]), rmin);
          sm[(D + j) * K1_THREADS + t] += 1;
          if (!found_before)
            for (int l = 0; l <= lz; ++l) sm[(slot0 + l) * K1_THREADS + t] += units;
        }
      }
    }
    if (bad) s_bad = 1;
    __syncthreads();
    k1_scan_columns(sm, s_carry, s_wsum, P.V, t);
    __syncthreads();
    if (one_tile && t == 0) {                        // the scan's totals are the pool sizes
      int acc = 0;
      for (int j = 0; j < P.P; ++j) { s_tot[j] = s_carry[D + j]; s_base[j] = acc; acc += s_tot[j]; }
    }
    if (!found_before && !s_bad) {
      // walk the thread's items in queue order; first item that overflows a slot ends the prefix
#pragma unroll
      for (int k = 0; k < K1_ITEMS; ++k) {
        if (!(info[k] & 16u)) continue;
        const int j = info[k] & 15, lz = (info[k] >> 6) & 3, units = (info[k] >> 8) & 0x1fff;
        const int slot0 = s_pinfo[j] >> 8;
        bool over = false;
        for (int l = 0; l <= lz; ++l) {
          int d = (sm[(slot0 + l) * K1_THREADS + t] += units);
          over |= d > s_cap[slot0 + l];
        }
        if (over) atomicMin(&s_n, i_first + k);
      }
    }
    __syncthreads();
    if (s_bad) break;
    const int n = min(s_n, n_act);
    // a pool needs its partition (positions and least-level durations) only if the selection
    // runs on it, i.e. one of its candidates is elastic; queues longer than a tile may learn
    // that too late, so they always write it
    u32 el_mask = 0;
#pragma unroll
    for (int k = 0; k < K1_ITEMS; ++k)
      if ((info[k] & 48u) == 48u && i_first + k < n) el_mask |= 1u << (info[k] & 15);
    if (el_mask) atomicOr(&s_el, (int)el_mask);
    __syncthreads();
    const u32 need = one_tile ? (u32)s_el : 0xffu;
#pragma unroll
    for (int k = 0; k < K1_ITEMS; ++k) {
      if (!(info[k] & 16u)) continue;
      const int i = i_first + k, j = info[k] & 15;
      const int pos = sm[(D + j) * K1_THREADS + t]++;
      const size_t part = row + s_base[j] + pos;
      if (i < n) {
        P.order[part] = i;
        atomicAdd(&s_m[j], 1);
      } else if ((need >> j) & 1u) {
        P.tmin[part] = tm[k];
        // the first waiting action of a pool is looked up by position; it sits right behind the
        // pool's candidates, whose count is final only now for this tile, so every waiting
        // action of a needed pool records its index (4 bytes) - cheap next to its duration
        P.order[part] = i;
      }
    }
    // "not scheduled" outputs of everything behind the prefix (candidates are written later)
    if (full && i_first >= n) {
      const int4 z = make_int4(0, 0, 0, 0), m1 = make_int4(-1, -1, -1, -1);
      const longlong2 a1 = make_longlong2(-1, -1);
#pragma unroll
      for (int k = 0; k < K1_ITEMS; k += 4) {
        *(int4*)(P.o_alloc + row + i_first + k) = z;
        *(int4*)(P.o_node + row + i_first + k) = m1;
        *(int4*)(P.o_off + row + i_first + k) = m1;
      }
#pragma unroll
      for (int k = 0; k < K1_ITEMS; k += 2) *(longlong2*)(P.o_act + row + i_first + k) = a1;
    } else {
#pragma unroll
      for (int k = 0; k < K1_ITEMS; ++k) {
        const int i = i_first + k;
        if ((info[k] & 16u) && i >= n) {
          P.o_alloc[row + i] = 0; P.o_node[row + i] = -1; P.o_off[row + i] = -1; P.o_act[row + i] = -1;
        }
      }
    }
    __syncthreads();
  }
  __syncthreads();
  const bool bad = s_bad != 0;
  // rows never looked at (beyond the scenario's queue), or everything of a bad scenario
  for (int i = (bad ? 0 : n_act) + t; i < P.N; i += K1_THREADS) {
    P.o_alloc[row + i] = 0; P.o_node[row + i] = -1; P.o_off[row + i] = -1; P.o_act[row + i] = -1;
  }
  if (t < P.P) {
    PoolMeta mt;
    mt.base = s_base[t]; mt.cbase = s_base[t]; mt.count = bad ? 0 : s_tot[t]; mt.m = bad ? 0 : s_m[t];
    mt.elastic = (s_el >> t) & 1;
    // waiting actions of a pool whose selection runs recorded their index behind the candidates
    mt.first_wait = (!bad && mt.elastic && mt.count > mt.m) ? P.order[row + s_base[t] + s_m[t]] : -1;
    P.meta[(size_t)sc * P.P + t] = mt;
  }
  if (t == 0) { P.o_status[sc] = bad ? TG_ST_BAD_ACTION : 0; P.o_total[sc] = 0; P.o_nsel[sc] = 0; }
}
