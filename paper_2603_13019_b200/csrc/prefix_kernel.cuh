// Kernel 1 of a round: one CTA per scenario.
//   - evaluates the duration model at each action's least level (Eq. 1),
//   - finds the candidate prefix: the longest queue prefix whose least-required units fit
//     every pool, nested chunk capacities included (Algorithm 1, line 2),
//   - splits the queue by pool (Algorithm 1, line 4): a stable partition whose positions are
//     written to the workspace, candidates of a pool first,
//   - writes the "not scheduled" outputs of everything behind the prefix.
#pragma once
#include "common.cuh"

#define K1_THREADS 256
#define K1_ITEMS 16
#define K1_TILE (K1_THREADS * K1_ITEMS)

// exclusive scan of every column sm[v][0..255] across the CTA, continuing from carry[v]
__device__ __forceinline__ void k1_scan_columns(int* sm, int* carry, int V, int lane, int warp) {
  for (int v = warp; v < V; v += K1_THREADS / 32) {
    int* col = sm + v * K1_THREADS;
    int x[8], sum = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = col[lane * 8 + k];
#pragma unroll
    for (int k = 0; k < 8; ++k) { int tv = x[k]; x[k] = sum; sum += tv; }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(TG_FULL, incl, o); if (lane >= o) incl += y; }
    int excl = incl - sum + carry[v];
#pragma unroll
    for (int k = 0; k < 8; ++k) col[lane * 8 + k] = x[k] + excl;
    int total = __shfl_sync(TG_FULL, incl, 31);
    __syncwarp();
    if (lane == 0) carry[v] += total;
  }
}

__global__ void __launch_bounds__(K1_THREADS) k_prefix(const __grid_constant__ Params P) {
  extern __shared__ int sm[];                       // [V][K1_THREADS] scan columns
  __shared__ int s_cap[4 * TG_MAX_POOLS];           // capacity of every demand slot
  __shared__ int s_carry[5 * TG_MAX_POOLS];
  __shared__ int s_tot[TG_MAX_POOLS], s_base[TG_MAX_POOLS], s_m[TG_MAX_POOLS];
  __shared__ int s_n, s_bad, s_el;

  const int sc = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const size_t row = (size_t)sc * P.N;
  const int n_act = min(max(P.n_actions[sc], 0), P.N);
  const int D = P.V - P.P;                          // demand slots come first, then one count slot per pool

  if (t < TG_MAX_POOLS) { s_tot[t] = 0; s_m[t] = 0; }
  if (t < 5 * TG_MAX_POOLS) s_carry[t] = 0;
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

  // pass A: actions per pool (gives the partition bases)
  for (int i0 = warp * 32; i0 < n_act; i0 += K1_THREADS) {
    int i = i0 + lane;
    int pj = i < n_act ? (int)P.a_pool[row + i] : 255;
    for (int j = 0; j < P.P; ++j) {
      u32 b = __ballot_sync(TG_FULL, pj == j);
      if (lane == 0 && b) atomicAdd(&s_tot[j], __popc(b));
    }
    if (i < n_act && pj >= P.P) s_bad = 1;
  }
  __syncthreads();
  if (t == 0) { int acc = 0; for (int j = 0; j < P.P; ++j) { s_base[j] = acc; acc += s_tot[j]; } }
  __syncthreads();

  if (!s_bad) {
    for (int tile0 = 0; tile0 < n_act; tile0 += K1_TILE) {
      for (int v = 0; v < P.V; ++v) sm[v * K1_THREADS + t] = 0;
      const bool found_before = s_n != INT_MAX;
      // info: bits 0-3 pool, 4 present, 5 elastic, 6-7 chunk level, 8-20 least units
      u32 info[K1_ITEMS];
      i64 tm[K1_ITEMS];
      const int i_first = tile0 + t * K1_ITEMS;
#pragma unroll
      for (int k = 0; k < K1_ITEMS; ++k) {
        int i = i_first + k;
        info[k] = 0; tm[k] = 0;
        if (i < n_act) {
          int j = P.a_pool[row + i];
          const PoolDev& pd = P.pool[j];
          int g, gang; u32 eff;
          if (!decode_levels(pd, P.a_unit[row + i], P.a_mask[row + i], g, gang, eff)) { s_bad = 1; continue; }
          int rmin = __ffs(eff);
          int units = g * rmin;
          int lz = pd.type == TG_POOL_GPU ? level_of(g, gang, rmin) : 0;
          info[k] = (u32)j | 16u | ((eff & (eff - 1)) ? 32u : 0u) | ((u32)lz << 6) | ((u32)units << 8);
          tm[k] = duration(clamp_param(P.a_s[row + i]), clamp_param(P.a_p[row + i]), rmin);
          sm[(D + j) * K1_THREADS + t] += 1;
          if (!found_before)
            for (int l = 0; l <= lz; ++l) sm[(pd.slot0 + l) * K1_THREADS + t] += units;
        }
      }
      __syncthreads();
      k1_scan_columns(sm, s_carry, P.V, lane, warp);
      __syncthreads();
      if (!found_before) {
        // walk the thread's items in queue order; first item that overflows a slot ends the prefix
#pragma unroll
        for (int k = 0; k < K1_ITEMS; ++k) {
          if (!(info[k] & 16u)) continue;
          int j = info[k] & 15, lz = (info[k] >> 6) & 3, units = (info[k] >> 8) & 0x1fff;
          const PoolDev& pd = P.pool[j];
          bool over = false;
          for (int l = 0; l <= lz; ++l) {
            int d = (sm[(pd.slot0 + l) * K1_THREADS + t] += units);
            over |= d > s_cap[pd.slot0 + l];
          }
          if (over) atomicMin(&s_n, i_first + k);
        }
      }
      __syncthreads();
      const int n = min(s_n, n_act);
#pragma unroll
      for (int k = 0; k < K1_ITEMS; ++k) {
        if (!(info[k] & 16u)) continue;
        int i = i_first + k, j = info[k] & 15;
        int pos = sm[(D + j) * K1_THREADS + t]++;
        size_t part = row + s_base[j] + pos;
        P.order[part] = i;
        P.tmin[part] = tm[k];
        if (i < n) {
          atomicAdd(&s_m[j], 1);
          if (info[k] & 32u) atomicOr(&s_el, 1 << j);
        } else {
          P.o_alloc[row + i] = 0; P.o_node[row + i] = -1; P.o_off[row + i] = -1; P.o_act[row + i] = -1;
        }
      }
      __syncthreads();
    }
  }
  __syncthreads();
  const bool bad = s_bad != 0;
  // rows never looked at (beyond the scenario's queue), or everything of a bad scenario
  for (int i = (bad ? 0 : n_act) + t; i < P.N; i += K1_THREADS) {
    P.o_alloc[row + i] = 0; P.o_node[row + i] = -1; P.o_off[row + i] = -1; P.o_act[row + i] = -1;
  }
  if (t < P.P) {
    PoolMeta mt;
    mt.base = s_base[t]; mt.count = bad ? 0 : s_tot[t]; mt.m = bad ? 0 : s_m[t];
    mt.elastic = (s_el >> t) & 1;
    P.meta[(size_t)sc * P.P + t] = mt;
  }
  if (t == 0) { P.o_status[sc] = bad ? TG_ST_BAD_ACTION : 0; P.o_total[sc] = 0; P.o_nsel[sc] = 0; }
}
