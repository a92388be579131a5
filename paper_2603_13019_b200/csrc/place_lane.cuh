// Placement of a batched round, one THREAD per (scenario, pool).  Placement is a short
// sequential loop over the kept candidates whose state is tiny (free cores per NUMA domain,
// one busy byte per GPU node), so 32 pools per warp instruction beat one pool per warp.
// The solve and finish kernels leave, per kept candidate in queue order, its unit byte and
// multiplicity (Params::preq) and the number kept (Params::keepn); this kernel applies the
// same rules as place.cuh (Sections 5.1-5.3) and writes place_node / place_off.
// Per-thread state lives in shared memory, byte v of thread t at v * KPL_THREADS + t.
#pragma once
#include "common.cuh"
#include "place.cuh"

#define KPL_THREADS 128
#define KPL_STATE 128       // state bytes per thread: NUMA domains of a core pool, nodes of a GPU pool
#define KPL_BATCH 8         // kept candidates whose request and index are loaded at once
#define KPL_LOAD_BATCH(i0)                                                     \
  u32 vq[KPL_BATCH]; int vo[KPL_BATCH];                                        \
  _Pragma("unroll") for (int b_ = 0; b_ < KPL_BATCH; ++b_) {                   \
    const bool on_ = (i0) + b_ < keep;                                         \
    vq[b_] = on_ ? rq[(i0) + b_] : 0u;                                         \
    vo[b_] = on_ ? ord[(i0) + b_] : 0;                                         \
  }

__global__ void __launch_bounds__(KPL_THREADS) k_place(const __grid_constant__ Params P) {
  __shared__ u8 sm[KPL_STATE * KPL_THREADS];
  const int x = blockIdx.x * KPL_THREADS + threadIdx.x;
  if (x >= P.S * P.P) return;
  const int sc = x % P.S, j = P.pool_order[x / P.S];     // a warp holds 32 scenarios of one pool
  const PoolDev& pd = P.pool[j];
  if (!pd.lane_place) return;
  const int keep = P.keepn[(size_t)sc * P.P + j];
  if (keep <= 0) return;
  const size_t row = (size_t)sc * P.N;
  const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
  const unsigned short* rq = P.preq + row + mt.base;
  const int* ord = P.order + row + mt.base;
  u8* st = sm + threadIdx.x;

  if (pd.type == TG_POOL_API) {                           // Section 5.1: offset = units consumed before
    int used = 0;
    for (int i0 = 0; i0 < keep; i0 += KPL_BATCH) {
      KPL_LOAD_BATCH(i0);
#pragma unroll
      for (int b = 0; b < KPL_BATCH; ++b) {
        if (i0 + b >= keep) break;
        const u32 v = vq[b];
        const size_t o = row + vo[b];
        P.o_node[o] = 0; P.o_off[o] = used;
        used += (int)(v & 0x7fu) * (int)(v >> 8);
      }
    }
    return;
  }

  if (pd.type == TG_POOL_CPU) {
    // Section 5.2 on a pool nobody occupies yet: cores are taken lowest id first, so the free
    // count per domain is the whole state; domains at or beyond `frontier` are untouched.
    const int G = pd.group, D = pd.capacity / G;
    int frontier = 0;
    for (int i0 = 0; i0 < keep; i0 += KPL_BATCH) {
      KPL_LOAD_BATCH(i0);
#pragma unroll
      for (int b = 0; b < KPL_BATCH; ++b) {
        if (i0 + b >= keep) break;
        const u32 v = vq[b];
        const int k = (int)(v & 0x7fu) * (int)(v >> 8);
        int best = -1, bf = INT_MAX;
        for (int d0 = 0; d0 < frontier; d0 += 8) {        // best fit: fewest free cores that still fit
          int f[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) f[u] = d0 + u < frontier ? (int)st[(d0 + u) * KPL_THREADS] : 0;
#pragma unroll
          for (int u = 0; u < 8; ++u) if (f[u] >= k && f[u] < bf) { bf = f[u]; best = d0 + u; }
        }
        if (best < 0 && frontier < D && G >= k) { best = frontier++; bf = G; }
        int first = -1, dom = -1;
        if (best >= 0) {
          first = best * G + (G - bf); dom = best;
          st[best * KPL_THREADS] = (u8)(bf - k);
        } else {                                          // no domain fits: ascending domains
          int need = k;
          for (int d = 0; d < D && need > 0; ++d) {
            const int f = d < frontier ? st[d * KPL_THREADS] : G;
            if (f == 0) continue;
            if (first < 0) { first = d * G + (G - f); dom = d; }
            const int take = min(f, need);
            st[d * KPL_THREADS] = (u8)(f - take);
            need -= take;
            if (d >= frontier) frontier = d + 1;
          }
        }
        const size_t o = row + vo[b];
        P.o_node[o] = dom; P.o_off[o] = first;
      }
    }
    return;
  }

  // Section 5.3: requests by size descending, then queue position; each takes the smallest
  // sufficient maximal free block, lowest (node, start), and the low end of a split block.
  // lv[l]: nodes that hold a maximal free block of 2^l GPUs.
  const int top = ilog2(pd.group), n_nodes = pd.n_nodes;
  const u32 pad = (~((1u << pd.group) - 1u)) & 0xffu;
  const u8* busy_row = P.gpu_busy ? P.gpu_busy + (size_t)sc * P.n_nodes_total + pd.node0 : nullptr;
  u64 lv[4] = {0, 0, 0, 0};
  for (int n = 0; n < n_nodes; ++n) {
    const u32 b = (busy_row ? busy_row[n] : 0u) | pad;
    st[n * KPL_THREADS] = (u8)b;
    const u32 lev = node_levels(b);
#pragma unroll
    for (int l = 0; l < 4; ++l) lv[l] |= (u64)((lev >> l) & 1u) << n;
  }
  for (int lz = top; lz >= 0; --lz) {
    const int z = 1 << lz;
    for (int i0 = 0; i0 < keep; i0 += KPL_BATCH) {
      KPL_LOAD_BATCH(i0);
#pragma unroll
      for (int bb = 0; bb < KPL_BATCH; ++bb) {
        if (i0 + bb >= keep) break;
        const u32 v = vq[bb];
        const int g = v & 0x7f, gang = (v >> 7) & 1, ri = v >> 8;
        const int nreq = gang ? (g * ri == z ? 1 : 0) : (g == z ? ri : 0);
        for (int rep = 0; rep < nreq; ++rep) {
          int bl = lz;
          u64 mask = 0;
          for (; bl <= top; ++bl) {
            mask = bl == 0 ? lv[0] : (bl == 1 ? lv[1] : (bl == 2 ? lv[2] : lv[3]));
            if (mask) break;
          }
          if (!mask) continue;                            // cannot happen: the selection fits
          const int node = __ffsll((long long)mask) - 1;
          u32 b = st[node * KPL_THREADS];
          const int start = node_block_start(b, bl);
          b |= ((1u << z) - 1u) << start;
          st[node * KPL_THREADS] = (u8)b;
          const u32 lev = node_levels(b);
          const u64 bit = 1ull << node;
#pragma unroll
          for (int l = 0; l < 4; ++l) lv[l] = (lv[l] & ~bit) | ((u64)((lev >> l) & 1u) << node);
          if (rep == 0) {
            const size_t o = row + vo[bb];
            P.o_node[o] = node; P.o_off[o] = start;
          }
        }
      }
    }
  }
}
