// Placement of a batched round, one THREAD per (scenario, pool).  Placement is a short
// sequential loop over the kept candidates whose state is tiny (free cores per NUMA domain,
// one busy byte per GPU node), so 32 pools per warp instruction beat one pool per warp.
// The solve and finish kernels leave, per kept candidate in queue order, its unit byte and
// multiplicity (Params::preq) and the number kept (Params::keepn); this kernel applies the
// same rules as place.cuh (Sections 5.1-5.3) and writes place_node / place_off.
//
// A warp holds 32 scenarios of one pool.  Its threads would touch 32 different rows with every
// load and store, so candidates go through shared memory 32 at a time: for each of the 32
// scenarios the warp loads that scenario's next 32 requests and indices with one coalesced
// access each, every thread then places its own scenario's 32 candidates, and the results are
// written back scenario by scenario.  Shared memory per warp: per-thread state (byte v of lane t
// at v * 32 + t) and the staged chunk (entry c of lane t at c * 33 + t).
#pragma once
#include "common.cuh"
#include "place.cuh"
#include "prefix_stream.cuh"

#define KPL_WARPS 2
#define KPL_THREADS (32 * KPL_WARPS)
#define KPL_DOMAINS 128     // NUMA domains of a core pool at most (two state bytes each); a GPU pool has at most 64 nodes
#define KPL_STATE (2 * KPL_DOMAINS)
#define KPL_NONE (-2)       // staged result of a candidate that this pass did not place

struct KplWarp {
  u8 state[KPL_STATE * 32];
  unsigned short rq[32 * 33];
  int idx[32 * 33];
  int off[32 * 33];
  short node[32 * 33];
};

// stage requests and indices [c0, c0 + 32) of all 32 scenarios of the warp (sixteen scenarios'
// loads in flight at once)
__device__ __forceinline__ void kpl_load(KplWarp& W, const unsigned short* rq, const int* ord, int keep, int c0, int lane) {
  for (int s0 = 0; s0 < 32; s0 += 16) {
    unsigned short vq[16]; int vo[16]; bool on[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int ks = __shfl_sync(TG_FULL, keep, s0 + u);
      const unsigned short* rs = (const unsigned short*)__shfl_sync(TG_FULL, (unsigned long long)rq, s0 + u);
      const int* os = (const int*)__shfl_sync(TG_FULL, (unsigned long long)ord, s0 + u);
      on[u] = c0 + lane < ks;
      vq[u] = on[u] ? rs[c0 + lane] : (unsigned short)0;
      vo[u] = on[u] ? os[c0 + lane] : 0;
    }
#pragma unroll
    for (int u = 0; u < 16; ++u)
      if (on[u]) { W.rq[lane * 33 + s0 + u] = vq[u]; W.idx[lane * 33 + s0 + u] = vo[u]; }
  }
  __syncwarp();
}
// write the staged results of candidates [c0, c0 + 32) of all 32 scenarios
__device__ __forceinline__ void kpl_store(const Params& P, KplWarp& W, size_t row, int keep, int c0, int lane) {
  __syncwarp();
#pragma unroll 8
  for (int s = 0; s < 32; ++s) {
    const int ks = __shfl_sync(TG_FULL, keep, s);
    const size_t rs = (size_t)__shfl_sync(TG_FULL, (unsigned long long)row, s);
    if (c0 + lane < ks) {
      const int nd = W.node[lane * 33 + s];
      if (nd != KPL_NONE) {
        const size_t o = rs + W.idx[lane * 33 + s];
        P.o_node[o] = nd; P.o_off[o] = W.off[lane * 33 + s];
      }
    }
  }
  __syncwarp();
}

// phase 0: the pools that the head kernel certified (decided by k_easy); phase 1: all the others, and
// the cleaning up behind scenarios with an invalid record.
// GPU pools of at most 128 nodes whose selection went through the solver: one WARP per (scenario, pool).
// The node masks live in lane registers and "lowest node with a free block of this size" is one warp
// reduction (place_gpu_reg's rule, Section 5.3), so a pool's placement is a short chain on a warp of
// its own instead of the longest per-thread loop of a warp that holds 32 pools.  Requests and indices
// are read from the kept-request rows, results go straight to place_node / place_off.
__global__ void __launch_bounds__(256) k_place_gpu(const __grid_constant__ Params P, const HeadState* hst) {
  const int lane = threadIdx.x & 31;
  const long long x = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (x >= (long long)P.S * P.P) return;
  const int sc = (int)(x % P.S), j = P.pool_order[x / P.S];
  const PoolDev& pd = P.pool[j];
  if (pd.type != TG_POOL_GPU || !pd.lane_place || pd.n_nodes > 128 || !((hst[sc].need >> j) & 1u)) return;
  if (P.o_status[sc] & TG_ST_BAD_ACTION) return;
  const int keep = P.keepn[(size_t)sc * P.P + j];
  if (keep <= 0) return;
  const size_t row = (size_t)sc * P.N;
  const i64 base = P.meta[(size_t)sc * P.P + j].cbase;
  const unsigned short* rq = P.preq + row + base;
  const int* ord = P.order + row + base;
  // Section 5.3: requests by size descending, then queue position; each takes the smallest
  // sufficient maximal free block, lowest (node, start), and the low end of a split block.
  const u8* busy_row = P.gpu_busy ? P.gpu_busy + (size_t)sc * P.n_nodes_total + pd.node0 : nullptr;
  const int top = ilog2(pd.group), n_nodes = pd.n_nodes;
  const u32 pad = (~((1u << pd.group) - 1u)) & 0xffu;
  u32 nm[4], lev[4];
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int v = lane + 32 * s;
    nm[s] = v < n_nodes ? ((busy_row ? busy_row[v] : 0u) | pad) : 0xffu;
    lev[s] = node_levels(nm[s]);
  }
  for (int lz = top; lz >= 0; --lz) {
    const int z = 1 << lz;
    for (int i0 = 0; i0 < keep; i0 += 32) {
      const int i = i0 + lane;
      int nreq = 0;
      if (i < keep) {
        const u32 v = rq[i];
        const int g = v & 0x7f, gang = (v >> 7) & 1, ri = v >> 8;
        nreq = gang ? (g * ri == z ? 1 : 0) : (g == z ? ri : 0);
      }
      int myn = -1, myo = -1;
      u32 bm = __ballot_sync(TG_FULL, nreq > 0);
      while (bm) {
        const int b = __ffs(bm) - 1; bm &= bm - 1;
        const int cnt = __shfl_sync(TG_FULL, nreq, b);
        for (int rep = 0; rep < cnt; ++rep) {
          u32 node = 0xffffffffu; int bl = lz;
          for (; bl <= top; ++bl) {                     // smallest sufficient block level, lowest node
            u32 key = 0xffffffffu;
#pragma unroll
            for (int s = 3; s >= 0; --s) if ((lev[s] >> bl) & 1u) key = (u32)(lane + 32 * s);
            node = __reduce_min_sync(TG_FULL, key);
            if (node != 0xffffffffu) break;
          }
          if (node == 0xffffffffu) continue;            // cannot happen: the selection fits
          int start = 0;
          if (lane == (int)(node & 31u)) {
#pragma unroll
            for (int s = 0; s < 4; ++s)
              if (s == (int)(node >> 5)) {
                start = node_block_start(nm[s], bl);
                nm[s] |= ((1u << z) - 1u) << start;
                lev[s] = node_levels(nm[s]);
              }
          }
          start = __shfl_sync(TG_FULL, start, node & 31u);
          if (rep == 0 && lane == b) { myn = (int)node; myo = start; }
        }
      }
      if (i < keep && myn >= 0) { const size_t o = row + ord[i]; P.o_node[o] = myn; P.o_off[o] = myo; }
    }
  }
}

// gpu_apart: the solver-side GPU pools are left to k_place_gpu.
__global__ void __launch_bounds__(KPL_THREADS) k_place(const __grid_constant__ Params P, const HeadState* hst, int phase, int gpu_apart) {
  __shared__ KplWarp s_w[KPL_WARPS];
  const int lane = threadIdx.x & 31;
  KplWarp& W = s_w[threadIdx.x >> 5];
  const int gw = blockIdx.x * KPL_WARPS + (threadIdx.x >> 5);
  const int wps = (P.S + 31) / 32;                        // warps per pool
  if (gw >= wps * P.P) return;
  const int j = P.pool_order[gw / wps], sc = (gw % wps) * 32 + lane;
  const PoolDev& pd = P.pool[j];
  // A scenario with an invalid record selects nothing.  The record may sit far behind the prefix,
  // where k_stream finds it while k_solve is already deciding the scenario's pools; so the last
  // kernel of the round takes back whatever was written for such a scenario.
  const bool bad = sc < P.S && (P.o_status[sc] & TG_ST_BAD_ACTION);
  if (bad && gw / wps == 0 && phase == 1) {
    const size_t r0 = (size_t)sc * P.N;
    for (int i = 0; i < min(hst[sc].n, P.N); ++i) { P.o_alloc[r0 + i] = 0; P.o_node[r0 + i] = -1; P.o_off[r0 + i] = -1; P.o_act[r0 + i] = -1; }
    P.o_total[sc] = 0; P.o_nsel[sc] = 0; P.o_status[sc] = TG_ST_BAD_ACTION;
  }
  if (!pd.lane_place) return;
  int keep = (sc < P.S && !bad) ? P.keepn[(size_t)sc * P.P + j] : 0;
  if (keep < 0) keep = 0;
  if (sc < P.S && (int)(((hst[sc].need >> j) & 1u) != 0u) != phase) keep = 0;   // the other phase's pool
  if (phase == 1 && gpu_apart && pd.type == TG_POOL_GPU) keep = 0;             // k_place_gpu has them
  const int maxkeep = warp_max32(keep);
  if (maxkeep == 0) return;
  const size_t row = (size_t)(sc < P.S ? sc : 0) * P.N;
  const i64 base = sc < P.S ? P.meta[(size_t)sc * P.P + j].cbase : 0;
  const unsigned short* rq = P.preq + row + base;
  const int* ord = P.order + row + base;
  u8* st = W.state + lane;

  if (pd.type == TG_POOL_API) {                           // Section 5.1: offset = units consumed before
    int used = 0;
    for (int c0 = 0; c0 < maxkeep; c0 += 32) {
      kpl_load(W, rq, ord, keep, c0, lane);
      const int nc = min(32, keep - c0);
      for (int c = 0; c < nc; ++c) {
        const u32 v = W.rq[c * 33 + lane];
        W.node[c * 33 + lane] = 0; W.off[c * 33 + lane] = used;
        used += (int)(v & 0x7fu) * (int)(v >> 8);
      }
      kpl_store(P, W, row, keep, c0, lane);
    }
    return;
  }

  if (pd.type == TG_POOL_CPU && pd.group <= 64) {
    // Section 5.2 on a pool nobody occupies yet: cores are taken lowest id first, so the free
    // count per domain is the whole state.  Domains at or beyond `frontier` are untouched; the
    // touched ones with free cores left are kept in one list per free count, ascending by domain
    // (head[f], next[d]), and `occ` has bit f-1 set when list f is not empty: the best fit (fewest
    // free cores that still fit, lowest domain among equals) is the head of the first list at
    // or above the request.
    const int G = pd.group, D = pd.capacity / G;
    u8* head = st;                                        // head[f - 1], f = 1 .. 64
    u8* next = st + 64 * 32;                              // next[d]
    u64 occ = 0;
    int frontier = 0;
    auto push = [&](int d, int f) {                       // insert domain d into list f, ascending
      const u64 bit = 1ull << (f - 1);
      int prev = -1, cur = (occ & bit) ? (int)head[(f - 1) * 32] : 0xff;
      while (cur != 0xff && cur < d) { prev = cur; cur = next[cur * 32]; }
      next[d * 32] = (u8)cur;
      if (prev < 0) head[(f - 1) * 32] = (u8)d; else next[prev * 32] = (u8)d;
      occ |= bit;
    };
    auto pop = [&](int f) {                               // take the lowest domain off list f
      const int d = head[(f - 1) * 32], nx = next[d * 32];
      if (nx == 0xff) occ &= ~(1ull << (f - 1)); else head[(f - 1) * 32] = (u8)nx;
      return d;
    };
    for (int c0 = 0; c0 < maxkeep; c0 += 32) {
      kpl_load(W, rq, ord, keep, c0, lane);
      const int nc = min(32, keep - c0);
      for (int c = 0; c < nc; ++c) {
        const u32 v = W.rq[c * 33 + lane];
        const int k = (int)(v & 0x7fu) * (int)(v >> 8);
        int first = -1, dom = -1;
        const u64 fit = k <= 64 ? occ >> (k - 1) : 0ull;   // lists with at least k free cores
        if (fit) {
          const int f = k + __ffsll((long long)fit) - 1;
          dom = pop(f); first = dom * G + (G - f);
          if (f - k > 0) push(dom, f - k);
        } else if (frontier < D && G >= k) {              // an untouched domain
          dom = frontier++; first = dom * G;
          if (G - k > 0) push(dom, G - k);
        } else {                                          // no domain fits: ascending domains
          int need = k;
          while (need > 0) {
            int lo = 0xff, lf = 0;                        // open domain of lowest id: the smallest list head
            for (u64 o = occ; o; o &= o - 1) {
              const int f = __ffsll((long long)o);
              const int d = head[(f - 1) * 32];
              if (d < lo) { lo = d; lf = f; }
            }
            int d, f;
            if (lo != 0xff) { d = pop(lf); f = lf; }
            else if (frontier < D) { d = frontier++; f = G; }
            else break;                                   // cannot happen: the selection fits
            if (first < 0) { first = d * G + (G - f); dom = d; }
            const int take = min(f, need);
            need -= take;
            if (f - take > 0) push(d, f - take);
          }
        }
        W.node[c * 33 + lane] = (short)dom; W.off[c * 33 + lane] = first;
      }
      kpl_store(P, W, row, keep, c0, lane);
    }
    return;
  }

  if (pd.type == TG_POOL_CPU) {
    // Section 5.2 on a pool nobody occupies yet: cores are taken lowest id first, so the free
    // count per domain is the whole state.  Domains at or beyond `frontier` are untouched; of the
    // touched ones only those with free cores left are kept, as an unordered list of
    // (domain, free) pairs - full domains can serve nobody, and the list stays short because
    // small requests keep filling the holes.
    const int G = pd.group, D = pd.capacity / G;
    u8* od = st;                                          // open domain ids
    u8* of = st + KPL_DOMAINS * 32;                       // their free cores
    int frontier = 0, n_open = 0;
    for (int c0 = 0; c0 < maxkeep; c0 += 32) {
      kpl_load(W, rq, ord, keep, c0, lane);
      const int nc = min(32, keep - c0);
      for (int c = 0; c < nc; ++c) {
        const u32 v = W.rq[c * 33 + lane];
        const int k = (int)(v & 0x7fu) * (int)(v >> 8);
        // best fit: fewest free cores that still fit, lowest domain among equals
        int bkey = INT_MAX, bslot = -1;
        for (int x = 0; x < n_open; ++x) {
          const int f = of[x * 32], key = (f << 8) | od[x * 32];
          if (f >= k && key < bkey) { bkey = key; bslot = x; }
        }
        int first = -1, dom = -1;
        if (bslot >= 0) {
          const int f = bkey >> 8;
          dom = bkey & 0xff; first = dom * G + (G - f);
          if (f - k > 0) of[bslot * 32] = (u8)(f - k);
          else { --n_open; od[bslot * 32] = od[n_open * 32]; of[bslot * 32] = of[n_open * 32]; }
        } else if (frontier < D && G >= k) {              // an untouched domain
          dom = frontier++; first = dom * G;
          if (G - k > 0) { od[n_open * 32] = (u8)dom; of[n_open * 32] = (u8)(G - k); ++n_open; }
        } else {                                          // no domain fits: ascending domains
          int need = k;
          while (need > 0) {
            int lo = INT_MAX, ls = -1;                    // open domain of lowest id
            for (int x = 0; x < n_open; ++x) { const int d = od[x * 32]; if (d < lo) { lo = d; ls = x; } }
            int d, f;
            if (ls >= 0) { d = lo; f = of[ls * 32]; }
            else if (frontier < D) { d = frontier++; f = G; }
            else break;                                   // cannot happen: the selection fits
            if (first < 0) { first = d * G + (G - f); dom = d; }
            const int take = min(f, need);
            need -= take;
            if (ls >= 0) {
              if (f - take > 0) of[ls * 32] = (u8)(f - take);
              else { --n_open; od[ls * 32] = od[n_open * 32]; of[ls * 32] = of[n_open * 32]; }
            } else if (f - take > 0) { od[n_open * 32] = (u8)d; of[n_open * 32] = (u8)(f - take); ++n_open; }
          }
        }
        W.node[c * 33 + lane] = (short)dom; W.off[c * 33 + lane] = first;
      }
      kpl_store(P, W, row, keep, c0, lane);
    }
    return;
  }

  // Section 5.3: requests by size descending, then queue position; each takes the smallest
  // sufficient maximal free block, lowest (node, start), and the low end of a split block.
  // lv[l]: nodes that hold a maximal free block of 2^l GPUs.
  const int top = ilog2(pd.group), n_nodes = pd.n_nodes;
  const u32 pad = (~((1u << pd.group) - 1u)) & 0xffu;
  const u8* busy_row = (P.gpu_busy && sc < P.S) ? P.gpu_busy + (size_t)sc * P.n_nodes_total + pd.node0 : nullptr;
  u64 lv[4] = {0, 0, 0, 0};
  for (int n = 0; n < n_nodes; ++n) {
    const u32 b = (busy_row ? busy_row[n] : 0u) | pad;
    st[n * 32] = (u8)b;
    const u32 lev = node_levels(b);
#pragma unroll
    for (int l = 0; l < 4; ++l) lv[l] |= (u64)((lev >> l) & 1u) << n;
  }
  for (int lz = top; lz >= 0; --lz) {
    const int z = 1 << lz;
    for (int c0 = 0; c0 < maxkeep; c0 += 32) {
      kpl_load(W, rq, ord, keep, c0, lane);
      const int nc = min(32, keep - c0);
      // candidates of the chunk that ask for blocks of this size
      u32 todo = 0;
      for (int c = 0; c < nc; ++c) {
        const u32 v = W.rq[c * 33 + lane];
        const int g = v & 0x7f, gang = (v >> 7) & 1, ri = v >> 8;
        if (gang ? g * ri == z : g == z) todo |= 1u << c;
        W.node[c * 33 + lane] = KPL_NONE;
      }
      // one request per thread and turn, so that threads with few requests do not sit through
      // the others' candidates
      int reps = 0, cc = 0;
      bool first = false;
      for (;;) {
        if (reps == 0 && todo) {
          cc = __ffs(todo) - 1; todo &= todo - 1;
          const u32 v = W.rq[cc * 33 + lane];
          reps = ((v >> 7) & 1) ? 1 : (int)(v >> 8);
          first = true;
        }
        if (!__any_sync(TG_FULL, reps > 0)) break;
        if (reps > 0) {
          --reps;
          int bl = lz;
          u64 mask = 0;
          for (; bl <= top; ++bl) {
            mask = bl == 0 ? lv[0] : (bl == 1 ? lv[1] : (bl == 2 ? lv[2] : lv[3]));
            if (mask) break;
          }
          if (mask) {                                     // always: the selection fits
            const int node = __ffsll((long long)mask) - 1;
            u32 b = st[node * 32];
            const int start = node_block_start(b, bl);
            b |= ((1u << z) - 1u) << start;
            st[node * 32] = (u8)b;
            const u32 lev = node_levels(b);
            const u64 bit = 1ull << node;
#pragma unroll
            for (int l = 0; l < 4; ++l) lv[l] = (lv[l] & ~bit) | ((u64)((lev >> l) & 1u) << node);
            if (first) { W.node[cc * 33 + lane] = (short)node; W.off[cc * 33 + lane] = start; }
          }
          first = false;
        }
      }
      kpl_store(P, W, row, keep, c0, lane);
    }
  }
}
