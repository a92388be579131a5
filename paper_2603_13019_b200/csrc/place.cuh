// Placement of what a pool's selection granted, one warp per (scenario, pool).
//   GPU pools (Section 5.3): chunks are aligned power-of-two intervals inside a node; requests
//     are served by size descending, then queue position; each takes the smallest sufficient
//     maximal free block, lowest (node, start) first, and the low end of a split block.
//   CPU pools (Section 5.2): cores are exclusive; an action's cores come from one NUMA domain
//     when one fits (fewest free cores that still fit, lowest index), lowest core ids first;
//     otherwise domains are filled in ascending order.
//   API pools (Section 5.1): the grant is accounted against the quota / concurrency limit.
#pragma once
#include "common.cuh"

// lowest start of a maximal free aligned block of size 2^bl in a node mask, or -1
__device__ __forceinline__ int find_block(u32 busy, int bl, int group) {
  const int bs = 1 << bl;
  const u32 ones = (1u << bs) - 1u;
  for (int st = 0; st < group; st += bs) {
    if (busy & (ones << st)) continue;
    if (bs < 8) {                                       // maximal: the enclosing block is not free
      int ps = st & ~(2 * bs - 1);
      u32 pones = ((1u << (2 * bs)) - 1u) << ps;
      if (!(busy & pones)) continue;
    }
    return st;
  }
  return -1;
}

// nm: node busy masks of the pool (updated).  keep candidates, multiplicities r[].
// owner (may be null): one entry per GPU of the pool, receives ids[i] for every GPU granted.
__device__ void place_gpu(const PoolDev& pd, u8* nm, int keep, const u8* cg, const u8* r,
                          int* pnode, int* poff, int lane, int* owner = nullptr, const int* ids = nullptr) {
  const int top = ilog2(pd.group);
  const u32 pad = (~((1u << pd.group) - 1u)) & 0xffu;
  for (int lz = top; lz >= 0; --lz) {
    const int z = 1 << lz;
    for (int i = 0; i < keep; ++i) {
      const int g = cg[i] & 0x7f, gang = cg[i] >> 7, ri = r[i];
      const int nreq = gang ? (g * ri == z ? 1 : 0) : (g == z ? ri : 0);
      for (int rep = 0; rep < nreq; ++rep) {
        int node = -1, start = -1;
        for (int bl = lz; bl <= top && node < 0; ++bl) {
          for (int v0 = 0; v0 < pd.n_nodes; v0 += 32) {
            int v = v0 + lane;
            bool has = v < pd.n_nodes && ((c_fblocks[nm[v] | pad] >> (8 * bl)) & 0xffu) != 0;
            u32 b = __ballot_sync(TG_FULL, has);
            if (b) { node = v0 + __ffs(b) - 1; start = find_block(nm[node] | pad, bl, pd.group); break; }
          }
        }
        if (node < 0 || start < 0) continue;            // cannot happen: the selection fits
        __syncwarp();
        if (lane == 0) {
          nm[node] |= (u8)(((1u << z) - 1u) << start);
          if (rep == 0) { pnode[i] = node; poff[i] = start; }
          if (owner) for (int b = 0; b < z; ++b) owner[node * pd.group + start + b] = ids[i];
        }
        __syncwarp();
      }
    }
  }
}

// busy: one bit per core (word array); dfree: free cores per domain.  Both updated.
__device__ void place_cpu(const PoolDev& pd, u32* busy, int* dfree, int keep, const u8* cg,
                          const u8* r, int* pnode, int* poff, int lane) {
  const int D = pd.capacity / pd.group;
  for (int i = 0; i < keep; ++i) {
    const int k = (cg[i] & 0x7f) * r[i];
    i64 key = TG_INF;
    for (int d = lane; d < D; d += 32) {
      int f = dfree[d];
      if (f >= k) key = min(key, ((i64)f << 32) | d);
    }
    key = warp_min64(key);
    if (lane == 0) {
      int lo = 0, hi = pd.capacity;
      if (key != TG_INF) { int d = (int)(key & 0xffffffff); lo = d * pd.group; hi = lo + pd.group; }
      int need = k, first = -1;
      for (int c = lo; c < hi && need > 0; ++c) {
        u32 w = busy[c >> 5];
        if (w == 0xffffffffu && (c & 31) == 0 && c + 32 <= hi) { c += 31; continue; }
        if (w >> (c & 31) & 1u) continue;
        busy[c >> 5] = w | (1u << (c & 31));
        dfree[c / pd.group] -= 1;
        if (first < 0) first = c;
        --need;
      }
      pnode[i] = first >= 0 ? first / pd.group : -1; poff[i] = first;
    }
    __syncwarp();
  }
}

// CPU placement on a pool nobody occupies yet (a single round).  Cores are only ever taken
// lowest id first, so the used cores of a domain are always a prefix of it: the free count per
// domain is the whole state and a grant's first core follows from it.  Same rule as place_cpu.
__device__ void place_cpu_fresh(const PoolDev& pd, int* dfree, int keep, const u8* cg, const u8* r,
                                int* pnode, int* poff, int lane) {
  const int D = pd.capacity / pd.group;
  for (int d = lane; d < D; d += 32) dfree[d] = pd.group;
  __syncwarp();
  for (int i0 = 0; i0 < keep; i0 += 32) {
    // this lane's candidate of the block of 32; its units are broadcast when its turn comes
    const int mine = i0 + lane < keep ? (cg[i0 + lane] & 0x7f) * r[i0 + lane] : 0;
    const int nb = min(32, keep - i0);
    for (int b = 0; b < nb; ++b) {
      const int k = __shfl_sync(TG_FULL, mine, b);
      i64 key = TG_INF;
      for (int d = lane; d < D; d += 32) {
        int f = dfree[d];
        if (f >= k) key = min(key, ((i64)f << 32) | d);
      }
      key = warp_min64(key);
      if (lane == 0) {
        int first = -1;
        if (key != TG_INF) {
          int d = (int)(key & 0xffffffff);
          first = d * pd.group + (pd.group - dfree[d]);
          dfree[d] -= k;
        } else {
          int need = k;
          for (int d = 0; d < D && need > 0; ++d) {
            int f = dfree[d];
            if (f == 0) continue;
            if (first < 0) first = d * pd.group + (pd.group - f);
            int take = min(f, need);
            dfree[d] = f - take; need -= take;
          }
        }
        pnode[i0 + b] = first >= 0 ? first / pd.group : -1; poff[i0 + b] = first;
      }
      __syncwarp();
    }
  }
}

// CPU placement on a pool with cores in use (trace replay): owner[c] < 0 marks a free core,
// dfree the free cores per domain.  Same rule as place_cpu; a grant writes ids[i] into owner.
__device__ void place_cpu_owner(const PoolDev& pd, int* owner, int* dfree, int keep, const u8* cg,
                                const u8* r, const int* ids, int* pnode, int* poff, int lane) {
  const int D = pd.capacity / pd.group;
  for (int i = 0; i < keep; ++i) {
    const int k = (cg[i] & 0x7f) * r[i];
    i64 key = TG_INF;
    for (int d = lane; d < D; d += 32) {
      int f = dfree[d];
      if (f >= k) key = min(key, ((i64)f << 32) | d);
    }
    key = warp_min64(key);
    int lo = 0, hi = pd.capacity;
    if (key != TG_INF) { int d = (int)(key & 0xffffffff); lo = d * pd.group; hi = lo + pd.group; }
    // lowest free cores of [lo, hi): 32 cores per pass, each lane claims by its rank among the free
    int need = k, first = -1;
    for (int c0 = lo; c0 < hi && need > 0; c0 += 32) {
      const int c = c0 + lane;
      const bool fr = c < hi && owner[c] < 0;
      const u32 b = __ballot_sync(TG_FULL, fr);
      const int rank = __popc(b & ((1u << lane) - 1u));
      if (fr && rank < need) { owner[c] = ids[i]; atomicSub(&dfree[c / pd.group], 1); }
      if (b && first < 0) first = c0 + __ffs(b) - 1;
      need -= min(need, __popc(b));
    }
    if (lane == 0) { pnode[i] = first >= 0 ? first / pd.group : -1; poff[i] = first; }
    __syncwarp();
  }
}

// ---- register-resident fast paths of a single round (fresh CPU pool, at most 128 domains /
// ---- GPU nodes): the state lives in lane registers, the arg-min is one redux, and every lane
// ---- keeps the result of "its" candidate of a block of 32 for a coalesced write.

// maximal free aligned blocks of a node: bit = first GPU of such a block (busy: 8 bits, padded)
struct NodeBlocks { u32 s1, s2, s4, s8; };
__device__ __forceinline__ NodeBlocks node_blocks(u32 busy) {
  const u32 fr = ~busy & 0xffu;
  const u32 pr = fr & (fr >> 1) & 0x55u;          // bit 2k: GPUs 2k, 2k+1 free
  const u32 nb = pr & (pr >> 2) & 0x11u;          // bit 4k: GPUs 4k .. 4k+3 free
  const u32 oc = nb & (nb >> 4) & 1u;             // the whole node free
  NodeBlocks b;
  b.s1 = fr & ~(pr | (pr << 1));
  b.s2 = pr & ~(nb | (nb << 2));
  b.s4 = nb & ~(oc | (oc << 4));
  b.s8 = oc;
  return b;
}
__device__ __forceinline__ u32 node_levels(u32 busy) {   // bit l: a maximal free block of 2^l GPUs exists
  const NodeBlocks b = node_blocks(busy);
  return (b.s1 ? 1u : 0u) | (b.s2 ? 2u : 0u) | (b.s4 ? 4u : 0u) | (b.s8 ? 8u : 0u);
}
__device__ __forceinline__ int node_block_start(u32 busy, int bl) {
  const NodeBlocks b = node_blocks(busy);
  const u32 m = bl == 0 ? b.s1 : (bl == 1 ? b.s2 : (bl == 2 ? b.s4 : b.s8));
  return __ffs(m) - 1;
}

// GPU placement with a service cache (Section 5.3, evict on execution).  The rule of place_gpu, and among
// the free blocks of the level it picks, one whose granted chunk (the block's low end) caches the
// request's instance goes first, then the lowest (node, start).  An instance is (service, chunk size);
// a chunk caches it iff every GPU of the chunk remembers its tag.  ctag / cuse: the pool's entries,
// [node][8][K] (tag 0 = empty, time of last use).  A grant makes the instance the most recently used
// one on every GPU of the chunk; on a miss a GPU overwrites an empty entry (lowest index), else its
// least recently used one (lowest index among equals), and miss[i] is set: candidate i then runs its
// restoration time longer.  svc: the scenario's service column (may be null), ids: action indices.
__device__ void place_gpu_cache(const PoolDev& pd, u8* nm, int keep, const u8* cg, const u8* r, const int* ids,
                                int* pnode, int* poff, u8* miss, const unsigned short* svc, u32* ctag, i64* cuse,
                                int K, i64 now, int lane, int* owner = nullptr) {
  const int top = ilog2(pd.group);
  const u32 pad = (~((1u << pd.group) - 1u)) & 0xffu;
  for (int i = lane; i < keep; i += 32) miss[i] = 0;
  __syncwarp();
  for (int lz = top; lz >= 0; --lz) {
    const int z = 1 << lz;
    for (int i = 0; i < keep; ++i) {
      const int g = cg[i] & 0x7f, gang = cg[i] >> 7, ri = r[i];
      const int nreq = gang ? (g * ri == z ? 1 : 0) : (g == z ? ri : 0);
      if (nreq == 0) continue;
      const u32 sv = svc ? svc[ids[i]] : 0xffffu;
      const u32 tag = sv == 0xffffu ? 0u : ((sv << 3) | (u32)lz) + 1u;
      for (int rep = 0; rep < nreq; ++rep) {
        u32 kmin = 0xffffffffu;
        for (int bl = lz; bl <= top && kmin == 0xffffffffu; ++bl) {
          u32 key = 0xffffffffu;
          for (int v = lane; v < pd.n_nodes; v += 32) {
            const NodeBlocks nb = node_blocks(nm[v] | pad);
            u32 starts = bl == 0 ? nb.s1 : (bl == 1 ? nb.s2 : (bl == 2 ? nb.s4 : nb.s8));
            while (starts) {
              const int st = __ffs(starts) - 1; starts &= starts - 1;
              bool hit = tag != 0;
              for (int b = st; b < st + z && hit; ++b) {
                bool has = false;
                for (int k = 0; k < K; ++k) has |= ctag[(size_t)(v * 8 + b) * K + k] == tag;
                hit = has;
              }
              key = min(key, (hit ? 0u : 1u << 30) | ((u32)v << 4) | (u32)st);
            }
          }
          kmin = __reduce_min_sync(TG_FULL, key);
        }
        if (kmin == 0xffffffffu) continue;              // cannot happen: the selection fits
        const int node = (int)((kmin >> 4) & 0x3ffffffu), start = (int)(kmin & 15u);
        const bool hit = (kmin >> 30) == 0;
        __syncwarp();
        if (lane == 0) {
          nm[node] |= (u8)(((1u << z) - 1u) << start);
          if (rep == 0) { pnode[i] = node; poff[i] = start; }
          if (owner) for (int b = 0; b < z; ++b) owner[node * pd.group + start + b] = ids[i];
          if (tag) {
            if (!hit) miss[i] = 1;
            for (int b = start; b < start + z; ++b) {
              u32* tg = ctag + (size_t)(node * 8 + b) * K;
              i64* us = cuse + (size_t)(node * 8 + b) * K;
              int at = -1;
              for (int k = 0; k < K && at < 0; ++k) if (tg[k] == tag) at = k;
              for (int k = 0; k < K && at < 0; ++k) if (tg[k] == 0) at = k;
              if (at < 0) { at = 0; for (int k = 1; k < K; ++k) if (us[k] < us[at]) at = k; }
              tg[at] = tag; us[at] = now;
            }
          }
        }
        __syncwarp();
      }
    }
  }
}

// Same placement rule as place_gpu; requires pd.n_nodes <= 128.  busy_row: the pool's node
// masks before the round (may be null).
__device__ void place_gpu_reg(const PoolDev& pd, const u8* busy_row, int keep, const u8* cg, const u8* r,
                              int* pnode, int* poff, int lane) {
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
        const int g = cg[i] & 0x7f, gang = cg[i] >> 7, ri = r[i];
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
      if (i < keep && myn >= 0) { pnode[i] = myn; poff[i] = myo; }
    }
  }
}

// Same placement rule as place_cpu_fresh; requires at most 128 domains of fewer than 65536 cores.
__device__ void place_cpu_fresh_reg(const PoolDev& pd, int keep, const u8* cg, const u8* r,
                                    int* pnode, int* poff, int lane) {
  const int G = pd.group, D = pd.capacity / G;
  u32 df[4];
#pragma unroll
  for (int s = 0; s < 4; ++s) df[s] = lane + 32 * s < D ? (u32)G : 0u;
  for (int i0 = 0; i0 < keep; i0 += 32) {
    const int i = i0 + lane;
    const int mine = i < keep ? (cg[i] & 0x7f) * r[i] : 0;
    int myn = -1, myo = -1;
    const int nb = min(32, keep - i0);
    for (int b = 0; b < nb; ++b) {
      const u32 k = (u32)__shfl_sync(TG_FULL, mine, b);
      u32 key = 0xffffffffu;
#pragma unroll
      for (int s = 0; s < 4; ++s) if (df[s] >= k) key = min(key, (df[s] << 16) | (u32)(lane + 32 * s));
      const u32 best = __reduce_min_sync(TG_FULL, key);
      int first = -1, dom = -1;
      if (best != 0xffffffffu) {                       // best fit: fewest free cores that still fit
        const int d = (int)(best & 0xffffu), f = (int)(best >> 16);
        first = d * G + (G - f); dom = d;
        if (lane == (d & 31)) {
#pragma unroll
          for (int s = 0; s < 4; ++s) if (s == (d >> 5)) df[s] -= k;
        }
      } else {                                         // no domain fits: fill domains in ascending order
        u32 need = k;
        for (int d = 0; d < D && need > 0; ++d) {
          u32 f = 0;
#pragma unroll
          for (int s = 0; s < 4; ++s) if (s == (d >> 5)) f = df[s];
          f = __shfl_sync(TG_FULL, f, d & 31);
          if (f == 0) continue;
          if (first < 0) { first = d * G + (G - (int)f); dom = d; }
          const u32 take = min(f, need);
          if (lane == (d & 31)) {
#pragma unroll
            for (int s = 0; s < 4; ++s) if (s == (d >> 5)) df[s] -= take;
          }
          need -= take;
        }
      }
      if (lane == b) { myn = dom; myo = first; }
    }
    if (i < keep) { pnode[i] = myn; poff[i] = myo; }
  }
}
