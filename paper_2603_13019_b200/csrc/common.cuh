// Shared device-side definitions of the scheduling-round kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

typedef long long i64;
typedef unsigned long long u64;
typedef unsigned int u32;
typedef unsigned char u8;

#define TG_INF 0x7fffffffffffffffLL
#define TG_PARAM_MAX (1LL << 40)
#define TG_MAX_POOLS 8
#define TG_POOL_CPU 0
#define TG_POOL_GPU 1
#define TG_POOL_API 2
#define TG_ST_BAD_ACTION 1
#define TG_ST_UNSORTED 2
#define TG_ST_WORKSPACE 4
#define TG_FULL 0xffffffffu

struct PoolDev {
  int type, capacity, group, window_us;
  int node0, n_nodes;   // GPU pools: first node in a gpu_busy row, node count
  int slot0, n_slots;   // demand slots in the prefix scan (GPU: 4 nested levels, else 1)
  int lane_place;       // batched path: the pool is placed by k_place, one thread per scenario
};

// per (scenario, pool) facts produced by the prefix kernel
struct PoolMeta {
  i64 base;       // the pool's list in `tmin` starts at scenario * max_actions + base
  i64 cbase;      // the pool's candidates in order / preq / the solver's arrays start at scenario * max_actions + cbase
  int count;      // actions of the pool in the queue (candidates only, if nobody will read its waiting list)
  int m;          // candidates of the pool (they occupy positions base .. base+m-1)
  int elastic;    // some candidate has more than one level
  int first_wait; // index of the pool's first waiting action, -1 if none (or the list is not needed)
};

struct Params {
  int S, N, P, depth, n_nodes_total, V;
  PoolDev pool[TG_MAX_POOLS];
  int pool_order[TG_MAX_POOLS];   // pools in the order their tasks are handed out (longest tasks first)
  // candidate arrays of the batched path: a pool has at most min(max_actions, capacity) candidates (each
  // takes a unit at least), so a scenario's rows are cand_off[j] .. cand_off[j+1] of cand_stride entries
  int cand_off[TG_MAX_POOLS + 1]; int cand_stride;
  i64 now;
  // inputs (device)
  const u8* a_pool; const u8* a_unit; const u32* a_mask;
  const i64* a_s; const i64* a_p; const i64* a_arrival;
  const int* n_actions; const u8* gpu_busy;
  // service cache of the GPU pools (cache_slots = 0: none)
  const unsigned short* a_service; const i64* a_restore; u32* cache_tag; i64* cache_use; int cache_slots;
  // further entries of the cost vectors (n_side = 0: none): entry e of (scenario, action) at e * side_plane + row + i
  int n_side; const u8* a_side_pool; const unsigned short* a_side_units; u64 side_plane;
  int* side_bad;     // [S] an entry of the scenario names no usable pool or amount
  int* side_res;     // [S][P] what the candidates ask of a pool beside their key resource
  // outputs (device)
  int* o_alloc; int* o_node; int* o_off; i64* o_act; i64* o_total; int* o_nsel; int* o_status;
  // workspace
  int* order;        // [S][N] action index at each partitioned position
  i64* tmin;         // [S][N] duration at the least level, partitioned order
  PoolMeta* meta;    // [S][P]
  unsigned short* preq;  // what k_place reads per kept candidate: unit byte | multiplicity << 8 (partitioned order)
  int* keepn;        // [S][P] candidates kept, -1 = placed elsewhere
  char* slabs; u64 slab_bytes; int n_workers;
  char* arena; u64 arena_bytes; u64* arena_top;
  int slot_tries;    // rounds of looking for a free arena slot (2 us apart) before a warp gives up
  const u32* ok_table;   // [TG_MAX_POOLS][256]: multiplicities a record with that unit byte may use on that pool (0: none)
};

// ceil(2^64 / r) for r = 2..32: floor(p / r) == umul64hi(p, c_recip[r]) for 0 <= p <= 2^40,
// because the rounding excess p * (r - 2^64 mod r) / (r * 2^64) stays below 2^-24 < 1/r.
__constant__ u64 c_recip[33];
// maximal free aligned blocks of a node, indexed by its busy mask: byte l = blocks of size 2^l
__constant__ u32 c_fblocks[256];

__device__ __forceinline__ i64 div_small(i64 p, int r) {
  return r == 1 ? p : (i64)__umul64hi((u64)p, c_recip[r]);
}
__device__ __forceinline__ i64 clamp_param(i64 v) { return v < 0 ? 0 : (v > TG_PARAM_MAX ? TG_PARAM_MAX : v); }
__device__ __forceinline__ i64 sat_add(i64 a, i64 b) {   // a, b >= 0
  u64 c = (u64)a + (u64)b;
  return c > (u64)TG_INF ? TG_INF : (i64)c;
}
__device__ __forceinline__ int ilog2(int v) { return 31 - __clz(v); }

struct Act {
  i64 s, p;
  u32 mask;   // usable multiplicities: bit r-1
  int g, gang;
};

// Usable levels of a record on its pool.  Returns false for records no pool can serve.
__device__ __forceinline__ bool decode_levels(const PoolDev& pd, u8 unit, u32 mask, int& g, int& gang, u32& eff) {
  g = unit & 0x7f;
  gang = (unit >> 7) && pd.type == TG_POOL_GPU;
  eff = 0;
  if (g == 0) return false;
  if (pd.type == TG_POOL_GPU) {
    bool p2 = (g & (g - 1)) == 0;
    if (gang) {
      u32 ok = 0;
      if (p2) {
        if (g <= pd.group) ok |= 1u;
        if (2 * g <= pd.group) ok |= 2u;
        if (4 * g <= pd.group) ok |= 8u;
        if (8 * g <= pd.group) ok |= 128u;
      }
      mask &= ok;
    } else if (!(p2 && g <= pd.group)) return false;
  }
  eff = mask;
  return mask != 0;
}

// Duration at multiplicity r (Eq. 1 in integer microseconds): s + floor(p / r)
__device__ __forceinline__ i64 duration(i64 s, i64 p, int r) { return s + div_small(p, r); }

// Chunk-size level that a grant of multiplicity r asks for
__device__ __forceinline__ int level_of(int g, int gang, int r) { return ilog2(gang ? g * r : g); }

// Warp reductions.  The SM moves one shuffle per cycle or two for all its warps, so the 32-bit
// ones use the reduction unit (one instruction), and the 64-bit ones are put together from
// 32-bit reductions.
__device__ __forceinline__ i64 warp_min64(i64 v) {      // any signed values
  const u64 u = (u64)v ^ 0x8000000000000000ull;          // order-preserving map to unsigned
  const u32 hi = (u32)(u >> 32);
  const u32 mhi = __reduce_min_sync(TG_FULL, hi);
  const u32 mlo = __reduce_min_sync(TG_FULL, hi == mhi ? (u32)u : 0xffffffffu);
  return (i64)((((u64)mhi << 32) | mlo) ^ 0x8000000000000000ull);
}
__device__ __forceinline__ i64 warp_sum64(i64 v) {      // 0 <= v, sum below 2^63
  const u32 a = __reduce_add_sync(TG_FULL, (u32)v & 0x3fffffu);
  const u32 b = __reduce_add_sync(TG_FULL, (u32)(v >> 22) & 0x3fffffu);
  const u32 c = __reduce_add_sync(TG_FULL, (u32)((u64)v >> 44));
  return (i64)((u64)a + ((u64)b << 22) + ((u64)c << 44));
}
__device__ __forceinline__ int warp_sum32(int v) { return (int)__reduce_add_sync(TG_FULL, (u32)v); }
__device__ __forceinline__ int warp_min32(int v) { return __reduce_min_sync(TG_FULL, v); }
__device__ __forceinline__ int warp_max32(int v) { return __reduce_max_sync(TG_FULL, v); }

// Free capacity per chunk level of a GPU pool: cap[l] = GPUs held in maximal free aligned
// blocks of size >= 2^l.  `busy` may be null (all free).  Warp-cooperative.
__device__ __forceinline__ void gpu_caps(const PoolDev& pd, const u8* busy, int lane, int cap[4]) {
  int F0 = 0, F1 = 0, F2 = 0, F3 = 0;
  u32 pad = (~((1u << pd.group) - 1u)) & 0xffu;   // GPUs beyond the node size count as busy
  for (int v = lane; v < pd.n_nodes; v += 32) {
    u32 b = (busy ? busy[pd.node0 + v] : 0u) | pad;
    u32 f = c_fblocks[b & 0xffu];
    F0 += f & 0xff; F1 += (f >> 8) & 0xff; F2 += (f >> 16) & 0xff; F3 += f >> 24;
  }
  F0 = warp_sum32(F0); F1 = warp_sum32(F1); F2 = warp_sum32(F2); F3 = warp_sum32(F3);
  cap[3] = F3 * 8; cap[2] = cap[3] + F2 * 4; cap[1] = cap[2] + F1 * 2; cap[0] = cap[1] + F0;
}

// The arena of large scratch: its lower 7/8 are equal slots that a warp borrows for one large DP
// table and gives back (48 slots of at least 64 MiB when the arena allows, else down to 4
// larger-as-possible ones); the rest is handed out by a bump pointer, never reused in a call.
#define TG_ARENA_MAX_SLOTS 48
__device__ __forceinline__ int arena_n_slots(const Params& P) {
  u64 n = (P.arena_bytes / 8 * 7) >> 26;
  return n < 4 ? 4 : (n > TG_ARENA_MAX_SLOTS ? TG_ARENA_MAX_SLOTS : (int)n);
}
__device__ __forceinline__ u64 arena_slot_bytes(const Params& P) { return ((P.arena_bytes / 8 * 7) / arena_n_slots(P)) & ~(u64)255; }
__device__ __forceinline__ u64 arena_bump_base(const Params& P) { return arena_slot_bytes(P) * arena_n_slots(P); }
