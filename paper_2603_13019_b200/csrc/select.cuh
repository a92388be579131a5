// Per-pool selection of a round, executed by one warp per (scenario, pool):
//   optimal discrete allocation of a candidate prefix (DPArrange, Algorithms 3 and 4),
//   completion-heap estimate of what keeps waiting (Algorithm 2), greedy eviction
//   (Algorithm 1, lines 8-14).
//
// The DP runs in "extra demand over everybody's least level" coordinates: a cell is the
// vector e = (e_1, e_2, e_4, e_8) of GPUs requested at chunk sizes >= 1, 2, 4, 8 beyond the
// least-level requests (for core / quota pools only e_1 = extra units exists).  A cell is
// feasible iff e_l <= free capacity at that level minus the least-level demand, so the
// feasible cells form a box; a level whose capacity equals the next smaller level's is
// implied by it and dropped from the box.  Two certificates skip the DP altogether:
// every candidate's best level fits (then each takes the smallest level reaching its lowest
// duration), or no spare unit exists (then everybody keeps the least level).
// Ties follow the canonical order: lowest duration sum, then fewest units, then
// (k_m, ..., k_1) lexicographically smallest.
#pragma once
#include "common.cuh"
#include "sims.cuh"

// Scratch of one worker warp: a window of shared memory first (what is read over and over in
// sequential loops belongs there), its slab in global memory once the window is full.
struct Slab {
  char* base; u64 cap; u64 used;          // global slab
  char* fbase; u32 fcap; u32 fused;       // shared-memory window (generic address), may be empty
  __device__ __forceinline__ void* take(u64 bytes) {
    bytes = (bytes + 15) & ~(u64)15;
    if (used + bytes > cap) return nullptr;
    void* p = base + used; used += bytes; return p;
  }
  // small arrays that sequential loops read again and again: the window if there is room
  __device__ __forceinline__ void* take_fast(u64 bytes) {
    bytes = (bytes + 15) & ~(u64)15;
    if (fused + bytes <= fcap) { void* p = fbase + fused; fused += (u32)bytes; return p; }
    return take(bytes);
  }
};

// warp-uniform bump allocation from the bump part of the arena
__device__ __forceinline__ void* arena_take(const Params& P, u64 bytes, int lane) {
  bytes = (bytes + 255) & ~(u64)255;
  const u64 half = arena_bump_base(P);
  u64 off = 0;
  if (lane == 0) off = atomicAdd(P.arena_top, bytes);
  off = __shfl_sync(TG_FULL, off, 0);
  if (half + off + bytes > P.arena_bytes) return nullptr;
  return P.arena + half + off;
}
// Borrow a slot (warp-uniform).  Waits, with a limit, for another warp to give one back; the
// holders never wait for anything, so the wait ends.  Returns -1 if the table does not fit a
// slot or the limit ran out.
__device__ __forceinline__ int slot_acquire(const Params& P, u64 bytes, int lane) {
  const u64 slot_bytes = arena_slot_bytes(P);
  int got = -1;
  if (lane == 0 && bytes <= slot_bytes) {
    int* flags = (int*)(P.arena_top + 8);
    const int ns = arena_n_slots(P);
    const int start = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5) % ns;
    for (int tries = 0; tries < P.slot_tries && got < 0; ++tries) {   // gives up after the round's slot_wait_us
      for (int k = 0; k < ns && got < 0; ++k) {
        const int s = (start + k) % ns;
        if (atomicCAS(&flags[s], 0, 1) == 0) got = s;
      }
      if (got < 0) __nanosleep(2000);
    }
  }
  return __shfl_sync(TG_FULL, got, 0);
}
__device__ __forceinline__ char* slot_ptr(const Params& P, int s) {
  return P.arena + (u64)s * arena_slot_bytes(P);
}
__device__ __forceinline__ void slot_release(const Params& P, int s, int lane) {
  __syncwarp();
  if (lane == 0 && s >= 0) { __threadfence(); atomicExch((int*)(P.arena_top + 8) + s, 0); }
}

struct PoolTask {
  // the pool
  int type, group;
  int cap[4];             // free capacity per chunk level (core / quota pools: cap[0] only)
  // candidates of the pool in queue order
  int m;
  const i64* cs; const i64* cp; const u32* cmask; const u8* cg;
  // what waits behind them on this pool: durations at the least level, and the first record
  const i64* ac_tmin; int n_ac;
  Act ac_first;
  // completion times (relative to now) of what is running on the pool
  const i64* seeds; int n_seeds;
  int depth;
  // results: multiplicity per candidate of the prefix under evaluation / of the accepted one
  u8* rsel; u8* rkeep;
  int* rowcand;           // scratch, m ints
  // shared memory of this warp for a winner tree (0 = none): address and capacity in slots
  u32 sim_base; int sim_cap;
};

// extra demand, per chunk level, of multiplicity r over the least multiplicity r0
__device__ __forceinline__ void extra_demand(int type, int g, int gang, int r0, int r, int d[4]) {
  d[0] = d[1] = d[2] = d[3] = 0;
  if (type != TG_POOL_GPU) { d[0] = g * (r - r0); return; }
  if (gang) {
    int z = g * r, z0 = g * r0, lz = ilog2(z), lz0 = ilog2(z0);
#pragma unroll
    for (int l = 0; l < 4; ++l) if (l <= lz) d[l] = z - (l <= lz0 ? z0 : 0);
  } else {
    int lz = ilog2(g);
#pragma unroll
    for (int l = 0; l < 4; ++l) if (l <= lz) d[l] = g * (r - r0);
  }
}

// smallest multiplicity that already reaches the duration of the largest one
__device__ __forceinline__ int best_level(i64 p, u32 mask) {
  int rmax = 32 - __clz(mask);
  i64 tb = div_small(p, rmax);
  u32 mm = mask;
  while (mm) {
    int r = __ffs(mm); mm &= mm - 1;
    if (div_small(p, r) == tb) return r;
  }
  return rmax;
}

// The box DP for boxes of at most 32 cells: lane c owns cell c, the row before lives in a
// register and a predecessor cell is fetched with one shuffle by the flattened offset.  The rows
// (T.rowcand[0..nrows)) are taken 32 at a time: every lane first lists, for its own row, the
// levels that stay inside the box (multiplicity, offset, extra demand per dimension, duration),
// then the rows are applied one after the other from broadcasts of those lists.  The choices
// (multiplicity and offset, two bytes per cell and row) go to the warp's shared-memory scratch
// at `scratch` (64 bytes per row).  Same recurrence and tie order as the general loop in
// solve_prefix.  Returns 1 when T.rsel holds the optimum; 0 when several end cells tie on value
// and units or a row has more than DPS_LEVELS levels inside the box (the caller then runs the
// general loop).
#define DPS_LEVELS 6
__device__ int dp_small(const PoolTask& T, int nrows, int ncell, const int ext[4], const int stride[4],
                        const bool kept[4], u32 scratch, int lane) {
  // cell coordinates of this lane, one 6-bit field per dimension; bit 5 of a field is a guard
  // that survives the subtraction of a demand iff the demand does not exceed the coordinate
  const u32 GUARD = 0x20u | (0x20u << 6) | (0x20u << 12) | (0x20u << 18);
  u32 pe = GUARD;
  int e0 = 0;
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    const int el = (lane / stride[l]) % ext[l];
    if (l == 0) e0 = el;
    pe |= (u32)el << (6 * l);
  }
  i64 prev = lane == 0 ? 0 : TG_INF;
  const bool via_smem = nrows <= 64;
  for (int t0 = 0; t0 < nrows; t0 += 32) {
    u32 pa[DPS_LEVELS], pb[DPS_LEVELS];                  // r | off << 8 ; demand fields
    i64 du[DPS_LEVELS];
    int nl = 0;
    bool too_many = false;
#pragma unroll
    for (int k = 0; k < DPS_LEVELS; ++k) { pa[k] = 0; pb[k] = 0; du[k] = 0; }
    if (t0 + lane < nrows) {
      const int i = T.rowcand[t0 + lane];
      const i64 s = T.cs[i], p = T.cp[i];
      const u32 mk = T.cmask[i];
      const int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7, r0 = __ffs(mk);
      u32 mm = mk;
      while (mm) {
        const int r = __ffs(mm); mm &= mm - 1;
        int d[4];
        extra_demand(T.type, g, gang, r0, r, d);
        u32 off = 0, dls = 0; bool inside = true;
#pragma unroll
        for (int l = 0; l < 4; ++l)
          if (kept[l]) { const int dl = d[l] >> l; inside &= dl < ext[l]; off += dl * stride[l]; dls |= (u32)(dl & 31) << (6 * l); }
        if (!inside) continue;
        if (nl >= DPS_LEVELS) { too_many = true; break; }
        const i64 dd = duration(s, p, r);
#pragma unroll
        for (int k = 0; k < DPS_LEVELS; ++k) if (k == nl) { pa[k] = (u32)r | (off << 8); pb[k] = dls; du[k] = dd; }
        ++nl;
      }
    }
    if (__any_sync(TG_FULL, too_many)) return 0;
    const int nb = min(32, nrows - t0);
    if (via_smem) {
      // up to 64 rows leave room behind the choices for the level lists of a block of rows: a row's
      // levels are then one broadcast load each instead of four shuffles
      const u32 lists = scratch + 4096u;
      __syncwarp();
#pragma unroll
      for (int k = 0; k < DPS_LEVELS; ++k)
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" :: "r"(lists + (u32)(lane * DPS_LEVELS + k) * 16u),
                     "r"(pa[k]), "r"(pb[k]), "r"((u32)du[k]), "r"((u32)((u64)du[k] >> 32)) : "memory");
      __syncwarp();
      for (int b = 0; b < nb; ++b) {
        // all level entries of the row are loaded before any is used, and the first four are applied without
        // a branch: their loads and shuffles do not depend on one another, only the running minimum does
        u32 va[DPS_LEVELS], vb[DPS_LEVELS], dlo[DPS_LEVELS], dhi[DPS_LEVELS];
#pragma unroll
        for (int k = 0; k < DPS_LEVELS; ++k)
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(va[k]), "=r"(vb[k]), "=r"(dlo[k]), "=r"(dhi[k])
                       : "r"(lists + (u32)(b * DPS_LEVELS + k) * 16u) : "memory");
        i64 best = TG_INF; u32 bestv = 0;
#pragma unroll
        for (int k = 0; k < DPS_LEVELS; ++k) {
          if (k >= 4 && va[k] == 0) break;               // the row has no further level (a multiplicity is never 0)
          const i64 dd = (i64)(((u64)dhi[k] << 32) | dlo[k]);
          const i64 pv = __shfl_up_sync(TG_FULL, prev, va[k] >> 8);
          const bool ok = va[k] != 0 && ((pe - vb[k]) & GUARD) == GUARD && pv != TG_INF;
          const i64 cand = pv + dd;
          if (ok && cand < best) { best = cand; bestv = va[k]; }
        }
        prev = lane < ncell ? best : TG_INF;
        asm volatile("st.shared.u16 [%0], %1;" :: "r"(scratch + (u32)(t0 + b) * 64u + (u32)lane * 2u), "h"((unsigned short)bestv) : "memory");
      }
      continue;
    }
    for (int b = 0; b < nb; ++b) {
      const int nlb = __shfl_sync(TG_FULL, nl, b);
      i64 best = TG_INF; u32 bestv = 0;
#pragma unroll
      for (int k = 0; k < DPS_LEVELS; ++k) {
        if (k < nlb) {                                   // levels ascend: the first best one stays
          const u32 va = __shfl_sync(TG_FULL, pa[k], b), vb = __shfl_sync(TG_FULL, pb[k], b);
          const i64 dd = __shfl_sync(TG_FULL, du[k], b);
          const i64 pv = __shfl_up_sync(TG_FULL, prev, va >> 8);
          const bool ok = ((pe - vb) & GUARD) == GUARD && pv != TG_INF;
          const i64 cand = pv + dd;
          if (ok && cand < best) { best = cand; bestv = va; }
        }
      }
      prev = lane < ncell ? best : TG_INF;
      asm volatile("st.shared.u16 [%0], %1;" :: "r"(scratch + (u32)(t0 + b) * 64u + (u32)lane * 2u), "h"((unsigned short)bestv) : "memory");
    }
  }
  __syncwarp();
  // best end cell: lowest value, then fewest extra units (index along dimension 0)
  const i64 bv = warp_min64(prev);
  if (bv == TG_INF) return 0;
  const int be = warp_min32(prev == bv ? e0 : INT_MAX);
  const u32 win = __ballot_sync(TG_FULL, prev == bv && e0 == be);
  if (__popc(win) != 1) return 0;
  int c = __ffs(win) - 1;
  for (int t = nrows - 1; t >= 0; --t) {                 // walk back, every lane the same path
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(scratch + (u32)t * 64u + (u32)c * 2u) : "memory");
    if (lane == (t & 31)) T.rsel[T.rowcand[t]] = (u8)(v & 0xff);
    c -= v >> 8;
  }
  __syncwarp();
  return 1;
}

// The same DP for several prefixes of the candidate list in one pass: the DP of a prefix is the DP
// of a longer one cut off after the prefix's last row and read inside the prefix's own, smaller
// box.  E lists, per prefix, the number of rows, the largest cell coordinates (6-bit fields) and
// where the multiplicities of the rows go.  Returns the set of prefixes solved (a prefix whose
// end cells tie is left out).
#define DPS_PREFIXES 4
struct DpEnds { int nq; int nrows_k[DPS_PREFIXES]; u32 lim[DPS_PREFIXES]; u8* out[DPS_PREFIXES]; };
__device__ u32 dp_small_multi(const PoolTask& T, int nrows, int ncell, const int ext[4], const int stride[4],
                        const bool kept[4], u32 scratch, int lane, const DpEnds& E) {
  // cell coordinates of this lane, one 6-bit field per dimension; bit 5 of a field is a guard
  // that survives the subtraction of a demand iff the demand does not exceed the coordinate
  const u32 GUARD = 0x20u | (0x20u << 6) | (0x20u << 12) | (0x20u << 18);
  u32 pe = GUARD;
  int e0 = 0;
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    const int el = (lane / stride[l]) % ext[l];
    if (l == 0) e0 = el;
    pe |= (u32)el << (6 * l);
  }
  i64 prev = lane == 0 ? 0 : TG_INF;
  int endc[DPS_PREFIXES], endrow[DPS_PREFIXES];
  u32 endlim[DPS_PREFIXES];
#pragma unroll
  for (int k = 0; k < DPS_PREFIXES; ++k) {
    endc[k] = -1;
    endrow[k] = k < E.nq ? E.nrows_k[k] : -1;            // in registers: the row loop looks at them every row
    endlim[k] = E.lim[k];
  }
  int next_end = INT_MAX;                                // first row count at which a prefix ends
#pragma unroll
  for (int k = 0; k < DPS_PREFIXES; ++k) if (endrow[k] >= 1) next_end = min(next_end, endrow[k]);
  for (int t0 = 0; t0 < nrows; t0 += 32) {
    u32 pa[DPS_LEVELS], pb[DPS_LEVELS];                  // r | off << 8 ; demand fields
    i64 du[DPS_LEVELS];
    int nl = 0;
    bool too_many = false;
#pragma unroll
    for (int k = 0; k < DPS_LEVELS; ++k) { pa[k] = 0; pb[k] = 0; du[k] = 0; }
    if (t0 + lane < nrows) {
      const int i = T.rowcand[t0 + lane];
      const i64 s = T.cs[i], p = T.cp[i];
      const u32 mk = T.cmask[i];
      const int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7, r0 = __ffs(mk);
      u32 mm = mk;
      while (mm) {
        const int r = __ffs(mm); mm &= mm - 1;
        int d[4];
        extra_demand(T.type, g, gang, r0, r, d);
        u32 off = 0, dls = 0; bool inside = true;
#pragma unroll
        for (int l = 0; l < 4; ++l)
          if (kept[l]) { const int dl = d[l] >> l; inside &= dl < ext[l]; off += dl * stride[l]; dls |= (u32)(dl & 31) << (6 * l); }
        if (!inside) continue;
        if (nl >= DPS_LEVELS) { too_many = true; break; }
        const i64 dd = duration(s, p, r);
#pragma unroll
        for (int k = 0; k < DPS_LEVELS; ++k) if (k == nl) { pa[k] = (u32)r | (off << 8); pb[k] = dls; du[k] = dd; }
        ++nl;
      }
    }
    if (__any_sync(TG_FULL, too_many)) return 0;
    const int nb = min(32, nrows - t0);
    for (int b = 0; b < nb; ++b) {
      const int nlb = __shfl_sync(TG_FULL, nl, b);
      i64 best = TG_INF; u32 bestv = 0;
#pragma unroll
      for (int k = 0; k < DPS_LEVELS; ++k) {
        if (k < nlb) {                                   // levels ascend: the first best one stays
          const u32 va = __shfl_sync(TG_FULL, pa[k], b), vb = __shfl_sync(TG_FULL, pb[k], b);
          const i64 dd = __shfl_sync(TG_FULL, du[k], b);
          const i64 pv = __shfl_up_sync(TG_FULL, prev, va >> 8);
          const bool ok = ((pe - vb) & GUARD) == GUARD && pv != TG_INF;
          const i64 cand = pv + dd;
          if (ok && cand < best) { best = cand; bestv = va; }
        }
      }
      prev = lane < ncell ? best : TG_INF;
      asm volatile("st.shared.u16 [%0], %1;" :: "r"(scratch + (u32)(t0 + b) * 64u + (u32)lane * 2u), "h"((unsigned short)bestv) : "memory");
      if (t0 + b + 1 == next_end) {
      next_end = INT_MAX;
#pragma unroll
      for (int k = 0; k < DPS_PREFIXES; ++k) {
        if (endrow[k] > t0 + b + 1) next_end = min(next_end, endrow[k]);
        if (endrow[k] == t0 + b + 1) {
          // best end cell of this prefix inside its own box: lowest value, then fewest extra units
          // (index along dimension 0); several such cells: left to the general loop
          const bool in = (((endlim[k] | GUARD) - (pe & ~GUARD)) & GUARD) == GUARD;
          const i64 pv = in ? prev : TG_INF;
          const i64 bv = warp_min64(pv);
          const int be = warp_min32((pv == bv && bv != TG_INF) ? e0 : INT_MAX);
          const u32 win = __ballot_sync(TG_FULL, pv == bv && bv != TG_INF && e0 == be);
          if (__popc(win) == 1) endc[k] = __ffs(win) - 1;
        }
      }
      }
    }
  }
  __syncwarp();
  u32 solved = 0;
#pragma unroll
  for (int k = 0; k < DPS_PREFIXES; ++k) {
    if (k >= E.nq || endc[k] < 0) continue;
    int c = endc[k];
    u8* out = E.out[k];
    for (int t = E.nrows_k[k] - 1; t >= 0; --t) {        // walk back, every lane the same path
      unsigned short v;
      asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(scratch + (u32)t * 64u + (u32)c * 2u) : "memory");
      if (lane == (t & 31)) out[T.rowcand[t]] = (u8)(v & 0xff);
      c -= v >> 8;
    }
    solved |= 1u << k;
  }
  __syncwarp();
  return solved;
}

// ---- marginal gains of a class of rows whose steps all have the same size ------------------
// A row with contiguous multiplicities r0 .. rmax offers the steps r0 -> r0+1 -> ... each worth one
// chunk of the class's size; step k (1-based) gains T(r0+k-1) - T(r0+k) >= 0.  If every row's gains
// are non-increasing (the floor in Eq. 1 can break that; such a class goes through its DP), the
// least duration sum with exactly x extra chunks is the sum at the least levels minus the x
// largest gains (separable convex resource allocation), and among allocations of equal value the
// canonical order (a later queue position gets less) takes equal gains from the earliest rows
// first.  So the steps are sorted by one key: gain descending, row ascending, step ascending, and
// every x is served by a prefix of that order; an allocation is read back from the threshold
// key at the cut.  All steps of a class have the same size, so comparing gains is comparing
// densities; nothing is divided.
#define MG_GAIN_BITS 41
#define MG_ROW_BITS 18
#define MG_GAIN_MAX ((1ull << MG_GAIN_BITS) - 1ull)
__device__ __forceinline__ u64 mg_key(i64 gain, int row, int step) {     // step 1-based, at most 31
  return ((MG_GAIN_MAX - (u64)gain) << (MG_ROW_BITS + 5)) | ((u64)row << 5) | (u64)(step - 1);
}
__device__ __forceinline__ i64 mg_gain(u64 key) { return (i64)(MG_GAIN_MAX - (key >> (MG_ROW_BITS + 5))); }
// contiguous multiplicities and non-increasing gains
__device__ __forceinline__ bool mg_row_ok(i64 s, i64 p, u32 mk) {
  const int r0 = __ffs(mk), rmax = 32 - __clz(mk);
  if (mk != ((rmax == 32 ? 0xffffffffu : ((1u << rmax) - 1u)) & ~((1u << (r0 - 1)) - 1u))) return false;
  i64 before = duration(s, p, r0), last_gain = TG_INF;
  for (int r = r0 + 1; r <= rmax; ++r) {
    const i64 now = duration(s, p, r), gain = before - now;
    if (gain > last_gain) return false;
    last_gain = gain; before = now;
  }
  return true;
}
// ascending bitonic sort of n (a power of two) keys by the calling warp
__device__ __forceinline__ void warp_sort_u64(u64* a, int n, int lane) {
  for (int k = 2; k <= n; k <<= 1)
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = lane; i < n; i += 32) {
        const int l = i ^ j;
        if (l > i) {
          const u64 x = a[i], y = a[l];
          if ((x > y) == ((i & k) == 0)) { a[i] = y; a[l] = x; }
        }
      }
      __syncwarp();
    }
}

// DPArrange on a fragmented GPU pool (Algorithm 4) when no row is a gang request: a row of chunk
// size 2^c only ever adds requests of that size, so the rows fall into four classes that
// interact through nothing but the nested capacities (extra GPUs at sizes >= 2^l <= Y[l]).  Per
// class a one-dimensional DP over "extra chunks of this size" gives f_c(x) = least duration sum of
// the class with exactly x extra chunks (same recurrence and tie order as the general loop);
// the classes are then merged from the largest size down,
//   G_c(e) = min over x of G_{c+1}((e - x) / 2) + f_c(x),   e <= Y[c] >> c  (e in chunks of 2^c),
// which replaces a table over the product of the four extents by tables over each of them.
// If two different splits between classes tie on a cell of the chosen path, the canonical order
// among them is not decided here: the function then returns 0 and the caller runs the general
// loop (as it does when the scratch does not suffice).  Rows are T.rowcand[0..nrows).
#define DPC_MAX_CELLS 4096
__device__ __noinline__ int dp_classes(const PoolTask& T, int nrows, const int Y[4], const int maxex[4], Slab slab, int lane) {
  // class sizes; which classes can go by their marginal gains
  int rows_c[4] = {0, 0, 0, 0}, mx_c[4] = {0, 0, 0, 0};  // rows and largest extra chunks per class
  bool gang_row = false;
  u32 not_convex = 0;
  i64 base_c[4] = {0, 0, 0, 0};                          // duration sum of the class at the least levels
  for (int t = lane; t < nrows; t += 32) {
    const int i = T.rowcand[t];
    const int g = T.cg[i] & 0x7f;
    if (T.cg[i] >> 7) gang_row = true;
    const u32 mk = T.cmask[i];
    const int c = ilog2(g), ex = (32 - __clz(mk)) - __ffs(mk);
    const i64 s = T.cs[i], p = T.cp[i];
    const i64 tl = duration(s, p, __ffs(mk));
    if (!mg_row_ok(s, p, mk)) not_convex |= 1u << c;
#pragma unroll
    for (int l = 0; l < 4; ++l) if (l == c) { rows_c[l] += 1; mx_c[l] += ex; base_c[l] += tl; }
  }
  if (__any_sync(TG_FULL, gang_row)) return 0;
  not_convex = __reduce_or_sync(TG_FULL, not_convex);
  int U[4];                                               // largest useful number of extra chunks per class
  bool by_gain[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    rows_c[l] = warp_sum32(rows_c[l]); mx_c[l] = warp_sum32(mx_c[l]); base_c[l] = warp_sum64(base_c[l]);
    U[l] = min(max(Y[l], 0) >> l, mx_c[l]);
    if (U[l] + 1 > DPC_MAX_CELLS || (Y[l] >> l) + 1 > 2 * DPC_MAX_CELLS) return 0;
    by_gain[l] = !((not_convex >> l) & 1u) && nrows < (1 << MG_ROW_BITS) && mx_c[l] >= 1;
  }
  (void)maxex;
  // scratch: per class f (final values), two work rows, choices or sorted step keys; merged tables
  i64* f[4]; u8* ch[4]; u64* keys[4]; int npad[4];
  i64* work = nullptr;
  int Umax = max(max(U[0], U[1]), max(U[2], U[3]));
  work = (i64*)slab.take(2 * (u64)(Umax + 1) * 8);
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    f[l] = (i64*)slab.take((u64)(U[l] + 1) * 8);
    npad[l] = 1;
    while (npad[l] < mx_c[l]) npad[l] <<= 1;
    keys[l] = by_gain[l] ? (u64*)slab.take((u64)npad[l] * 8) : nullptr;
    ch[l] = by_gain[l] ? (u8*)f[l] : (u8*)slab.take((u64)max(rows_c[l], 1) * (U[l] + 1));
    if (by_gain[l] && !keys[l]) return 0;
  }
  // merged tables: E[l] cells in chunks of 2^l, value, chosen cell of the level above, tie flag
  int E[4];
  i64* G[4]; int* gsel[4]; u8* gtie[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    E[l] = max(Y[l], 0) >> l;
    G[l] = (i64*)slab.take((u64)(E[l] + 1) * 8);
    gsel[l] = (int*)slab.take((u64)(E[l] + 1) * 4);
    gtie[l] = (u8*)slab.take((u64)(E[l] + 1));
  }
  if (!work || !gtie[3] || !gtie[0] || !ch[3] || !ch[0]) return 0;
#pragma unroll
  for (int l = 0; l < 4; ++l) if (!f[l] || !ch[l] || !G[l] || !gsel[l] || !gtie[l]) return 0;

  // ---- step keys of the classes that go by their gains: every row writes its steps behind those
  // ---- of the rows before it (one scan per class and block of 32 rows)
  {
    int fill[4] = {0, 0, 0, 0};
    for (int t0 = 0; t0 < nrows; t0 += 32) {
      const int t = t0 + lane;
      int c = -1, ex = 0, r0 = 1; i64 s = 0, p = 0;
      if (t < nrows) {
        const int i = T.rowcand[t];
        const u32 mk = T.cmask[i];
        c = ilog2(T.cg[i] & 0x7f); r0 = __ffs(mk); ex = (32 - __clz(mk)) - r0;
        s = T.cs[i]; p = T.cp[i];
      }
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        if (!by_gain[l]) continue;
        const int mine = c == l ? ex : 0;
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(TG_FULL, incl, o); if (lane >= o) incl += y; }
        if (c == l) {
          u64* dst = keys[l] + fill[l] + incl - mine;
          i64 before = duration(s, p, r0);
          for (int k = 1; k <= ex; ++k) {
            const i64 now = duration(s, p, r0 + k);
            dst[k - 1] = mg_key(before - now, t, k);
            before = now;
          }
        }
        fill[l] += __shfl_sync(TG_FULL, incl, 31);
      }
    }
#pragma unroll
    for (int l = 0; l < 4; ++l)
      if (by_gain[l]) for (int x = mx_c[l] + lane; x < npad[l]; x += 32) keys[l][x] = ~0ull;
    __syncwarp();
  }

  // ---- per class: f_c(x), least duration sum with exactly x extra chunks
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    const int Uc = U[c];
    if (by_gain[c]) {
      // sorted steps (in the warp's shared memory when they fit), then f_c(x) = base - the x largest gains
      u64* srt = keys[c];
      const int n = npad[c];
      if (T.sim_base && n * 8 <= T.sim_cap * 16) {
        u64* sm = (u64*)__cvta_shared_to_generic((size_t)T.sim_base);
        for (int x = lane; x < n; x += 32) sm[x] = srt[x];
        __syncwarp();
        warp_sort_u64(sm, n, lane);
        for (int x = lane; x < n; x += 32) srt[x] = sm[x];
        __syncwarp();
      } else warp_sort_u64(srt, n, lane);
      i64 run = base_c[c];                               // f_c at the start of the block of 32
      for (int x0 = 0; x0 <= Uc; x0 += 32) {
        // f_c(x0 + lane) = run - gains of the steps x0 .. x0+lane-1 (an exclusive scan)
        const int x = x0 + lane;
        i64 gsum = (x >= 1 && x <= Uc) ? mg_gain(srt[x - 1]) : 0;   // lane holds the gain of step x-1
        if (x0 > 0 && lane == 0) gsum = 0;               // step x0-1 went into `run` already
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const i64 y = __shfl_up_sync(TG_FULL, gsum, o); if (lane >= o) gsum += y; }
        if (x <= Uc) f[c][x] = run - gsum;
        // carry: f_c(x0 + 32) needs the gain of step x0+31 as well
        const i64 tail = (x0 + 32 <= Uc) ? mg_gain(srt[x0 + 31]) : 0;
        run = run - __shfl_sync(TG_FULL, gsum, 31) - tail;
      }
      __syncwarp();
      continue;
    }
    i64* prev = work; i64* cur = work + (Umax + 1);
    for (int u = lane; u <= Uc; u += 32) prev[u] = u == 0 ? 0 : TG_INF;
    __syncwarp();
    int tc = 0;
    for (int t = 0; t < nrows; ++t) {
      const int i = T.rowcand[t];
      if (ilog2(T.cg[i] & 0x7f) != c) continue;
      const u32 mk = T.cmask[i];
      const int r0 = __ffs(mk);
      const i64 s = T.cs[i], p = T.cp[i];
      u8* chr = ch[c] + (u64)tc * (Uc + 1);
      for (int u = lane; u <= Uc; u += 32) {
        i64 best = TG_INF; int bestr = 0;
        u32 mm = mk;
        while (mm) {
          const int r = __ffs(mm); mm &= mm - 1;
          const int du = r - r0;
          if (du > u) break;                              // levels ascend
          const i64 pv = prev[u - du];
          if (pv == TG_INF) continue;
          const i64 cand = pv + duration(s, p, r);
          if (cand < best) { best = cand; bestr = r; }
        }
        cur[u] = best; chr[u] = (u8)bestr;
      }
      __syncwarp();
      i64* tmp = prev; prev = cur; cur = tmp;
      ++tc;
    }
    for (int u = lane; u <= Uc; u += 32) f[c][u] = prev[u];
    __syncwarp();
  }
  // ---- merge, largest chunks first
  for (int e = lane; e <= E[3]; e += 32) { G[3][e] = e <= U[3] ? f[3][e] : TG_INF; gsel[3][e] = 0; gtie[3][e] = 0; }
  __syncwarp();
#pragma unroll 1
  for (int c = 2; c >= 0; --c) {
    const int Ec = E[c], Uc = U[c], Eup = E[c + 1];
    for (int e = lane; e <= Ec; e += 32) {
      i64 best = TG_INF; int bu = 0; bool tie = false;
      for (int up = 0; up <= Eup && 2 * up <= e; ++up) {
        const int x = e - 2 * up;
        if (x > Uc) continue;
        const i64 a = G[c + 1][up], b = f[c][x];
        if (a == TG_INF || b == TG_INF) continue;
        const i64 cand = a + b;
        if (cand < best) { best = cand; bu = up; tie = gtie[c + 1][up] != 0; }
        else if (cand == best) tie = true;
      }
      G[c][e] = best; gsel[c][e] = bu; gtie[c][e] = tie ? 1 : 0;
    }
    __syncwarp();
  }
  // ---- best end cell: lowest value, then fewest extra GPUs
  i64 bv = TG_INF;
  for (int e = lane; e <= E[0]; e += 32) bv = min(bv, G[0][e]);
  bv = warp_min64(bv);
  if (bv == TG_INF) return 0;
  int be = INT_MAX;
  for (int e = lane; e <= E[0]; e += 32) if (G[0][e] == bv) be = min(be, e);
  be = warp_min32(be);
  // ---- walk back: cells of the merged tables, then the rows of every class
  int cell[4];
  cell[0] = be;
  bool tied = gtie[0][be] != 0;
#pragma unroll
  for (int c = 0; c < 3; ++c) cell[c + 1] = gsel[c][cell[c]];
  if (tied) return 0;
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    int u = c < 3 ? cell[c] - 2 * cell[c + 1] : cell[3];
    const int Uc = U[c];
    if (by_gain[c]) {
      // the x steps in front of the sorted order are taken: a row gets its steps up to the threshold key
      const u64 thr = u >= 1 ? keys[c][u - 1] : 0ull;
      for (int t = lane; t < nrows; t += 32) {
        const int i = T.rowcand[t];
        if (ilog2(T.cg[i] & 0x7f) != c) continue;
        const u32 mk = T.cmask[i];
        const int r0 = __ffs(mk), ex = (32 - __clz(mk)) - r0;
        const i64 s = T.cs[i], p = T.cp[i];
        int take = 0;
        if (u >= 1) {
          i64 before = duration(s, p, r0);
          for (int k = 1; k <= ex; ++k) {
            const i64 now = duration(s, p, r0 + k);
            if (mg_key(before - now, t, k) > thr) break;  // a row's keys ascend with the step
            take = k; before = now;
          }
        }
        T.rsel[i] = (u8)(r0 + take);
      }
      continue;
    }
    int tc = rows_c[c];
    if (lane == 0) {
      for (int t = nrows - 1; t >= 0; --t) {
        const int i = T.rowcand[t];
        if (ilog2(T.cg[i] & 0x7f) != c) continue;
        --tc;
        const int r = ch[c][(u64)tc * (Uc + 1) + u];
        T.rsel[i] = (u8)r;
        u -= r - __ffs(T.cmask[i]);
      }
    }
  }
  __syncwarp();
  return 1;
}

// The box DP on the REACHABLE cells only, for boxes whose dense table would not fit: Algorithm 4's
// state space is the product of the four chunk-count ranges, but a row only moves a state by one of
// a handful of demand vectors, so few cells are ever reached.  A state is the extra-demand vector
// packed into one key (one bit field per kept dimension); the states of a row are built from those
// of the row before through a hash table (open addressing; a cell keeps the least
// duration sum << 6 | multiplicity, i.e. the lowest value and among equals the smallest level,
// which is what the dense loop's ascending levels with strict '<' keep), compacted into the next
// list, and their (key, multiplicity) pairs are kept per row for the walk back.  Same end-cell rule
// as the dense loop: lowest value, then fewest extra units, then the allocations compared from the
// last row down.  Everything lives in [mem, mem + bytes).  Returns 1 (T.rsel written), 0 if the
// memory does not suffice or a value outgrows its field.
#define SP_EMPTY 0xffffffffffffffffull
__device__ __forceinline__ u64 sp_hash(u64 k) { k ^= k >> 29; k *= 0xbf58476d1ce4e5b9ull; k ^= k >> 32; return k; }
__device__ __noinline__ int dp_sparse(const PoolTask& T, int nrows, const int ext[4], const bool kept[4],
                                      char* mem, u64 bytes, int lane) {
  // bit fields of a key
  int shift[4], width[4], total_bits = 0;
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    width[l] = kept[l] ? 32 - __clz(max(ext[l] - 1, 1)) : 0;
    shift[l] = total_bits; total_bits += width[l];
  }
  if (total_bits > 60) return 0;
  // memory: two state lists and the hash table at the end, the rows' (key, multiplicity) pairs from the front
  const u64 cap_states = bytes / 2 / (2 * 16 + 4 * 16);          // each list 16 B per state, table 4 slots of 16 B per state
  if (cap_states < 64) return 0;
  u64* lk[2]; i64* lv[2];
  char* top = mem + bytes;
  u64 tab_slots = 1; while (tab_slots < 4 * cap_states) tab_slots <<= 1; tab_slots >>= 1;   // largest power of two <= 4 cap
  top -= tab_slots * 16; u64* tk = (u64*)top; u64* tv = tk + tab_slots;
  for (int x = 0; x < 2; ++x) { top -= cap_states * 16; lk[x] = (u64*)top; lv[x] = (i64*)(lk[x] + cap_states); }
  char* store = mem;                                             // grows towards `top`
  // per row: where its pairs start and how many (kept in the store itself, in front of the pairs)
  u64* row_dir = (u64*)store; store += (u64)nrows * 16;
  if (store > top) return 0;
  u64 n = 1;
  if (lane == 0) { lk[0][0] = 0; lv[0][0] = 0; }
  __syncwarp();
  int cur = 0;
  for (int t = 0; t < nrows; ++t) {
    const int i = T.rowcand[t];
    const int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7;
    const u32 mk = T.cmask[i];
    const int r0 = __ffs(mk), nlev = __popc(mk);
    const i64 s = T.cs[i], p = T.cp[i];
    // table of this row: a power of two of at least four slots per candidate state
    u64 want = n * (u64)nlev * 2, slots = 64;
    while (slots < want && slots < tab_slots) slots <<= 1;
    for (u64 x = lane; x < slots; x += 32) { tk[x] = SP_EMPTY; tv[x] = ~0ull; }
    __syncwarp();
    u64 distinct = 0;
    bool fail = false;
    for (u64 x0 = 0; x0 < n; x0 += 32) {
      const u64 x = x0 + lane;
      const bool on = x < n;
      const u64 key = on ? lk[cur][x] : 0;
      const i64 val = on ? lv[cur][x] : 0;
      u32 mm = mk;
      while (mm) {
        const int r = __ffs(mm); mm &= mm - 1;
        int d[4];
        extra_demand(T.type, g, gang, r0, r, d);
        u64 nk = key; bool inside = on;
#pragma unroll
        for (int l = 0; l < 4; ++l)
          if (kept[l]) {
            const int dl = d[l] >> l;
            const int e = (int)((key >> shift[l]) & ((1ull << width[l]) - 1ull));
            inside &= e + dl < ext[l];
            nk += (u64)dl << shift[l];
          }
        const i64 cand = val + duration(s, p, r);
        if (inside && cand >= (1ll << 56)) { fail = true; inside = false; }
        if (inside) {
          const u64 packed = ((u64)cand << 6) | (u64)r;
          u64 h = sp_hash(nk) & (slots - 1);
          for (u64 probe = 0; probe < slots; ++probe) {
            const u64 seen = atomicCAS((unsigned long long*)&tk[h], SP_EMPTY, nk);
            if (seen == SP_EMPTY || seen == nk) { atomicMin((unsigned long long*)&tv[h], packed); if (seen == SP_EMPTY) ++distinct; break; }
            h = (h + 1) & (slots - 1);
            if (probe + 1 == slots) fail = true;
          }
        }
      }
    }
    __syncwarp();
    distinct = (u64)warp_sum64((i64)distinct);
    if (__any_sync(TG_FULL, fail) || distinct > cap_states || distinct > slots / 2 + 32) return 0;
    // compact the table into the next list and into the row's store
    if (store + distinct * 16 > top) return 0;
    u64* sk = (u64*)store; u64* sr = sk + distinct;
    if (lane == 0) { row_dir[2 * t] = (u64)(store - mem); row_dir[2 * t + 1] = distinct; }
    store += distinct * 16;
    u64 filled = 0;
    for (u64 x0 = 0; x0 < slots; x0 += 32) {
      const u64 x = x0 + lane;
      const u64 k = tk[x];
      const bool has = k != SP_EMPTY;
      const u32 b = __ballot_sync(TG_FULL, has);
      if (has) {
        const u64 at = filled + __popc(b & ((1u << lane) - 1u));
        const u64 pv = tv[x];
        lk[cur ^ 1][at] = k; lv[cur ^ 1][at] = (i64)(pv >> 6);
        sk[at] = k; sr[at] = pv & 63ull;
      }
      filled += __popc(b);
    }
    __syncwarp();
    n = distinct; cur ^= 1;
  }
  // best end state: lowest value, then fewest extra units (dimension 0)
  const u64 m0 = (1ull << width[0]) - 1ull;
  i64 bv = TG_INF;
  for (u64 x = lane; x < n; x += 32) bv = min(bv, lv[cur][x]);
  bv = warp_min64(bv);
  if (bv == TG_INF) return 0;
  int be = INT_MAX;
  for (u64 x = lane; x < n; x += 32) if (lv[cur][x] == bv) be = min(be, (int)((lk[cur][x] >> shift[0]) & m0));
  be = warp_min32(be);
  // the tied end states walk back together; at each row (last first) those with the smallest multiplicity stay
  const int TIE_CAP = 32;
  u64 tied = SP_EMPTY;                                     // lane x holds the x-th tied key
  int nt = 0;
  for (u64 x0 = 0; x0 < n; x0 += 32) {
    const u64 x = x0 + lane;
    const bool hit = x < n && lv[cur][x] == bv && (int)((lk[cur][x] >> shift[0]) & m0) == be;
    const u32 b = __ballot_sync(TG_FULL, hit);
    if (nt + __popc(b) > TIE_CAP) return 0;
    // hand the hits to lanes nt, nt+1, ...
    for (u32 bb = b; bb; bb &= bb - 1) {
      const int src = __ffs(bb) - 1;
      const u64 k = __shfl_sync(TG_FULL, hit ? lk[cur][x] : 0ull, src);
      if (lane == nt) tied = k;
      ++nt;
    }
  }
  for (int t = nrows - 1; t >= 0; --t) {
    const int i = T.rowcand[t];
    const u64* sk = (const u64*)(mem + row_dir[2 * t]);
    const u64 cnt = row_dir[2 * t + 1];
    const u64* sr = sk + cnt;
    // every tied key looks up its multiplicity in this row (all lanes scan for one key at a time)
    int myr = 255;
    for (int y = 0; y < nt; ++y) {
      const u64 k = __shfl_sync(TG_FULL, tied, y);
      int found = 255;
      for (u64 x = lane; x < cnt; x += 32) if (sk[x] == k) found = (int)sr[x];
      found = warp_min32(found);
      if (lane == y) myr = found;
    }
    const int rm = warp_min32(lane < nt ? myr : 255);
    if (rm == 255) return 0;                               // cannot happen: every kept key was written by this row
    if (lane == 0) T.rsel[i] = (u8)rm;
    int d[4];
    extra_demand(T.type, T.cg[i] & 0x7f, T.cg[i] >> 7, __ffs(T.cmask[i]), rm, d);
    u64 delta = 0;
#pragma unroll
    for (int l = 0; l < 4; ++l) if (kept[l]) delta += (u64)(d[l] >> l) << shift[l];
    // keep the keys whose multiplicity is the smallest, move them to the row before, drop duplicates
    const bool stay = lane < nt && myr == rm;
    const u64 prevk = tied - delta;
    const u32 sb = __ballot_sync(TG_FULL, stay);
    u64 next = SP_EMPTY;
    int nn = 0;
    for (u32 bb = sb; bb; bb &= bb - 1) {
      const int src = __ffs(bb) - 1;
      const u64 k = __shfl_sync(TG_FULL, prevk, src);
      const bool dup = __any_sync(TG_FULL, lane < nn && next == k);
      if (!dup) { if (lane == nn) next = k; ++nn; }
    }
    tied = next; nt = nn;
  }
  __syncwarp();
  return 1;
}

// Optimal allocation of candidates [0, q) -> T.rsel[0..q), duration sum -> *opt.
// *all_best tells that every candidate got its best level (then so does every shorter prefix).
// Returns false if the workspace is too small.
__device__ bool solve_prefix(const Params& P, const PoolTask& T, int q, Slab slab, int lane, i64* opt,
                             bool* all_best = nullptr) {
  if (all_best) *all_best = false;
  const bool gpu = T.type == TG_POOL_GPU;
  int dmin[4] = {0, 0, 0, 0}, dbest[4] = {0, 0, 0, 0};
  i64 tmin_sum = 0, tbest_sum = 0;
  for (int i = lane; i < q; i += 32) {
    int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7;
    u32 mk = T.cmask[i];
    int r0 = __ffs(mk), rb = best_level(T.cp[i], mk);
    int lz0 = gpu ? level_of(g, gang, r0) : 0, lzb = gpu ? level_of(g, gang, rb) : 0;
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      if (l <= lz0) dmin[l] += g * r0;
      if (l <= lzb) dbest[l] += g * rb;
    }
    tmin_sum += duration(T.cs[i], T.cp[i], r0);
    tbest_sum += duration(T.cs[i], T.cp[i], rb);
  }
  bool fits_best = true;
  int Y[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    dmin[l] = warp_sum32(dmin[l]); dbest[l] = warp_sum32(dbest[l]);
    Y[l] = T.cap[l] - dmin[l];
    if (l == 0 || gpu) fits_best &= dbest[l] <= T.cap[l];
  }
  tmin_sum = warp_sum64(tmin_sum); tbest_sum = warp_sum64(tbest_sum);
  if (fits_best) {
    for (int i = lane; i < q; i += 32) T.rsel[i] = (u8)best_level(T.cp[i], T.cmask[i]);
    __syncwarp();
    *opt = tbest_sum;
    if (all_best) *all_best = true;
    return true;
  }
  if (Y[0] <= 0) {
    for (int i = lane; i < q; i += 32) T.rsel[i] = (u8)__ffs(T.cmask[i]);
    __syncwarp();
    *opt = tmin_sum;
    return true;
  }

  // ---- DP over the box of feasible extra-demand vectors
  int nrows = 0;
  int maxex[4] = {0, 0, 0, 0};
  for (int i0 = 0; i0 < q; i0 += 32) {
    int i = i0 + lane;
    bool el = false;
    if (i < q) {
      u32 mk = T.cmask[i];
      el = (mk & (mk - 1)) != 0;
      T.rsel[i] = (u8)__ffs(mk);
      if (el) {
        int d[4];
        extra_demand(T.type, T.cg[i] & 0x7f, T.cg[i] >> 7, __ffs(mk), 32 - __clz(mk), d);
#pragma unroll
        for (int l = 0; l < 4; ++l) maxex[l] += d[l];
      }
    }
    u32 b = __ballot_sync(TG_FULL, el);
    if (el) T.rowcand[nrows + __popc(b & ((1u << lane) - 1u))] = i;
    nrows += __popc(b);
  }
  int ext[4], stride[4];
  bool kept[4];
  u64 cells = 1;
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    maxex[l] = warp_sum32(maxex[l]);
    kept[l] = l == 0 || (gpu && T.cap[l] < T.cap[l - 1]);
    int bound = min(Y[l], maxex[l]);
    ext[l] = kept[l] ? (max(bound, 0) >> l) + 1 : 1;
    stride[l] = (int)cells;
    if (cells <= (1ull << 30)) cells *= (u64)ext[l];
  }
  __syncwarp();
  // (the out-of-line routines get a copy of the task, so that this one can stay in registers)
  if (gpu && cells > 32 && (kept[1] || kept[2] || kept[3]) && dp_classes(PoolTask(T), nrows, Y, maxex, slab, lane)) {
    i64 sum = 0;
    for (int i = lane; i < q; i += 32) sum += duration(T.cs[i], T.cp[i], T.rsel[i]);
    *opt = warp_sum64(sum);
    return true;
  }
  if (cells > (1ull << 30)) cells = (1ull << 30) + 1;       // (never dense: the reachable cells only, below)
  const int ncell = (int)cells;
  if (ncell <= 32 && T.sim_base && nrows * 4 <= T.sim_cap &&
      dp_small(T, nrows, ncell, ext, stride, kept, T.sim_base, lane)) {
    i64 sum = 0;
    for (int i = lane; i < q; i += 32) sum += duration(T.cs[i], T.cp[i], T.rsel[i]);
    *opt = warp_sum64(sum);
    return true;
  }
  i64* val = (i64*)slab.take(2 * cells * sizeof(i64));
  u8* choice = val ? (u8*)slab.take((u64)nrows * cells) : nullptr;
  const int slot = -1;
  if (!choice) {
    // the dense table does not fit the warp's slab: only the reachable cells, in a borrowed slot of the arena
    const int sl = slot_acquire(P, 1, lane);
    if (sl < 0) return false;
    const int done = dp_sparse(PoolTask(T), nrows, ext, kept, slot_ptr(P, sl), arena_slot_bytes(P), lane);
    slot_release(P, sl, lane);
    if (!done) return false;
    i64 sum = 0;
    for (int i = lane; i < q; i += 32) sum += duration(T.cs[i], T.cp[i], T.rsel[i]);
    *opt = warp_sum64(sum);
    return true;
  }
  i64* prev = val; i64* cur = val + cells;
  for (int c = lane; c < ncell; c += 32) prev[c] = c == 0 ? 0 : TG_INF;
  __syncwarp();
  for (int t = 0; t < nrows; ++t) {
    const int i = T.rowcand[t];
    const int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7;
    const u32 mk = T.cmask[i];
    const int r0 = __ffs(mk);
    const i64 s = T.cs[i], p = T.cp[i];
    u8* ch = choice + (u64)t * cells;
    for (int c = lane; c < ncell; c += 32) {
      int e[4];
#pragma unroll
      for (int l = 0; l < 4; ++l) e[l] = (c / stride[l]) % ext[l];
      i64 best = TG_INF; int bestr = 0;
      u32 mm = mk;
      while (mm) {
        int r = __ffs(mm); mm &= mm - 1;
        int d[4];
        extra_demand(T.type, g, gang, r0, r, d);
        int off = 0; bool ok = true;
#pragma unroll
        for (int l = 0; l < 4; ++l)
          if (kept[l]) { int dl = d[l] >> l; ok &= dl <= e[l]; off += dl * stride[l]; }
        if (!ok) continue;
        i64 pv = prev[c - off];
        if (pv == TG_INF) continue;
        i64 cand = pv + duration(s, p, r);
        if (cand < best) { best = cand; bestr = r; }
      }
      cur[c] = best; ch[c] = (u8)bestr;
    }
    __syncwarp();
    i64* tmp = prev; prev = cur; cur = tmp;
  }
  // best cell of the last row: lowest value, then fewest extra units (e_1 = index along dim 0)
  i64 bv = TG_INF;
  for (int c = lane; c < ncell; c += 32) bv = min(bv, prev[c]);
  bv = warp_min64(bv);
  if (bv == TG_INF) { slot_release(P, slot, lane); return false; }   // cannot happen for an accommodated prefix
  int be = INT_MAX;
  for (int c = lane; c < ncell; c += 32) if (prev[c] == bv) be = min(be, c % ext[0]);
  be = warp_min32(be);
  int cnt = 0, bc = -1;
  for (int c = lane; c < ncell; c += 32) if (prev[c] == bv && c % ext[0] == be) { ++cnt; bc = max(bc, c); }
  cnt = warp_sum32(cnt); bc = warp_max32(bc);
  int fail = 0;
  if (lane == 0) {
    if (cnt == 1) {
      int c = bc;
      for (int t = nrows - 1; t >= 0; --t) {
        int i = T.rowcand[t];
        int r = choice[(u64)t * cells + c];
        T.rsel[i] = (u8)r;
        int d[4];
        extra_demand(T.type, T.cg[i] & 0x7f, T.cg[i] >> 7, __ffs(T.cmask[i]), r, d);
#pragma unroll
        for (int l = 0; l < 4; ++l) if (kept[l]) c -= (d[l] >> l) * stride[l];
      }
    } else {
      // several end cells tie on value and units: walk back all of them at once, keeping at
      // each task (latest first) the cells whose choice is the smallest
      const int TIE_CAP = 64;
      int lst[TIE_CAP], nl = 0;
      for (int c = 0; c < ncell; ++c)
        if (prev[c] == bv && c % ext[0] == be) { if (nl < TIE_CAP) lst[nl++] = c; else fail = 1; }
      for (int t = nrows - 1; t >= 0; --t) {
        int i = T.rowcand[t];
        const u8* ch = choice + (u64)t * cells;
        int rm = 255;
        for (int x = 0; x < nl; ++x) rm = min(rm, (int)ch[lst[x]]);
        T.rsel[i] = (u8)rm;
        int d[4];
        extra_demand(T.type, T.cg[i] & 0x7f, T.cg[i] >> 7, __ffs(T.cmask[i]), rm, d);
        int off = 0;
#pragma unroll
        for (int l = 0; l < 4; ++l) if (kept[l]) off += (d[l] >> l) * stride[l];
        int nn = 0;
        for (int x = 0; x < nl; ++x) {
          if (ch[lst[x]] != rm) continue;
          int c = lst[x] - off;
          bool dup = false;
          for (int y = 0; y < nn; ++y) dup |= lst[y] == c;
          if (!dup) lst[nn++] = c;
        }
        nl = nn;
      }
    }
  }
  fail = __shfl_sync(TG_FULL, fail, 0);
  slot_release(P, slot, lane);
  if (fail) return false;
  __syncwarp();
  i64 sum = 0;
  for (int i = lane; i < q; i += 32) sum += duration(T.cs[i], T.cp[i], T.rsel[i]);
  *opt = warp_sum64(sum);
  return true;
}

// Optimal allocations of the prefixes q0, q0-1, .., q0-nq+1 (nq <= DPS_PREFIXES) in one go: out[k]
// receives the multiplicities of prefix q0-k, opt[k] its duration sum.  Same results as
// solve_prefix for each of them.  The sums of a shorter prefix follow from the longer one by taking
// one candidate out, the certificates are applied per prefix, and the prefixes that need the DP
// share one pass of dp_small over the rows of the longest.  Returns the set of prefixes done; the
// others (a box beyond 32 cells, tied end cells, ...) are left to solve_prefix.
// *all_best: the longest prefix, and hence every one, has all candidates at their best level.
__device__ __noinline__ u32 solve_multi(const PoolTask& T, int q0, int nq, u8* const out[DPS_PREFIXES],
                                        i64 opt[DPS_PREFIXES], int lane, bool* all_best) {
  const bool gpu = T.type == TG_POOL_GPU;
  *all_best = false;
  // ---- the longest prefix: demand and duration sums at the least and at the best levels, rows
  int dmin[4] = {0, 0, 0, 0}, dbest[4] = {0, 0, 0, 0}, maxex[4] = {0, 0, 0, 0};
  i64 tmin_sum = 0, tbest_sum = 0;
  int nrows = 0;
  for (int i0 = 0; i0 < q0; i0 += 32) {
    const int i = i0 + lane;
    bool el = false;
    if (i < q0) {
      const int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7;
      const u32 mk = T.cmask[i];
      const int r0 = __ffs(mk), rb = best_level(T.cp[i], mk);
      const int lz0 = gpu ? level_of(g, gang, r0) : 0, lzb = gpu ? level_of(g, gang, rb) : 0;
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        if (l <= lz0) dmin[l] += g * r0;
        if (l <= lzb) dbest[l] += g * rb;
      }
      tmin_sum += duration(T.cs[i], T.cp[i], r0);
      tbest_sum += duration(T.cs[i], T.cp[i], rb);
      el = (mk & (mk - 1)) != 0;
    }
    const u32 b = __ballot_sync(TG_FULL, el);
    if (el) T.rowcand[nrows + __popc(b & ((1u << lane) - 1u))] = i;
    nrows += __popc(b);
  }
#pragma unroll
  for (int l = 0; l < 4; ++l) { dmin[l] = warp_sum32(dmin[l]); dbest[l] = warp_sum32(dbest[l]); }
  tbest_sum = warp_sum64(tbest_sum);
  __syncwarp();
  {
    bool fits_best = true;
#pragma unroll
    for (int l = 0; l < 4; ++l) if (l == 0 || gpu) fits_best &= dbest[l] <= T.cap[l];
    if (fits_best) {                                     // the common easy case: nothing else is needed
      for (int i = lane; i < q0; i += 32) out[0][i] = (u8)best_level(T.cp[i], T.cmask[i]);
      __syncwarp();
      opt[0] = tbest_sum; *all_best = true;
      return 1u;
    }
  }
  tmin_sum = warp_sum64(tmin_sum);
  for (int t = lane; t < nrows; t += 32) {               // largest extra demand of the rows
    const int i = T.rowcand[t];
    const u32 mk = T.cmask[i];
    int d[4];
    extra_demand(T.type, T.cg[i] & 0x7f, T.cg[i] >> 7, __ffs(mk), 32 - __clz(mk), d);
#pragma unroll
    for (int l = 0; l < 4; ++l) maxex[l] += d[l];
  }
#pragma unroll
  for (int l = 0; l < 4; ++l) maxex[l] = warp_sum32(maxex[l]);

  // ---- every prefix: certificates, box
  bool kept[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) kept[l] = l == 0 || (gpu && T.cap[l] < T.cap[l - 1]);
  int state[DPS_PREFIXES];                               // 0 needs the DP, 1 all at the best level, 2 all at the least
  int ext[4] = {1, 1, 1, 1};
  DpEnds E;
  E.nq = 0;
  int slot[DPS_PREFIXES];                                // prefix -> entry of E
  u32 done = 0;
#pragma unroll
  for (int k = 0; k < DPS_PREFIXES; ++k) {
    state[k] = -1; slot[k] = -1; opt[k] = 0;
    if (k >= nq) continue;
    if (k > 0) {                                         // take candidate q0 - k out of the sums
      const int i = q0 - k;
      const int g = T.cg[i] & 0x7f, gang = T.cg[i] >> 7;
      const u32 mk = T.cmask[i];
      const int r0 = __ffs(mk), rb = best_level(T.cp[i], mk);
      const int lz0 = gpu ? level_of(g, gang, r0) : 0, lzb = gpu ? level_of(g, gang, rb) : 0;
      int d[4] = {0, 0, 0, 0};
      const bool el = (mk & (mk - 1)) != 0;
      if (el) { extra_demand(T.type, g, gang, r0, 32 - __clz(mk), d); --nrows; }
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        if (l <= lz0) dmin[l] -= g * r0;
        if (l <= lzb) dbest[l] -= g * rb;
        maxex[l] -= d[l];
      }
      tmin_sum -= duration(T.cs[i], T.cp[i], r0);
      tbest_sum -= duration(T.cs[i], T.cp[i], rb);
    }
    bool fits_best = true;
#pragma unroll
    for (int l = 0; l < 4; ++l) if (l == 0 || gpu) fits_best &= dbest[l] <= T.cap[l];
    if (fits_best) { state[k] = 1; opt[k] = tbest_sum; done |= 1u << k; if (k == 0) *all_best = true; continue; }
    if (T.cap[0] - dmin[0] <= 0) { state[k] = 2; opt[k] = tmin_sum; done |= 1u << k; continue; }
    state[k] = 0;
    u32 lim = 0;
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      const int bound = min(T.cap[l] - dmin[l], maxex[l]);
      const int ek = kept[l] ? (max(bound, 0) >> l) + 1 : 1;
      ext[l] = max(ext[l], ek);
      lim |= (u32)min(ek - 1, 63) << (6 * l);
    }
    slot[k] = E.nq;
#pragma unroll
    for (int x = 0; x < DPS_PREFIXES; ++x) if (x == E.nq) { E.nrows_k[x] = nrows; E.lim[x] = lim; E.out[x] = out[k]; }
    ++E.nq;
  }
  // ---- multiplicities without the DP: best level where certified, least level elsewhere
  for (int i = lane; i < q0; i += 32) {
    const u32 mk = T.cmask[i];
    const u8 r0 = (u8)__ffs(mk), rb = (u8)best_level(T.cp[i], mk);
#pragma unroll
    for (int k = 0; k < DPS_PREFIXES; ++k)
      if (k < nq && i < q0 - k) out[k][i] = state[k] == 1 ? rb : r0;
  }
  __syncwarp();
  if (E.nq == 0) return done;

  // ---- one DP pass for the prefixes that need it
  int stride[4];
  u64 cells = 1;
#pragma unroll
  for (int l = 0; l < 4; ++l) { stride[l] = (int)cells; cells *= (u64)ext[l]; }
  const int nrows_all = E.nrows_k[0];                    // the longest of them comes first
  if (cells > 32 || !T.sim_base || nrows_all * 4 > T.sim_cap || nrows_all < 1) return done;
  const u32 solved = dp_small_multi(T, nrows_all, (int)cells, ext, stride, kept, T.sim_base, lane, E);
#pragma unroll
  for (int k = 0; k < DPS_PREFIXES; ++k) {
    if (k >= nq || slot[k] < 0 || !((solved >> slot[k]) & 1u)) continue;
    i64 sum = 0;
    for (int i = lane; i < q0 - k; i += 32) sum += duration(T.cs[i], T.cp[i], out[k][i]);
    opt[k] = warp_sum64(sum);
    done |= 1u << k;
  }
  return done;
}

// d-th smallest set bit (d = 0 is the lowest) as a multiplicity
__device__ __forceinline__ int nth_level(u32 mask, int d) {
  for (int k = 0; k < d; ++k) mask &= mask - 1;
  return __ffs(mask);
}

// Completion-heap estimate (Algorithm 2, estimate) of everything that is not in the prefix
// [0, q), whose multiplicities are alloc[0..q): evicted candidates first, then the pool's waiting
// actions.  Lane d simulates depth d+1.
__device__ bool estimate_rest(const Params& P, const PoolTask& T, int q, const u8* alloc, Slab slab, int lane, i64* est) {
  const int n_ev = T.m - q;
  const int n_rest = n_ev + T.n_ac;
  if (n_rest == 0) { *est = 0; return true; }
  i64 fs, fp; u32 fm;
  if (n_ev > 0) { fs = T.cs[q]; fp = T.cp[q]; fm = T.cmask[q]; }
  else { fs = T.ac_first.s; fp = T.ac_first.p; fm = T.ac_first.mask; }
  const int dmax = min(min(T.depth, __popc(fm)), 32);
  const int H = T.n_seeds + q;
  if (H <= 256) {
    // the whole warp on one simulation, one depth (the largest level tried is the best one):
    // 32-bit times on a sorted array first, packed 64-bit keys if a time leaves 32 bits
    bool overflow;
    const i64 fd = duration(fs, fp, nth_level_of(fm, dmax - 1));
    auto seed_of = [&](int i) { return i < T.n_seeds ? T.seeds[i]
                                                     : duration(T.cs[i - T.n_seeds], T.cp[i - T.n_seeds], alloc[i - T.n_seeds]); };
    auto dur_of = [&](int k) { return k == 0 ? fd
                                   : (k < n_ev ? duration(T.cs[q + k], T.cp[q + k], __ffs(T.cmask[q + k])) : T.ac_tmin[k - n_ev]); };
    i64 fast;
    if (H <= 32) fast = sorted_sim<1>(H, n_rest, seed_of, dur_of, lane, &overflow);
    else if (H <= 64) fast = sorted_sim<2>(H, n_rest, seed_of, dur_of, lane, &overflow);
    else if (H <= 96) fast = sorted_sim<3>(H, n_rest, seed_of, dur_of, lane, &overflow);
    else if (H <= 128) fast = sorted_sim<4>(H, n_rest, seed_of, dur_of, lane, &overflow);
    else if (H <= 192) fast = sorted_sim<6>(H, n_rest, seed_of, dur_of, lane, &overflow);
    else fast = sorted_sim<8>(H, n_rest, seed_of, dur_of, lane, &overflow);
    if (!overflow) { *est = fast; return true; }
    const i64 val = warp_sim<8>(
        H, n_rest,
        [&](int i) { return i < T.n_seeds ? T.seeds[i]
                                          : duration(T.cs[i - T.n_seeds], T.cp[i - T.n_seeds], alloc[i - T.n_seeds]); },
        [&](int k) { return k == 0 ? fd
                          : (k < n_ev ? duration(T.cs[q + k], T.cp[q + k], __ffs(T.cmask[q + k])) : T.ac_tmin[k - n_ev]); },
        lane, &overflow);
    if (!overflow) { *est = val; return true; }
  } else if (T.sim_base && H <= T.sim_cap) {
    // one lane, one depth (the largest level tried is the best one), tree in shared memory
    i64 val = 0; int bad = 0;
    if (lane == 0) {
      bool overflow;
      const i64 fd = duration(fs, fp, nth_level_of(fm, dmax - 1));
      val = tree_sim2<9, 3>(
          T.sim_base, H, n_rest,
          [&](int i) { return i < T.n_seeds ? T.seeds[i]
                                            : duration(T.cs[i - T.n_seeds], T.cp[i - T.n_seeds], alloc[i - T.n_seeds]); },
          [&](int k) { return k == 0 ? fd
                            : (k < n_ev ? duration(T.cs[q + k], T.cp[q + k], __ffs(T.cmask[q + k])) : T.ac_tmin[k - n_ev]); },
          &overflow);
      bad = overflow;
    }
    __syncwarp();
    bad = __shfl_sync(TG_FULL, bad, 0);
    if (!bad) { *est = __shfl_sync(TG_FULL, val, 0); return true; }
  }
  i64* heaps = (i64*)slab.take((u64)dmax * H * sizeof(i64));
  if (!heaps) heaps = (i64*)arena_take(P, (u64)dmax * H * sizeof(i64), lane);
  if (!heaps) return false;
  for (int d = 0; d < dmax; ++d)
    for (int i = lane; i < H; i += 32)
      heaps[(u64)d * H + i] = i < T.n_seeds ? T.seeds[i]
                                            : duration(T.cs[i - T.n_seeds], T.cp[i - T.n_seeds], alloc[i - T.n_seeds]);
  __syncwarp();
  i64 tmp = TG_INF;
  if (lane < dmax) {
    i64* h = heaps + (u64)lane * H;
    for (int st = H / 2 - 1; st >= 0; --st) {           // heapify
      i64 v = h[st]; int pos = st;
      for (;;) {
        int c = 2 * pos + 1;
        if (c >= H) break;
        if (c + 1 < H && h[c + 1] < h[c]) ++c;
        if (h[c] < v) { h[pos] = h[c]; pos = c; } else break;
      }
      h[pos] = v;
    }
    tmp = 0;
    for (int e = 0; e < n_rest; ++e) {
      i64 dur;
      if (e == 0) dur = duration(fs, fp, nth_level(fm, lane));
      else if (e < n_ev) dur = duration(T.cs[q + e], T.cp[q + e], __ffs(T.cmask[q + e]));
      else dur = T.ac_tmin[e - n_ev];
      i64 v = h[0] + dur;                                // pop the earliest completion, push ts + T
      tmp = sat_add(tmp, v);
      int pos = 0;
      for (;;) {
        int c = 2 * pos + 1;
        if (c >= H) break;
        i64 hc = h[c];
        if (c + 1 < H) { i64 h2 = h[c + 1]; if (h2 < hc) { hc = h2; ++c; } }
        if (hc < v) { h[pos] = hc; pos = c; } else break;
      }
      h[pos] = v;
    }
  }
  __syncwarp();
  *est = warp_min64(tmp);
  return true;
}

// An eviction step that cannot pay.  Let the first q+1 candidates be kept with multiplicities
// `kept`, and let `fewer` be the optimal multiplicities of the first q alone.  If the two agree on
// the first q candidates and candidate q's kept duration is no longer than at the largest level
// the estimate would try for it, then objective(q) >= objective(q+1):
//   * both objectives share the duration sum of the first q candidates;
//   * with q+1 kept, candidate q adds T_q(kept) and occupies one completion slot from T_q(kept) on;
//     with q kept, it is the first waiting action: it adds ts + T_q(level d) >= T_q(kept), where
//     ts >= 0 is the earliest completion, and that slot is busy until then;
//   * so the completion multiset after the step dominates the other one slot by slot (the slot
//     the smaller list lacks counts as never free), dominance survives every further
//     "pop the earliest, push earliest + T" step, every popped time is >=, and every later
//     waiting action runs at its least level in the first sum and at that or a larger level in
//     the second.
// Algorithm 1 stops at the first step whose objective does not decrease, so neither estimate is
// needed.  Warp-uniform result.
__device__ __forceinline__ bool eviction_cannot_pay(const PoolTask& T, int q, const u8* kept, const u8* fewer,
                                                    int lane) {
  bool same = true;
  for (int i = lane; i < q; i += 32) same &= kept[i] == fewer[i];
  if (!__all_sync(TG_FULL, same)) return false;
  const u32 mk = T.cmask[q];
  const int dmax = min(T.depth, __popc(mk));
  return duration(T.cs[q], T.cp[q], kept[q]) <= duration(T.cs[q], T.cp[q], nth_level_of(mk, dmax - 1));
}

// Once an eviction has been accepted the loop tends to go on, and every further step is a DP plus
// a simulation that depend on nothing but the prefix length.  So the next EVB steps are evaluated
// at once: their DPs one after the other, their simulations side by side, one lane each, on
// binary winner trees in the warp's shared memory; then the steps are accepted in order while
// the objective decreases (Algorithm 1, lines 10-14).  Starts from `keep` kept candidates
// (multiplicities T.rkeep, objective obj).  Returns the number finally kept, -1 if the workspace
// is too small, -2 if this path does not apply (the caller goes on step by step).
#define EVB 4
#define EVB_SLOTS 112       // slots of one of the EVB trees
__device__ __noinline__ int evict_batch(const Params& P, const PoolTask& T, Slab slab, int lane, i64 obj, int keep) {
  if (!T.sim_base || T.sim_cap < EVB * EVB_SLOTS || T.n_seeds + keep - 1 > EVB_SLOTS) return -2;
  u8* rs = (u8*)slab.take((u64)EVB * T.m);
  if (!rs) return -2;
  while (keep > 1) {
    const int keep0 = keep, nb = min(EVB, keep - 1);
    i64 optk[EVB];
    u32 stopmask = 0;
    int cnt = 0;
    u8* outs[DPS_PREFIXES];
#pragma unroll
    for (int k = 0; k < EVB; ++k) outs[k] = rs + (u64)k * T.m;
    bool ab;
    const u32 got = solve_multi(T, keep0 - 1, nb, outs, optk, lane, &ab);   // one DP pass for all steps where that applies
#pragma unroll 1
    for (int k = 0; k < EVB; ++k) {
      if (k < nb && !stopmask) {
        const int q = keep0 - 1 - k;
        if (!((got >> k) & 1u)) {
          PoolTask T2 = T;
          T2.rsel = outs[k];
          if (!solve_prefix(P, T2, q, slab, lane, &optk[k])) {
            if (k == 0) return -1;
            break;                                       // a step the loop may never reach: decided when it comes first
          }
        }
        if (eviction_cannot_pay(T, q, k == 0 ? T.rkeep : outs[k - 1], outs[k], lane)) stopmask |= 1u << k;
        cnt = k + 1;
      }
    }
    // the simulations of the steps that need one: lane k runs step k
    i64 est = 0;
    bool redo = false;
    if (lane < cnt && !((stopmask >> lane) & 1u)) {
      const int q = keep0 - 1 - lane, n_ev = T.m - q, n_rest = n_ev + T.n_ac;
      const u8* alloc = rs + (u64)lane * T.m;
      const u32 fm = T.cmask[q];
      const i64 fd = duration(T.cs[q], T.cp[q], nth_level_of(fm, min(min(T.depth, __popc(fm)), 32) - 1));
      est = tree_sim2<7, 3>(
          T.sim_base + (u32)lane * (EVB_SLOTS * 16), T.n_seeds + q, n_rest,
          [&](int i) { return i < T.n_seeds ? T.seeds[i]
                                            : duration(T.cs[i - T.n_seeds], T.cp[i - T.n_seeds], alloc[i - T.n_seeds]); },
          [&](int k) { return k == 0 ? fd
                            : (k < n_ev ? duration(T.cs[q + k], T.cp[q + k], __ffs(T.cmask[q + k])) : T.ac_tmin[k - n_ev]); },
          &redo);
    }
    __syncwarp();
    const u32 redomask = __ballot_sync(TG_FULL, redo);   // packed keys overflowed: exact estimate instead
#pragma unroll 1
    for (int k = 0; k < EVB; ++k) {
      if (k >= cnt) break;
      if ((stopmask >> k) & 1u) return keep;
      const int q = keep0 - 1 - k;
      i64 ek = __shfl_sync(TG_FULL, est, k);
      if ((redomask >> k) & 1u) {
        if (!estimate_rest(P, T, q, rs + (u64)k * T.m, slab, lane, &ek)) return -1;
      }
      const i64 nobj = sat_add(optk[k], ek);
      if (nobj >= obj) return keep;
      obj = nobj; keep = q;
      for (int i = lane; i < q; i += 32) T.rkeep[i] = rs[(u64)k * T.m + i];
      __syncwarp();
    }
  }
  return keep;
}

// Greedy eviction (Algorithm 1, lines 8-14), continued from a state in which the first `keep`
// candidates are kept with multiplicities T.rkeep and duration sum `opt_keep`; `obj` is their
// objective if `have_obj`, else it is computed when first needed.  Returns the number of
// candidates finally kept, or -1 if the workspace is too small.
__device__ int evict_resume(const Params& P, const PoolTask& T, Slab slab, int lane, i64 obj, int keep,
                            bool have_obj = true, i64 opt_keep = 0) {
  i64 opt, est;
  // (most chains end with the step after the first accepted eviction: that step is taken alone,
  // and only a chain that goes on looks several steps ahead)
  for (int t = T.m - keep + 1; t <= T.m - 1; ++t) {
    const int q = T.m - t;
    if (!solve_prefix(P, T, q, slab, lane, &opt)) return -1;
    if (eviction_cannot_pay(T, q, T.rkeep, T.rsel, lane)) break;
    if (!have_obj) {
      if (!estimate_rest(P, T, keep, T.rkeep, slab, lane, &est)) return -1;
      obj = sat_add(opt_keep, est); have_obj = true;
    }
    if (!estimate_rest(P, T, q, T.rsel, slab, lane, &est)) return -1;
    i64 nobj = sat_add(opt, est);
    if (nobj >= obj) break;
    obj = nobj; keep = q;
    for (int i = lane; i < q; i += 32) T.rkeep[i] = T.rsel[i];
    __syncwarp();
    const int kb = evict_batch(P, PoolTask(T), slab, lane, obj, keep);   // an eviction was accepted: look further ahead
    if (kb != -2) return kb;
  }
  return keep;
}

// A single candidate: nothing can be evicted (the head stays), and DPArrange for one task is the feasible
// level of least duration, the smallest one among equals (value, then units).  Lane r-1 tries multiplicity r.
__device__ __forceinline__ void solve_single(const PoolTask& T, int lane) {
  const int g = T.cg[0] & 0x7f, gang = T.cg[0] >> 7, r = lane + 1;
  const u32 mk = T.cmask[0];
  bool ok = (mk >> lane) & 1u;
  if (ok) {
    const int lz = T.type == TG_POOL_GPU ? level_of(g, gang, r) : 0;
    int cap = T.cap[0];
#pragma unroll
    for (int l = 1; l < 4; ++l) if (l == lz) cap = T.cap[l];
    ok = g * r <= cap;
  }
  const i64 key = ok ? ((duration(T.cs[0], T.cp[0], r) << 6) | (i64)r) : TG_INF;
  const i64 best = warp_min64(key);
  // (the least level fits: the prefix admitted the action)
  if (lane == 0) { const u8 rr = best == TG_INF ? (u8)__ffs(mk) : (u8)(best & 63); T.rsel[0] = rr; T.rkeep[0] = rr; }
  __syncwarp();
}

// The whole loop, starting from the full candidate list.
__device__ int evict_loop(const Params& P, const PoolTask& T, Slab slab, int lane) {
  if (T.m == 1) { solve_single(T, lane); return 1; }
  i64 opt;
  if (!solve_prefix(P, T, T.m, slab, lane, &opt)) return -1;
  for (int i = lane; i < T.m; i += 32) T.rkeep[i] = T.rsel[i];
  __syncwarp();
  return evict_resume(P, T, slab, lane, 0, T.m, false, opt);
}
