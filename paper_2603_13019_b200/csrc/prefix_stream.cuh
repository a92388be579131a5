// First two kernels of a batched round.
//
// k_head, one warp per scenario, walks the queue 32 actions at a time until the candidate
// prefix ends (Algorithm 1, line 2): lane v keeps the running least-level demand of demand
// slot v (one slot per core / quota pool, four nested chunk levels per GPU pool), lane j the
// number of actions of pool j seen so far; a chunk's demand goes through one warp scan per
// slot and the first action that overflows a slot ends the prefix.  Candidates get their
// position inside their pool (Algorithm 1, line 4) and their index is written to the pool's
// part of `order`.  The same walk sums every slot's demand at the candidates' LARGEST levels:
// where that fits, every candidate gets its best level, no eviction can pay and nobody will
// read the pool's waiting list.
//
// k_stream, one CTA per scenario, streams everything behind the head 4096 actions at a time
// (16 per thread, 128-bit loads): records are validated, and only for the pools that may need
// an estimate the least-level durations (Eq. 1) of the waiting actions are appended, in queue
// order, to the pool's list in `tmin`.
//
// k_fill writes "not scheduled" to every output row behind the candidate prefix (128-bit
// stores).  Nothing else touches those rows, so it runs on a stream of its own beside all
// kernels that follow k_head.
//
// Partitioned arrays (order, tmin and the solver's arrays) give every (scenario, pool) its own
// row of max_actions entries, so a position never depends on another pool's count and the
// queue is read once.
#pragma once
#include "common.cuh"

#define KS_THREADS 256
#define KS_ITEMS 16
#define KS_TILE (KS_THREADS * KS_ITEMS)

// what k_head leaves for k_stream
struct HeadState {
  int hs;                     // first action the stream has to look at (a multiple of 32, or n_actions)
  u32 need;                   // pools whose waiting list may be read
  int bad;                    // an invalid record was seen
  int n;                      // length of the candidate prefix
  int cur[TG_MAX_POOLS];      // actions of every pool in [0, hs)
};

__device__ __forceinline__ int warp_incl_scan32(int x, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(TG_FULL, x, o); if (lane >= o) x += y; }
  return x;
}

// Further entries of the cost vectors (Section 4.1): an entry has to name a quota / concurrency pool other
// than the action's key pool and an amount of 1 .. its capacity.  One thread per action; a scenario with
// a bad entry is flagged for k_head, which then decides nothing of it.
__global__ void __launch_bounds__(256) k_side_check(const __grid_constant__ Params P) {
  // sixteen consecutive actions of one scenario per thread (128-bit loads) where the rows allow it
  const bool vec = (P.N % 16 == 0) && (P.side_plane % 16 == 0) &&
                   ((((size_t)P.a_pool | (size_t)P.a_side_pool) & 15) == 0) && (((size_t)P.a_side_units & 15) == 0);
  const size_t total = (size_t)P.S * P.N, step = (size_t)gridDim.x * blockDim.x;
  if (vec) {
    for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < total / 16; q += step) {
      const size_t o = q * 16;
      const int sc = (int)(o / P.N), i0 = (int)(o - (size_t)sc * P.N);
      const int n = min(max(P.n_actions[sc], 0), P.N) - i0;    // records of this group that exist
      if (n <= 0) continue;
      bool bad = false;
      for (int e = 0; e < P.n_side; ++e) {
        __align__(16) u8 k[16];
        *(uint4*)k = *(const uint4*)(P.a_side_pool + e * P.side_plane + o);
        const uint4 kk = *(const uint4*)k;
        if ((kk.x & kk.y & kk.z & kk.w) == 0xffffffffu) continue;   // no entry in the whole group
        __align__(16) unsigned short c[16];
        __align__(16) u8 kp[16];
        *(uint4*)c = *(const uint4*)(P.a_side_units + e * P.side_plane + o);
        *(uint4*)(c + 8) = *(const uint4*)(P.a_side_units + e * P.side_plane + o + 8);
        *(uint4*)kp = *(const uint4*)(P.a_pool + o);
#pragma unroll
        for (int x = 0; x < 16; ++x) {
          if (x >= n || k[x] == 0xff) continue;
          const int kx = k[x] < P.P ? k[x] : 0;
          bad |= k[x] >= P.P || P.pool[kx].type != TG_POOL_API || k[x] == kp[x] || c[x] < 1 || c[x] > P.pool[kx].capacity;
        }
      }
      if (bad) P.side_bad[sc] = 1;
    }
    return;
  }
  for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += step) {
    const int sc = (int)(o / P.N), i = (int)(o - (size_t)sc * P.N);
    if (i >= min(max(P.n_actions[sc], 0), P.N)) continue;
    bool bad = false;
    for (int e = 0; e < P.n_side; ++e) {
      const int k = P.a_side_pool[e * P.side_plane + o];
      if (k == 0xff) continue;
      const int c = P.a_side_units[e * P.side_plane + o];
      bad |= k >= P.P || P.pool[k < P.P ? k : 0].type != TG_POOL_API || k == P.a_pool[o] || c < 1 ||
             c > P.pool[k < P.P ? k : 0].capacity;
    }
    if (bad) P.side_bad[sc] = 1;
  }
}

// SIDE: the actions carry further cost-vector entries (Section 4.1); the plain instance keeps its registers.
template <bool SIDE>
__global__ void __launch_bounds__(256) k_head(const __grid_constant__ Params P, HeadState* hst) {
  const int lane = threadIdx.x & 31;
  const int sc = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
  if (sc >= P.S) return;
  const size_t row = (size_t)sc * P.N;
  const size_t prow = (size_t)sc * P.P * P.N;       // pool j's part starts at prow + j * N
  const int n_act = min(max(P.n_actions[sc], 0), P.N);
  const int D = P.V - P.P;                          // demand slots

  // lane v < D: capacity, running least-level demand and candidates' largest-level demand of slot v
  // lane j < P: actions / candidates / first waiting action of pool j, and the pool's description
  int capreg = 0, run = 0, mxd = 0, cnt = 0, mreg = 0, fwreg = -1;
  int sres = 0;                                     // lane v: what the candidates ask of slot v beside their key resource
  u32 pinfo = 0;                                    // type | GPUs per node << 4 | slot0 << 8
  for (int j = 0; j < P.P; ++j) {
    const PoolDev& pd = P.pool[j];
    if (pd.type == TG_POOL_GPU) {
      int cap[4];
      gpu_caps(pd, P.gpu_busy ? P.gpu_busy + (size_t)sc * P.n_nodes_total : nullptr, lane, cap);
#pragma unroll
      for (int l = 0; l < 4; ++l) if (lane == pd.slot0 + l) capreg = cap[l];
    } else if (lane == pd.slot0) capreg = pd.capacity;
    if (lane == j) pinfo = (u32)pd.type | ((u32)(pd.type == TG_POOL_GPU ? pd.group : 0) << 4) | ((u32)pd.slot0 << 8);
  }

  u32 el = 0, need = 0;
  bool bad = false;
  int hs = n_act, n_pref = n_act;
  const u32 lt = (1u << lane) - 1u;
  // the records of the next chunk are loaded while this one is worked on
  int nj = 0; u32 nun = 0, nmk = 0; i64 ns = 0, np_ = 0;
  int nk0 = 0xff, nu0 = 0, nk1 = 0xff, nu1 = 0;    // further entries of the cost vectors
  if (SIDE && lane < n_act) {
    nk0 = P.a_side_pool[row + lane]; nu0 = P.a_side_units[row + lane];
    if (P.n_side > 1) { nk1 = P.a_side_pool[P.side_plane + row + lane]; nu1 = P.a_side_units[P.side_plane + row + lane]; }
  }
  if (lane < n_act) { nj = P.a_pool[row + lane]; nun = P.a_unit[row + lane]; nmk = P.a_mask[row + lane]; ns = P.a_s[row + lane]; np_ = P.a_p[row + lane]; }
  for (int c0 = 0; c0 < n_act; c0 += 32) {
    const int i = c0 + lane;
    const bool present = i < n_act;
    const int j = nj; const u32 un = nun, mk = nmk; const i64 s = ns, p = np_;
    const int k0 = nk0, k1 = nk1;
    int su0 = nu0, su1 = nu1;
    if (SIDE) {
      const int i2 = i + 32;
      nk0 = 0xff; nk1 = 0xff; nu0 = 0; nu1 = 0;
      if (i2 < n_act) {
        nk0 = P.a_side_pool[row + i2]; nu0 = P.a_side_units[row + i2];
        if (P.n_side > 1) { nk1 = P.a_side_pool[P.side_plane + row + i2]; nu1 = P.a_side_units[P.side_plane + row + i2]; }
      }
    }
    {
      const int i2 = i + 32;
      nj = 0; nun = 0; nmk = 0; ns = 0; np_ = 0;
      if (i2 < n_act) { nj = P.a_pool[row + i2]; nun = P.a_unit[row + i2]; nmk = P.a_mask[row + i2]; ns = P.a_s[row + i2]; np_ = P.a_p[row + i2]; }
    }
    bool valid = present && j < P.P;
    const u32 pi = __shfl_sync(TG_FULL, pinfo, valid ? j : 0);
    PoolDev pd;
    pd.type = pi & 15; pd.group = (pi >> 4) & 15;
    const int slot0 = pi >> 8;
    int g = 1, gang = 0; u32 eff = 1;
    if (valid) valid = decode_levels(pd, (u8)un, mk, g, gang, eff);
    bad |= present && !valid;
    const bool gpu = pd.type == TG_POOL_GPU;
    const int rmin = __ffs(eff), rmax = 32 - __clz(eff);
    const int units = g * rmin, mxu = g * rmax;
    const int lz = gpu ? level_of(g, gang, rmin) : 0, lzx = gpu ? level_of(g, gang, rmax) : 0;
    // further entries of the cost vector: the slot they charge and the amount (slot -1: none)
    int ss0 = -1, ss1 = -1;
    if (SIDE) {
      const u32 p0 = __shfl_sync(TG_FULL, pinfo, k0 < P.P ? k0 : 0), p1 = __shfl_sync(TG_FULL, pinfo, k1 < P.P ? k1 : 0);
      if (valid && k0 < P.P) ss0 = p0 >> 8;
      if (valid && k1 < P.P) ss1 = p1 >> 8;
    }
    // least-level demand: one scan per slot; the first action that overflows a slot ends the prefix
    // First the chunk's total per slot (one warp reduction each): only the chunk in which a slot
    // overflows needs the scans that tell which action does it.
    int tot_mine = 0;                                  // lane v: the chunk's demand on slot v
    for (int v = 0; v < D; ++v) {
      const int c = ((valid && v >= slot0 && v <= slot0 + lz) ? units : 0) + (ss0 == v ? su0 : 0) + (ss1 == v ? su1 : 0);
      const int tot = __reduce_add_sync(TG_FULL, c);
      if (lane == v) tot_mine = tot;
    }
    bool over = false;
    if (__any_sync(TG_FULL, lane < D && run + tot_mine > capreg)) {
      for (int v = 0; v < D; ++v) {
        const int c = ((valid && v >= slot0 && v <= slot0 + lz) ? units : 0) + (ss0 == v ? su0 : 0) + (ss1 == v ? su1 : 0);
        const int incl = warp_incl_scan32(c, lane);
        const int rv = __shfl_sync(TG_FULL, run, v), cv = __shfl_sync(TG_FULL, capreg, v);
        over |= c > 0 && rv + incl > cv;
      }
    }
    run += tot_mine;                                   // beyond the prefix the totals are not used any more
    const u32 ob = __ballot_sync(TG_FULL, over);
    const int f = ob ? __ffs(ob) - 1 : 32;           // lanes >= f wait
    const bool cand = valid && lane < f;
    // position inside the pool
    int pos = __shfl_sync(TG_FULL, cnt, valid ? j : 0);  // the pool's count before this chunk
    const u32 below_f = f >= 32 ? TG_FULL : ((1u << f) - 1u);
    for (int jj = 0; jj < P.P; ++jj) {
      const u32 b = __ballot_sync(TG_FULL, valid && j == jj);
      if (valid && j == jj) pos += __popc(b & lt);
      if (lane == jj) { cnt += __popc(b); mreg += __popc(b & below_f); }
    }
    if (cand) {
      P.order[(size_t)sc * P.cand_stride + P.cand_off[j] + pos] = i;
      if (eff & (eff - 1)) el |= 1u << j;
    }
    for (int v = 0; v < D; ++v) {
      const int sd = cand ? (ss0 == v ? su0 : 0) + (ss1 == v ? su1 : 0) : 0;
      const int c = ((cand && v >= slot0 && v <= slot0 + lzx) ? mxu : 0) + sd;
      const int tot = __reduce_add_sync(TG_FULL, c);
      if (lane == v) mxd += tot;
      if (SIDE) { const int st = __reduce_add_sync(TG_FULL, sd); if (lane == v) sres += st; }
    }
    if (ob) {
      // The prefix is complete.  A pool may need its waiting list only if one of its candidates
      // is elastic and the candidates' largest levels do not all fit.
      const u32 unfit = __ballot_sync(TG_FULL, lane < D && mxd > capreg);
      const u32 elw = __reduce_or_sync(TG_FULL, el);
      for (int jj = 0; jj < P.P; ++jj) {
        const u32 slots = ((1u << P.pool[jj].n_slots) - 1u) << P.pool[jj].slot0;
        if (((elw >> jj) & 1u) && (unfit & slots)) need |= 1u << jj;
      }
      const int mj = __shfl_sync(TG_FULL, mreg, valid ? j : 0);
      const bool waits = valid && lane >= f;
      if (waits && ((need >> j) & 1u))
        P.tmin[prow + (size_t)j * P.N + pos] = duration(clamp_param(s), clamp_param(p), rmin);
      for (int jj = 0; jj < P.P; ++jj) {               // the pool's first waiting action
        const u32 b = __ballot_sync(TG_FULL, waits && j == jj && pos == mj);
        if (lane == jj && b) fwreg = c0 + __ffs(b) - 1;
      }
      hs = min(c0 + 32, n_act); n_pref = c0 + f;
      break;
    }
  }
  const u32 elw = __reduce_or_sync(TG_FULL, el);
  if (hs == n_act && n_pref == n_act) {
    // the whole queue is the candidate prefix: the same test tells which pools are certified
    const u32 unfit = __ballot_sync(TG_FULL, lane < D && mxd > capreg);
    for (int jj = 0; jj < P.P; ++jj) {
      const u32 slots = ((1u << P.pool[jj].n_slots) - 1u) << P.pool[jj].slot0;
      if (((elw >> jj) & 1u) && (unfit & slots)) need |= 1u << jj;
    }
  }
  const int anybad = (__any_sync(TG_FULL, bad) || (SIDE && P.side_bad[sc])) ? 1 : 0;
  if (SIDE) {
    const int sr = __shfl_sync(TG_FULL, sres, lane < P.P ? P.pool[lane].slot0 : 0);
    if (lane < P.P) P.side_res[(size_t)sc * P.P + lane] = sr;
  }
  if (lane < P.P) {
    PoolMeta mt;
    mt.base = (i64)sc * (P.P - 1) * P.N + (i64)lane * P.N;   // row + base = prow + lane * N
    mt.cbase = (i64)sc * (P.cand_stride - P.N) + P.cand_off[lane];   // row + cbase = sc * cand_stride + cand_off
    // an invalid record among the actions seen here: nothing of the scenario is decided
    mt.count = anybad ? 0 : cnt; mt.m = anybad ? 0 : mreg; mt.elastic = anybad ? 0 : ((elw >> lane) & 1u);
    mt.first_wait = anybad ? -1 : fwreg;
    P.meta[(size_t)sc * P.P + lane] = mt;
    hst[sc].cur[lane] = cnt;
  }
  if (lane == 0) {
    hst[sc].hs = hs; hst[sc].need = need; hst[sc].bad = anybad; hst[sc].n = n_pref;
    P.o_status[sc] = anybad ? TG_ST_BAD_ACTION : 0; P.o_total[sc] = 0; P.o_nsel[sc] = 0;
  }
}

// exclusive scan of one int per thread over the CTA; *total = sum.  wsum: 8 ints of scratch.
__device__ __forceinline__ int ks_block_scan(int x, int* wsum, int t, int* total) {
  const int lane = t & 31, warp = t >> 5;
  const int incl = warp_incl_scan32(x, lane);
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  int off = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < KS_THREADS / 32; ++w) { const int v = wsum[w]; if (w < warp) off += v; tot += v; }
  __syncthreads();
  *total = tot;
  return off + incl - x;
}

__global__ void __launch_bounds__(KS_THREADS, 5) k_stream(const __grid_constant__ Params P, const HeadState* hst) {
  __shared__ int s_m[TG_MAX_POOLS], s_first[TG_MAX_POOLS], s_cur[TG_MAX_POOLS], s_scan[KS_THREADS / 32];
  __shared__ int s_bad;
  // usable multiplicities by (pool, unit byte): a record's usable levels are its mask ANDed with the
  // entry, and a record with none is invalid (decode_levels, tabulated once per round description)
  __shared__ __align__(16) u32 s_ok[TG_MAX_POOLS * 256];

  const int sc = blockIdx.x, t = threadIdx.x;
  const size_t row = (size_t)sc * P.N;
  const size_t prow = (size_t)sc * P.P * P.N;
  const int n_act = min(max(P.n_actions[sc], 0), P.N);
  const HeadState H = hst[sc];
  const u32 need = H.need;
  const bool vec = (P.N % 16 == 0) && ((((size_t)P.a_pool | (size_t)P.a_unit | (size_t)P.a_mask) & 15) == 0);
  if (t < TG_MAX_POOLS) {
    s_m[t] = t < P.P ? P.meta[(size_t)sc * P.P + t].m : 0;
    s_first[t] = INT_MAX;
  }
  for (int x = t; x < TG_MAX_POOLS * 256 / 4; x += KS_THREADS) ((uint4*)s_ok)[x] = ((const uint4*)P.ok_table)[x];
  if (t == 0) s_bad = H.bad;
  __syncthreads();

  if (t < TG_MAX_POOLS) s_cur[t] = H.cur[t];          // actions of every pool seen so far
  __syncthreads();
  for (int tile0 = H.hs; tile0 < n_act; tile0 += KS_TILE) {   // a bad scenario is streamed on: its rows are rewritten below
    const int i_first = tile0 + t * KS_ITEMS;
    const bool full = vec && i_first + KS_ITEMS <= n_act;
    __align__(16) u8 rp[KS_ITEMS], ru[KS_ITEMS];
    // validate; keep the least multiplicity of the records whose pool may need its list
    bool bad = false;
    u32 rmin4[KS_ITEMS / 4];                          // one byte per record, 0 = not listed
    {
      __align__(16) u32 rm[KS_ITEMS];
      if (full) {
        *(uint4*)rp = *(const uint4*)(P.a_pool + row + i_first);
        *(uint4*)ru = *(const uint4*)(P.a_unit + row + i_first);
#pragma unroll
        for (int k = 0; k < KS_ITEMS; k += 4) *(uint4*)(rm + k) = *(const uint4*)(P.a_mask + row + i_first + k);
      } else {
#pragma unroll
        for (int k = 0; k < KS_ITEMS; ++k) {
          const int i = i_first + k;
          rp[k] = i < n_act ? P.a_pool[row + i] : 0xff;
          ru[k] = i < n_act ? P.a_unit[row + i] : 1;
          rm[k] = i < n_act ? P.a_mask[row + i] : 1;
        }
      }
#pragma unroll
      for (int k = 0; k < KS_ITEMS / 4; ++k) rmin4[k] = 0;
#pragma unroll
      for (int k = 0; k < KS_ITEMS; ++k) {
        if (!full && i_first + k >= n_act) continue;
        const int j = rp[k];
        const u32 eff = j < TG_MAX_POOLS ? rm[k] & s_ok[j * 256 + ru[k]] : 0u;   // pools beyond the description hold zeros
        bad |= eff == 0;
        if ((need >> j) & 1u) rmin4[k >> 2] |= (u32)__ffs(eff) << (8 * (k & 3));
      }
    }
    if (bad) s_bad = 1;
    // waiting lists of the pools that may need them; a position follows from the pool bytes alone
    for (u32 nm = need; nm; nm &= nm - 1) {
      const int j = __ffs(nm) - 1;
      u32 mine = 0;
#pragma unroll
      for (int k = 0; k < KS_ITEMS; ++k) if (rp[k] == j) mine |= 1u << k;
      const int before = s_cur[j];
      int tot;
      int pos = before + ks_block_scan(__popc(mine), s_scan, t, &tot);
      if (t == 0) s_cur[j] = before + tot;               // read again only after the barrier that ends the tile
      if (!mine) continue;
      const int m_j = s_m[j];
      i64* dst = P.tmin + prow + (size_t)j * P.N;
      // the thread's listed records, four at a time: their s / p loads are in flight together
      const u64 rlo = (u64)rmin4[0] | ((u64)rmin4[1] << 32), rhi = (u64)rmin4[2] | ((u64)rmin4[3] << 32);
      for (u32 rest = mine; rest;) {
        i64 sv[4], pv[4]; int kk[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          kk[x] = rest ? __ffs(rest) - 1 : -1;
          rest &= rest - 1;
          sv[x] = kk[x] >= 0 ? P.a_s[row + i_first + kk[x]] : 0;
          pv[x] = kk[x] >= 0 ? P.a_p[row + i_first + kk[x]] : 0;
        }
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          if (kk[x] < 0) continue;
          const int rmin = (int)(((kk[x] < 8 ? rlo : rhi) >> (8 * (kk[x] & 7))) & 0xffu);
          if (rmin) dst[pos] = duration(clamp_param(sv[x]), clamp_param(pv[x]), rmin);   // 0: invalid record, the scenario is flagged
          if (pos == m_j) s_first[j] = i_first + kk[x];   // the pool's first waiting action
          ++pos;
        }
      }
    }
    __syncthreads();
  }
  __syncthreads();
  const bool bad = s_bad != 0;
  // nobody will write the candidates of a bad scenario: their rows are "not scheduled" too
  if (bad) for (int i = t; i < min(H.n, P.N); i += KS_THREADS) {
    P.o_alloc[row + i] = 0; P.o_node[row + i] = -1; P.o_off[row + i] = -1; P.o_act[row + i] = -1;
  }
  if (t < P.P) {
    PoolMeta* mt = P.meta + (size_t)sc * P.P + t;
    if (bad) { mt->count = 0; mt->m = 0; mt->first_wait = -1; }
    else if ((need >> t) & 1u) {
      mt->count = s_cur[t];
      if (s_first[t] != INT_MAX) mt->first_wait = s_first[t];
    } else mt->count = mt->m;                          // a list nobody reads counts as empty
  }
  // status, total and count were initialised by k_head; k_solve may be adding to them already
  if (t == 0 && bad) atomicOr(&P.o_status[sc], TG_ST_BAD_ACTION);
}

// "not scheduled" (Eq. 2 has no value for an action that stays queued): units 0, node -1, offset -1,
// ACT -1 for every action behind its scenario's candidate prefix (the candidates' rows are written
// by the kernels that decide them, which may run at the same time).  Consecutive threads take
// consecutive groups of four actions, so a warp's store covers whole contiguous sectors.
__global__ void __launch_bounds__(256) k_fill(const __grid_constant__ Params P, const HeadState* hst) {
  const bool vec = (P.N % 4 == 0) &&
                   ((((size_t)P.o_alloc | (size_t)P.o_node | (size_t)P.o_off | (size_t)P.o_act) & 15) == 0);
  const u32 stride = gridDim.x * blockDim.x, tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (vec) {
    const u32 qpr = (u32)P.N / 4, quads = (u32)P.S * qpr;   // S * N <= 2^31
    const int4 z = make_int4(0, 0, 0, 0), m1 = make_int4(-1, -1, -1, -1);
    const longlong2 a1 = make_longlong2(-1, -1);
    for (u32 q = tid; q < quads; q += stride) {
      const u32 sc = q / qpr;
      const int i0 = (int)(q - sc * qpr) * 4, n = hst[sc].n;
      if (i0 + 4 <= n) continue;
      const size_t o = (size_t)q * 4;
      if (i0 >= n) {
        *(int4*)(P.o_alloc + o) = z; *(int4*)(P.o_node + o) = m1; *(int4*)(P.o_off + o) = m1;
        *(longlong2*)(P.o_act + o) = a1; *(longlong2*)(P.o_act + o + 2) = a1;
      } else {
        for (int k = n - i0; k < 4; ++k) { P.o_alloc[o + k] = 0; P.o_node[o + k] = -1; P.o_off[o + k] = -1; P.o_act[o + k] = -1; }
      }
    }
  } else {
    const size_t total = (size_t)P.S * P.N;
    for (size_t o = tid; o < total; o += stride) {
      if ((int)(o % P.N) < hst[o / P.N].n) continue;
      P.o_alloc[o] = 0; P.o_node[o] = -1; P.o_off[o] = -1; P.o_act[o] = -1;
    }
  }
}
