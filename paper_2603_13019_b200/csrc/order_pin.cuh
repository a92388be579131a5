// Front ends of a round that change what the scheduler sees as its queue.
//
// k_order (Section 4.2: Algorithm 1 takes the queue in any order): one CTA per scenario sorts the
// queue by a policy key -- least-level duration (Eq. 1) ascending or descending, or arrival time --
// with the queue position as second key, so equal keys keep their order.  Keys and positions live
// in shared memory (8 or 12 B per action, padded to a power of two); the sort is a bitonic network.
// k_gather / k_scatter move the records into sorted order and the results back to the actions' own
// positions, so the kernels of the round run unchanged on the sorted queue.
//
// k_pin (Section 5.2: per-node CPU scheduling): one warp per scenario walks the queue; the first
// action of a trajectory pins it to the CPU node (= CPU pool) with the most free memory among those
// with enough cores for the action's least level and enough free memory for the whole trajectory;
// every action of a pinned trajectory gets its node as pool.
#pragma once
#include "common.cuh"

#define KO_THREADS 512
#define KO_MAX_N 16384

struct OrderIo {
  int policy;            // 1: shortest least-level duration first, 2: longest first, 3: earliest arrival first
  int n_pad;             // max_actions rounded up to a power of two
  int* perm;             // [S][N] action index at each sorted position
};

// maximum over the warp of values >= -1
__device__ __forceinline__ i64 warp_max64_from_m1(i64 v) {
  const u64 u = (u64)(v + 1);
  const u32 hi = (u32)(u >> 32);
  const u32 mhi = __reduce_max_sync(TG_FULL, hi);
  const u32 mlo = __reduce_max_sync(TG_FULL, hi == mhi ? (u32)u : 0u);
  return (i64)(((u64)mhi << 32) | mlo) - 1;
}

__device__ __forceinline__ bool ko_less(u64 ka, u32 ia, u64 kb, u32 ib) { return ka < kb || (ka == kb && ia < ib); }

// WIDE = false: duration keys stay below 2^42 and positions below 2^14, so key and position are one 64-bit
// word (8 B per action); WIDE = true (arrival times, any 64-bit value): key and position side by side (12 B).
template <bool WIDE>
__global__ void __launch_bounds__(KO_THREADS) k_order(const __grid_constant__ Params P, const OrderIo O) {
  extern __shared__ __align__(16) unsigned char ko_smem[];
  u64* key = (u64*)ko_smem;
  u32* idx = (u32*)(key + O.n_pad);                    // WIDE only
  const int sc = blockIdx.x, t = threadIdx.x;
  const size_t row = (size_t)sc * P.N;
  const int n = min(max(P.n_actions[sc], 0), P.N);
  for (int i = t; i < O.n_pad; i += KO_THREADS) {
    u64 k = ~0ull;                                     // padding and the positions behind the queue stay where they are
    if (i < n) {
      if (WIDE) k = (u64)(P.a_arrival ? P.a_arrival[row + i] : 0) ^ 0x8000000000000000ull;
      else {
        const int j = P.a_pool[row + i];
        int g, gang; u32 eff;
        i64 T = 0;                                     // a record no pool can serve has key 0
        if (j < P.P && decode_levels(P.pool[j], P.a_unit[row + i], P.a_mask[row + i], g, gang, eff))
          T = duration(clamp_param(P.a_s[row + i]), clamp_param(P.a_p[row + i]), __ffs(eff));
        k = O.policy == 2 ? (u64)((1ll << 42) - T) : (u64)T;
      }
    }
    if (WIDE) { key[i] = k; idx[i] = (u32)i; }
    else key[i] = i < n ? (k << 14) | (u64)i : (~0ull << 14) | (u64)i;
  }
  __syncthreads();
  for (int size = 2; size <= O.n_pad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int x = t; x < O.n_pad / 2; x += KO_THREADS) {
        // pair (lo, lo + stride); ascending where bit `size` of lo is clear
        const int lo = ((x & ~(stride - 1)) << 1) | (x & (stride - 1)), hi = lo + stride;
        const u64 ka = key[lo], kb = key[hi];
        const bool up = (lo & size) == 0;
        if (WIDE) {
          const u32 ia = idx[lo], ib = idx[hi];
          if (ko_less(kb, ib, ka, ia) == up) { key[lo] = kb; key[hi] = ka; idx[lo] = ib; idx[hi] = ia; }
        } else if ((kb < ka) == up) { key[lo] = kb; key[hi] = ka; }
      }
      __syncthreads();
    }
  }
  for (int i = t; i < P.N; i += KO_THREADS) O.perm[row + i] = WIDE ? (int)idx[i] : (int)(key[i] & 0x3fffu);
}

// The same sort for the duration keys when the padded queue gives every thread EPT >= 1 whole elements
// (thread t holds positions t * EPT .. t * EPT + EPT - 1 in registers): compare-exchanges at strides below EPT
// stay inside a thread, strides below 32 * EPT go through warp shuffles, and only the strides beyond that
// through shared memory (one conflict-free store / load of every element per such stage).
template <int EPT>
__global__ void __launch_bounds__(KO_THREADS) k_order_regs(const __grid_constant__ Params P, const OrderIo O) {
  extern __shared__ __align__(16) unsigned char ko_smem[];
  u64* sm = (u64*)ko_smem;                             // [EPT][KO_THREADS]
  const int sc = blockIdx.x, t = threadIdx.x, lane = t & 31;
  const size_t row = (size_t)sc * P.N;
  const int n = min(max(P.n_actions[sc], 0), P.N);
  u64 v[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = t * EPT + e;
    u64 k = ~0ull << 14;                               // padding and the positions behind the queue stay where they are
    if (i < n) {
      const int j = P.a_pool[row + i];
      int g, gang; u32 eff;
      i64 T = 0;                                       // a record no pool can serve has key 0
      if (j < P.P && decode_levels(P.pool[j], P.a_unit[row + i], P.a_mask[row + i], g, gang, eff))
        T = duration(clamp_param(P.a_s[row + i]), clamp_param(P.a_p[row + i]), __ffs(eff));
      k = (O.policy == 2 ? (u64)((1ll << 42) - T) : (u64)T) << 14;
    }
    v[e] = k | (u64)i;
  }
  for (int size = 2; size <= O.n_pad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      if (stride < EPT) {
        // cs is a compile-time copy of the stride, so that v[] stays in registers
#pragma unroll
        for (int cs = 1; cs < EPT; cs <<= 1) {
          if (cs != stride) continue;
#pragma unroll
          for (int e = 0; e < EPT; ++e) {
            if (e & cs) continue;
            const bool up = ((t * EPT + e) & size) == 0;
            const u64 a = v[e], b = v[e | cs];
            if ((b < a) == up) { v[e] = b; v[e | cs] = a; }
          }
        }
      } else if (stride < 32 * EPT) {
        const int m = stride / EPT;                    // partner lane = lane ^ m
        const bool lower = (lane & m) == 0;
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
          const u64 o = __shfl_xor_sync(TG_FULL, v[e], m);
          const bool up = ((t * EPT + e) & size) == 0;
          const u64 lo_v = o < v[e] ? o : v[e], hi_v = o < v[e] ? v[e] : o;
          v[e] = (lower == up) ? lo_v : hi_v;
        }
      } else {
        const int m = stride / EPT;                    // partner thread = t ^ m
        const bool lower = (t & m) == 0;
        __syncthreads();
#pragma unroll
        for (int e = 0; e < EPT; ++e) sm[e * KO_THREADS + t] = v[e];
        __syncthreads();
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
          const u64 o = sm[e * KO_THREADS + (t ^ m)];
          const bool up = ((t * EPT + e) & size) == 0;
          const u64 lo_v = o < v[e] ? o : v[e], hi_v = o < v[e] ? v[e] : o;
          v[e] = (lower == up) ? lo_v : hi_v;
        }
      }
    }
  }
  // through shared memory once more, so that a warp writes consecutive positions
  __syncthreads();
#pragma unroll
  for (int e = 0; e < EPT; ++e) ((u32*)sm)[t * EPT + e] = (u32)(v[e] & 0x3fffu);
  __syncthreads();
  for (int i = t; i < P.N; i += KO_THREADS) O.perm[row + i] = (int)((u32*)sm)[i];
}

// the record columns in sorted order
struct GatherIo {
  const int* perm;
  u8* pool; u8* unit; u32* mask; i64* s; i64* p; i64* arrival;     // staged copies (arrival may be null)
};

__global__ void __launch_bounds__(256) k_gather(const __grid_constant__ Params P, const GatherIo G) {
  const size_t total = (size_t)P.S * P.N;
  for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (size_t)gridDim.x * blockDim.x) {
    const size_t row = o - o % P.N;
    const size_t src = row + G.perm[o];
    G.pool[o] = P.a_pool[src]; G.unit[o] = P.a_unit[src]; G.mask[o] = P.a_mask[src];
    G.s[o] = P.a_s[src]; G.p[o] = P.a_p[src];
    if (G.arrival) G.arrival[o] = P.a_arrival[src];
  }
}

// the results back at the actions' own positions
struct ScatterIo {
  const int* perm;
  const int* alloc; const int* node; const int* off; const i64* act;   // staged results, sorted order
  int* o_alloc; int* o_node; int* o_off; i64* o_act;
};

__global__ void __launch_bounds__(256) k_scatter(const __grid_constant__ Params P, const ScatterIo X) {
  const size_t total = (size_t)P.S * P.N;
  for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (size_t)gridDim.x * blockDim.x) {
    const size_t dst = o - o % P.N + X.perm[o];
    X.o_alloc[dst] = X.alloc[o]; X.o_node[dst] = X.node[o]; X.o_off[dst] = X.off[o]; X.o_act[dst] = X.act[o];
  }
}

struct PinIo {
  const int* trajectory; const u32* traj_mem; int max_traj;
  int* traj_node; i64* mem_free; u8* pool_out; int* n_admitted;
};

// One chunk of up to 32 consecutive queue actions, one per lane (`have`: the lane holds one; rec = its record
// index).  Lane j < P keeps node j's free memory (mf) and cores (-1: not a CPU node).  The actions whose
// trajectory has no node yet are taken one after the other, lowest lane first.  Returns the lane of the first
// action whose trajectory finds no node (32 if none); pool_of = the lane's pool afterwards (its trajectory's
// node, or its own pool; untouched for a lane without an action); the actions from the returned lane on keep
// their pools.
__device__ __forceinline__ int pin_chunk(const Params& P, const u8* a_pool, size_t rec, bool have, const int* trajectory,
                                         const u32* traj_mem, int max_traj, int* tn, i64& mf, int cores, int lane,
                                         int& pool_of) {
  int pj = 0xff, t = -1, node = -1, need = 0; u32 mem = 0;
  bool mine = false;                                    // an action of the CPU manager with a trajectory
  if (have) {
    pj = a_pool[rec];
    t = trajectory[rec];
    mine = t >= 0 && t < max_traj && pj < P.P && P.pool[pj].type == TG_POOL_CPU;
    if (mine) {
      node = tn[t]; mem = traj_mem[rec];
      const u32 mk = P.a_mask[rec];
      need = (int)(P.a_unit[rec] & 0x7f) * (mk ? __ffs(mk) : 0);   // cores of the least level
    }
  }
  int first_out = 32;
  u32 open = __ballot_sync(TG_FULL, mine && node < 0);
  while (open) {
    const int b = __ffs(open) - 1;
    const int bt = __shfl_sync(TG_FULL, t, b), bneed = __shfl_sync(TG_FULL, need, b);
    const u32 bmem = __shfl_sync(TG_FULL, mem, b);
    // the eligible node with the most free memory, lowest index on ties
    const bool ok = cores >= 0 && cores >= bneed && mf >= (i64)bmem;
    const i64 best = warp_max64_from_m1(ok ? mf : -1);
    const u32 who = __ballot_sync(TG_FULL, ok && mf == best);
    if (!who) {                                         // no node: the admitted queue ends before this action
      first_out = b;
      if (lane >= b) mine = false;                      // nothing from it on is touched
      break;
    }
    const int bn = __ffs(who) - 1;
    if (lane == bn) mf -= (i64)bmem;
    if (lane == 0) tn[bt] = bn;
    if (mine && t == bt) node = bn;                     // later actions of the trajectory in this chunk follow
    open = __ballot_sync(TG_FULL, mine && node < 0) & ~((2u << b) - 1u);
  }
  if (have) pool_of = (mine && node >= 0) ? node : pj;
  __syncwarp();
  return first_out;
}

__global__ void __launch_bounds__(256) k_pin(const __grid_constant__ Params P, const PinIo X) {
  const int lane = threadIdx.x & 31;
  const int sc = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
  if (sc >= P.S) return;
  const size_t row = (size_t)sc * P.N;
  const int n = min(max(P.n_actions[sc], 0), P.N);
  int* tn = X.traj_node + (size_t)sc * X.max_traj;
  // lane j < P: node j's free memory and cores (-1 cores: not a CPU node)
  i64 mf = 0; int cores = -1;
  if (lane < P.P && P.pool[lane].type == TG_POOL_CPU) { mf = X.mem_free[(size_t)sc * P.P + lane]; cores = P.pool[lane].capacity; }
  int admitted = n;
  for (int c0 = 0; c0 < P.N; c0 += 32) {
    const int i = c0 + lane;
    int pool_of = i < P.N ? P.a_pool[row + i] : 0xff;
    if (admitted == n && c0 < n) {                      // (behind the admitted queue the pool column is copied)
      const int out = pin_chunk(P, P.a_pool, row + i, i < n, X.trajectory, X.traj_mem, X.max_traj, tn, mf, cores, lane, pool_of);
      if (out < 32) admitted = c0 + out;
    }
    if (i < P.N) X.pool_out[row + i] = (u8)pool_of;
  }
  if (lane < P.P && cores >= 0) X.mem_free[(size_t)sc * P.P + lane] = mf;
  if (lane == 0) X.n_admitted[sc] = admitted;
}
