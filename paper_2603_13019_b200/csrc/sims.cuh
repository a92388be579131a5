// Completion-heap simulations of Algorithm 2 (estimate), one THREAD per simulation.
//
// A round needs, per elastic (scenario, pool), the objective of the full candidate list and of
// the list without its last candidate (the first eviction step), each at `depth` levels of the
// first waiting action: 2 * depth independent sequential simulations of |waiting| pop-min /
// push steps.  Each runs on its own 4-ary min-heap in shared memory, laid out interleaved by
// thread (element e of thread t at e * SIM_THREADS + t) so that a warp's accesses never
// conflict whatever nodes its threads touch.  A block serves 64 consecutive simulations
// (same pool, neighbouring scenarios); the kernel is launched once per heap-capacity class and
// a block whose largest heap is not of the class leaves at once.
#pragma once
#include "common.cuh"

#define SIM_THREADS 64

// per (scenario, pool) state handed from the solve kernel to the simulations and the finish kernel
struct TaskState {
  i64 opt[2];     // optimal duration sum of all m candidates / of the first m-1
  i64 est[2];     // estimate of the rest for those two prefixes: min over depths (atomicMin)
  int flags;      // TS_* bits
  int pad;
};
#define TS_SOLVED 1   // both prefixes solved, heap seeds written
#define TS_FAILED 2   // workspace too small

__device__ __forceinline__ int nth_level_of(u32 mask, int d) {
  for (int k = 0; k < d; ++k) mask &= mask - 1;
  return __ffs(mask);
}

// replace the root of thread t's heap by v and restore the heap (rows H..H+3 hold +inf)
__device__ __forceinline__ void heap4_sift(i64* hp, int t, int H, int pos, i64 v) {
  for (;;) {
    int c = 4 * pos + 1;
    if (c >= H) break;
    i64 a0 = hp[(c + 0) * SIM_THREADS + t], a1 = hp[(c + 1) * SIM_THREADS + t];
    i64 a2 = hp[(c + 2) * SIM_THREADS + t], a3 = hp[(c + 3) * SIM_THREADS + t];
    int b01 = a1 < a0 ? 1 : 0, b23 = a3 < a2 ? 3 : 2;
    i64 m01 = a1 < a0 ? a1 : a0, m23 = a3 < a2 ? a3 : a2;
    int bi = m23 < m01 ? b23 : b01;
    i64 bm = m23 < m01 ? m23 : m01;
    if (bm < v) { hp[pos * SIM_THREADS + t] = bm; pos = c + bi; } else break;
  }
  hp[pos * SIM_THREADS + t] = v;
}

// hcap_lo < (largest heap of the block) <= hcap_hi selects the blocks of this launch.
// use_global: heaps live in the arena instead of shared memory (very large heaps).
__global__ void __launch_bounds__(SIM_THREADS) k_sims(const __grid_constant__ Params P, TaskState* ts,
                                                      const i64* seed2, int hcap_lo, int hcap_hi, int use_global) {
  extern __shared__ i64 hp_smem[];
  __shared__ int s_hmax;
  __shared__ i64* s_gl;
  const int t = threadIdx.x;
  const long long sim = (long long)blockIdx.x * SIM_THREADS + t;
  const long long n_sims = (long long)P.P * P.S * 2 * P.depth;
  if (t == 0) s_hmax = 0;
  __syncthreads();

  bool active = false;
  int H = 0, n_list = 0, e = 0, d = 0;
  const i64* seeds = nullptr; const i64* lst = nullptr;
  i64 first_dur = 0;
  TaskState* st = nullptr;
  if (sim < n_sims) {
    d = (int)(sim % P.depth);
    long long x = sim / P.depth;
    e = (int)(x & 1); x >>= 1;
    const int sc = (int)(x % P.S), j = (int)(x / P.S);
    const PoolMeta mt = P.meta[(size_t)sc * P.P + j];
    st = ts + (size_t)sc * P.P + j;
    const int n_ac = mt.count - mt.m;
    if (mt.elastic && mt.m >= 1 + e && (e + n_ac) > 0 && (st->flags & TS_SOLVED)) {
      const size_t row = (size_t)sc * P.N;
      const PoolDev& pd = P.pool[j];
      // first remaining action: the evicted last candidate (e = 1) or the first waiting one
      const int idx = P.order[row + mt.base + mt.m - e];
      int g, gang; u32 fm;
      decode_levels(pd, P.a_unit[row + idx], P.a_mask[row + idx], g, gang, fm);
      if (d < min(P.depth, __popc(fm))) {
        active = true;
        first_dur = duration(clamp_param(P.a_s[row + idx]), clamp_param(P.a_p[row + idx]), nth_level_of(fm, d));
        H = mt.m - e;
        seeds = (e ? seed2 : P.tmin) + row + mt.base;
        lst = P.tmin + row + mt.base + mt.m + (1 - e);
        n_list = n_ac - (1 - e);
      }
    }
  }
  if (active) atomicMax(&s_hmax, H);
  __syncthreads();
  const int hmax = s_hmax;
  if (hmax == 0 || hmax <= hcap_lo || hmax > hcap_hi) return;
  i64* hp = hp_smem;
  if (use_global) {
    if (t == 0) {
      u64 bytes = ((u64)(hmax + 4) * SIM_THREADS * sizeof(i64) + 255) & ~(u64)255;
      u64 off = atomicAdd(P.arena_top, bytes);
      s_gl = off + bytes <= P.arena_bytes ? (i64*)(P.arena + off) : nullptr;
    }
    __syncthreads();
    hp = s_gl;
    if (!hp) { if (active) atomicOr(&st->flags, TS_FAILED); return; }
  }
  if (!active) return;

  for (int i = 0; i < H; ++i) hp[i * SIM_THREADS + t] = seeds[i];
  for (int i = H; i < H + 4; ++i) hp[i * SIM_THREADS + t] = TG_INF;
  for (int s0 = (H - 2) / 4; s0 >= 0 && H > 1; --s0) heap4_sift(hp, t, H, s0, hp[s0 * SIM_THREADS + t]);

  i64 tmp = 0;
  i64 dur = first_dur;
  for (int k = 0; k <= n_list; ++k) {
    i64 nxt = k < n_list ? lst[k] : 0;                 // fetch the next duration early
    i64 v = hp[t] + dur;                               // pop the earliest completion, push ts + T
    tmp = sat_add(tmp, v);
    heap4_sift(hp, t, H, 0, v);
    dur = nxt;
  }
  atomicMin((u64*)&st->est[e], (u64)tmp);
}
