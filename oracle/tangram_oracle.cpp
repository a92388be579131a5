// TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT.
//
// Plain, slow, sequential CPU oracle of the elastic scheduling round of ARL-Tangram
// (arxiv 2603.13019).  It exists so that the CUDA library can be checked against it
// bit for bit; only tests, the smoke check and the CPU-baseline leg of the benchmark
// may call it.  It shares no code with the CUDA path.
//
// What follows the paper step by step (heuristic, so no closed-form definition):
//   * Eq. 1 (duration at m units) in its integer-microsecond form        -> duration()
//   * Algorithm 1 (Elastic Resource Scheduling): candidate prefix, split by key
//     resource, all-inelastic shortcut, greedy eviction                   -> schedule_round()
//   * Algorithm 2 (ACTs approximation): exact part + completion-heap estimate
//                                                                        -> approx_objective(), estimate()
//   * Algorithm 3 (topology-agnostic DPArrange) with the Basic DP operator -> dp_basic()
//   * Algorithm 4 (GPU-topology-aware DP operator): chunk-count state, mixed-radix
//     Encode/Decode                                                       -> dp_gpu(), encode(), decode()
//   * Section 5.1 (quota / concurrency limits), Section 5.2 (exclusive cores, same
//     NUMA domain first), Section 5.3 (aligned power-of-two chunks, smallest
//     sufficient chunk, split)                                            -> place_*()
//   * Section 3 workflow (submit, queue, schedule, execute, return)       -> replay loop
//
// Readings taken where the paper is silent, ambiguous or garbled (all restated in the
// design document; R-numbers are local to this build):
//   R1  T(r) = s + floor(p / r) in integer microseconds, r = units / g; s, p clamped to
//       [0, 2^40].  (Eq. 1 is real valued; this is its invariant + scalable form.)
//   R2  "inelastic" means the action has exactly one allowed level.
//   R3  The candidate prefix is one prefix of the whole queue, across all pools.
//   R4  DPArrange returns the best over all unit totals j <= n, not only j = n (with
//       discrete level sets j = n can be unreachable).
//   R5  Ties: minimise sum of durations, then total units, then (k_m, ..., k_1)
//       lexicographically, i.e. a later queue position gets less.  This is what strict
//       '<' with ascending k and ascending j yields in Algorithm 3.
//   R6  Eviction steps t = 1 .. |C_j|-1; the head candidate is never evicted.
//   R7  estimate(): every depth iteration works on its own copy of the heap; an empty
//       remaining list costs 0; times are relative to 'now'.  Depth d uses the d-th
//       smallest level of the first remaining action and stops when it has fewer
//       levels; all other remaining actions take their smallest level.  A pop frees one
//       slot regardless of units (the paper's approximation).  Only actions running on
//       the same pool seed the heap.
//   R11 A multiset of aligned power-of-two chunk requests fits the free space iff for
//       every size s the units requested at sizes >= s do not exceed the units held in
//       maximal free aligned blocks of size >= s.
//   R12 Algorithm 4's state counts granted requests per chunk size; a level of g*r units
//       is r chunks of g GPUs, or one chunk of g*r GPUs for GANG actions.  A state is
//       valid iff R11 holds for it.
//   R13 GPU placement handles requests by (size descending, queue position ascending),
//       each taking the smallest sufficient free block, lowest (node, start) on ties, low
//       end of a split block.  CPU placement: queue order; best-fit NUMA domain (fewest
//       free cores that still fit, lowest index on ties), lowest core ids; otherwise
//       ascending domains.  API pools report the units consumed before the grant.
//   R14 Objective sums saturate at INT64_MAX.
//   R17 Quota pools refill to capacity at multiples of their window.
//   R19 Service cache (Section 5.3, evict on execution): every GPU remembers up to K service
//       instances, an instance being (service id, chunk size) since different degrees of
//       parallelism of a service count as distinct services; a chunk caches an instance iff
//       every GPU of the chunk remembers it.
//   R20 Among the free blocks of the level that the allocation rule picks (smallest
//       sufficient), one whose granted chunk (its low end) caches the requested instance is
//       preferred; then lowest (node, start).
//   R21 A grant refreshes the instance's last use on every GPU of the chunk; on a miss each
//       GPU first overwrites an empty entry (lowest index), else its least recently used one
//       (lowest index among equals).
//   R22 An action one of whose chunks missed runs restore_us longer (restoration from host
//       memory precedes execution).  The scheduler's duration model does not see this: it
//       decides before the placement.
//   R23 Cost vectors (Section 4.1, vectorized resource cost): besides its key resource an
//       action may name up to two further pools with a fixed amount each (memory beside the
//       cores, quotas of other sites).  Such a pool is a quota or concurrency pool other than
//       the key pool and the amount lies in 1 .. its capacity; anything else is a bad record.
//       Only the key resource is elastic (the paper's assumption), durations follow it alone.
//   R24 accommodate (Algorithm 1, candidate prefix): an action fits if its least key level
//       and every further amount fit on top of what the actions before it in the queue ask.
//   R25 R_k handed to DPArrange for pool k is what is free minus the further amounts that ALL
//       candidates of the prefix ask of k, whatever their key pool; an evicted candidate's
//       amounts are not handed back within the round.
//   R26 A started action consumes its further amounts (a quota pool counts them in the
//       window, a concurrency pool holds them until the action finishes); an evicted one
//       consumes nothing.  They are booked after all pools have placed their key grants, so
//       a quota pool's place_off counts what was used before the round plus the key grants
//       ahead in queue order.
//   R27 Other queue orders (Section 4.2: the algorithm works with other ordering algorithms): the
//       waiting queue is sorted by a key before the round -- shortest or longest duration at the
//       least level (Eq. 1), or earliest arrival -- equal keys in queue order; everything after
//       that is Algorithm 1 on the sorted queue.  An invalid record has key 0.
//   R28 Per-node CPU scheduling (Section 5.2): every CPU pool is one node with a scheduler of its
//       own.  In queue order, the first action of a trajectory pins it: among the nodes with at
//       least as many cores as the action's least level and at least the trajectory's memory
//       free, the one with the most free memory (lowest index on ties) takes the trajectory and
//       sets its memory aside; all its actions run there.  An action whose trajectory finds no
//       node ends the admitted queue (first come first served: what stands behind it waits).
//   R29 In a replay the trajectories are pinned as their actions arrive: an arrival whose trajectory
//       finds no node waits outside the queue, and so does everything that arrives after it; it
//       is tried again every round.  When the action marked as its trajectory's last one ends,
//       the trajectory's memory goes back to its node and the trajectory is no longer pinned.
//
// The paper prints no worked example of a schedule.  estimate() and the eviction loop are
// heuristics; they are pinned by closed forms, by an independent list-scheduling statement
// and by cases worked by hand in the tests (two accepted evictions and a refused third,
// evicted candidates ahead of the waiting list, a running action of the same pool in the
// heap, saturating sums), DPArrange by exhaustive enumeration, the chunk test by brute-force
// packing, placement by worked examples; the service cache, the cost vectors, the queue orders
// and the trajectory pinning by hand-worked cases of their own (same-level preference, LRU order,
// restoration once per action; an amount that ends the prefix, a later candidate's amount set
// aside, an evicted candidate that consumes nothing, concurrency and quota bookkeeping over
// rounds; keys and ties of the three orders, the ordered round against the plain round on the
// permuted records, a one-core trace whose three orders differ; most-free-memory node, the core and
// memory filters, the admitted queue, a replay in which an arrival waits at the gate until a
// trajectory's last action gives its memory back).
#include <algorithm>
#include <climits>
#include <cstdint>
#include <cstring>
#include <functional>
#include <map>
#include <queue>
#include <vector>

namespace {

typedef long long i64;
const i64 INF = LLONG_MAX;
const i64 PARAM_MAX = 1LL << 40;
enum { POOL_CPU = 0, POOL_GPU = 1, POOL_API = 2 };
enum { STATUS_OK = 0, STATUS_BAD_ACTION = 1, STATUS_UNSORTED = 2 };

struct PoolDesc { int type, capacity, group, window_us; };

struct Action {
  int pool = 0, g = 1;
  bool gang = false, valid = true;
  std::vector<int> r;       // allowed multiplicities, ascending
  i64 s = 0, p = 0, arrival = 0;
  int service = -1;         // requested service (GPU pools), -1: none
  i64 restore = 0;          // restoration time if the granted chunk does not cache the instance
  std::vector<std::pair<int, int> > side;   // further (pool, amount) entries of the cost vector (R23)
  bool elastic() const { return r.size() > 1; }
};

i64 clamp_param(i64 v) { return v < 0 ? 0 : (v > PARAM_MAX ? PARAM_MAX : v); }
i64 sat_add(i64 a, i64 b) { return a > INF - b ? INF : a + b; }           // a, b >= 0 (R14)
bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }
int log2i(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

// Eq. 1, integer form (R1): duration of the action at multiplicity r (= g*r units).
i64 duration(const Action& a, int r) { return a.s + a.p / r; }

Action decode_action(int pool, int unit, uint32_t mask, i64 s, i64 p, i64 arrival,
                     const std::vector<PoolDesc>& pools) {
  Action a;
  a.pool = pool; a.g = unit & 0x7F; a.gang = (unit & 0x80) != 0;
  a.s = clamp_param(s); a.p = clamp_param(p); a.arrival = arrival;
  if (pool < 0 || pool >= (int)pools.size() || a.g == 0) { a.valid = false; return a; }
  const PoolDesc& pd = pools[pool];
  if (pd.type != POOL_GPU) a.gang = false;
  if (pd.type == POOL_GPU && !a.gang && !(is_pow2(a.g) && a.g <= pd.group)) { a.valid = false; return a; }
  for (int r = 1; r <= 32; ++r) {
    if (!(mask >> (r - 1) & 1u)) continue;
    if (pd.type == POOL_GPU && a.gang && !(is_pow2(a.g * r) && a.g * r <= pd.group)) continue;
    a.r.push_back(r);
  }
  if (a.r.empty()) a.valid = false;
  return a;
}

// ------------------------------------------------------------- GPU chunk topology
// Section 5.3: a chunk is [start, start + 2^a) with 2^a dividing start.  The free space
// of a node is described by its maximal free aligned blocks.
void free_blocks_of(uint8_t busy, int start, int size, int F[4]) {
  int bits = ((1 << size) - 1) << start;
  if ((busy & bits) == 0) { F[log2i(size)]++; return; }
  if (size == 1) return;
  free_blocks_of(busy, start, size / 2, F);
  free_blocks_of(busy, start + size / 2, size / 2, F);
}

void free_block_counts(const std::vector<uint8_t>& node_busy, int group, int F[4]) {
  F[0] = F[1] = F[2] = F[3] = 0;
  for (uint8_t b : node_busy) free_blocks_of(b, 0, group, F);
}

// R11: requests n[l] of size 2^l fit into free blocks F[l] of size 2^l.
bool chunks_fit(const int n[4], const int F[4]) {
  int demand = 0, room = 0;
  for (int l = 3; l >= 0; --l) {
    demand += n[l] << l;
    room += F[l] << l;
    if (demand > room) return false;
  }
  return true;
}

// what a level adds to the request counts (R12)
void add_level(const Action& a, int r, int n[4], int sign) {
  if (a.gang) n[log2i(a.g * r)] += sign;
  else n[log2i(a.g)] += sign * r;
}

// Algorithm 4, Encode / Decode with radices N_s + 1.
i64 encode(const int n[4], const int N[4]) {
  return n[0] + (i64)(N[0] + 1) * (n[1] + (i64)(N[1] + 1) * (n[2] + (i64)(N[2] + 1) * n[3]));
}
void decode(i64 j, const int N[4], int n[4]) {
  n[0] = (int)(j % (N[0] + 1)); j /= (N[0] + 1);
  n[1] = (int)(j % (N[1] + 1)); j /= (N[1] + 1);
  n[2] = (int)(j % (N[2] + 1)); j /= (N[2] + 1);
  n[3] = (int)j;
}

// ------------------------------------------------------------- DPArrange (Alg. 3, 4)
struct Cell { i64 value; int choice; };   // choice = multiplicity r given to the row's task
typedef std::map<i64, Cell> Row;          // DP index j -> cell (only finite cells are stored)

struct DpTable {
  bool gpu = false;
  std::vector<Row> rows;                          // GPU operator: rows[i] = first i tasks
  std::vector<std::vector<Cell> > dense;          // Basic operator: dense[i][j], value INF = invalid
  int N[4] = {0, 0, 0, 0};
  int units_of(i64 j) const {
    if (!gpu) return (int)j;
    int n[4]; decode(j, N, n);
    return n[0] + 2 * n[1] + 4 * n[2] + 8 * n[3];
  }
  const Cell& at(int i, i64 j) const { return gpu ? rows[i].at(j) : dense[i][(size_t)j]; }
  // finite cells of row q in ascending DP index
  std::vector<std::pair<i64, Cell> > cells(int q) const {
    std::vector<std::pair<i64, Cell> > out;
    if (gpu) out.assign(rows[q].begin(), rows[q].end());
    else
      for (size_t j = 0; j < dense[q].size(); ++j)
        if (dense[q][j].value != INF) out.push_back(std::make_pair((i64)j, dense[q][j]));
    return out;
  }
};

// Algorithm 3 with the Basic DP operator: j = units used by the first i tasks.
// Prev(j,k) = j-k; IsValid(j', S_1..i-1) (is j' an exact sum of one level per earlier
// task) holds exactly when dp[i-1][j'] is finite, so the finite cells are the valid ones.
DpTable dp_basic(const std::vector<const Action*>& C, int U) {
  DpTable t;
  int m = (int)C.size();
  i64 sum_max = 0;
  for (const Action* a : C) sum_max += (i64)a->g * a->r.back();
  int n = (int)std::min<i64>(U, sum_max);                       // End(U), End(S)
  t.dense.assign(m + 1, std::vector<Cell>(n + 1, Cell{INF, 0}));
  std::vector<std::vector<Cell> >& dp = t.dense;
  dp[0][0].value = 0;
  int start_prev = 0, start_cur = m ? C[0]->g * C[0]->r.front() : 0;   // Start(S_1)
  for (int i = 1; i <= m; ++i) {
    const Action& a = *C[i - 1];
    for (int j = start_cur; j <= n; ++j) {
      for (int r : a.r) {                                       // ascending k
        int jp = j - a.g * r;                                   // Prev(j, k)
        if (jp < start_prev || dp[i - 1][jp].value == INF) continue;  // IsValid
        i64 cand = dp[i - 1][jp].value + duration(a, r);
        if (cand < dp[i][j].value) dp[i][j] = Cell{cand, r};
      }
    }
    start_prev = start_cur;
    if (i < m) start_cur += C[i]->g * C[i]->r.front();          // Start(S_1..i+1)
  }
  return t;
}

// Algorithm 3 with the GPU operator (Alg. 4, R12): j = Encode(request counts).  The
// dense index space is far too large to sweep, so only reachable states are stored and a
// row is built by extending the previous one; for a fixed target the smallest level wins
// ties, which is what the sweep over ascending k with strict '<' does.
// With 'prune' a state of row i is kept only if the least-required requests of tasks
// i+1..m still fit on top of it: the other states cannot lead to any state of the last
// row, so the result is the same and only the work shrinks (a test compares both).
DpTable dp_gpu(const std::vector<const Action*>& C, const int F[4], bool prune) {
  DpTable t;
  t.gpu = true;
  int room = 0;
  for (int l = 3; l >= 0; --l) { room += F[l] << l; t.N[l] = room >> l; }   // most requests of size 2^l
  int m = (int)C.size();
  std::vector<std::vector<int> > later(m + 1, std::vector<int>(4, 0));      // min requests of tasks i+1..m
  for (int i = m - 1; i >= 0; --i) {
    later[i] = later[i + 1];
    add_level(*C[i], C[i]->r.front(), later[i].data(), +1);
  }
  t.rows.resize(m + 1);
  int zero[4] = {0, 0, 0, 0};
  t.rows[0][encode(zero, t.N)] = Cell{0, 0};
  for (int i = 1; i <= m; ++i) {
    const Action& a = *C[i - 1];
    for (const auto& kv : t.rows[i - 1]) {
      int n[4]; decode(kv.first, t.N, n);
      for (int r : a.r) {
        int nn[4] = {n[0], n[1], n[2], n[3]};
        add_level(a, r, nn, +1);
        if (!chunks_fit(nn, F)) continue;                        // IsValid
        if (prune) {
          int all[4] = {nn[0] + later[i][0], nn[1] + later[i][1], nn[2] + later[i][2], nn[3] + later[i][3]};
          if (!chunks_fit(all, F)) continue;
        }
        i64 cand = kv.second.value + duration(a, r);
        i64 j = encode(nn, t.N);
        auto it = t.rows[i].find(j);
        if (it == t.rows[i].end()) t.rows[i][j] = Cell{cand, r};
        else if (cand < it->second.value || (cand == it->second.value && r < it->second.choice))
          it->second = Cell{cand, r};
      }
    }
  }
  return t;
}

i64 dp_prev(const DpTable& t, const Action& a, i64 j, int r) {
  if (!t.gpu) return j - (i64)a.g * r;
  int n[4]; decode(j, t.N, n);
  add_level(a, r, n, -1);
  return encode(n, t.N);
}

// Backtrack (Alg. 3, last loop) from state j of row q; alloc[i] = multiplicity of task i.
std::vector<int> backtrack(const DpTable& t, const std::vector<const Action*>& C, int q, i64 j) {
  std::vector<int> alloc(q, 0);
  for (int i = q; i >= 1; --i) {
    int r = t.at(i, j).choice;
    alloc[i - 1] = r;
    j = dp_prev(t, *C[i - 1], j, r);
  }
  return alloc;
}

// Result of DPArrange under R4 / R5: the best cell of the last row.  Returns false when
// the tasks do not fit at all (cannot happen for prefixes of an accommodated candidate list).
bool best_of_last_row(const DpTable& t, const std::vector<const Action*>& C,
                      i64* value, std::vector<int>* alloc) {
  int q = (int)C.size();
  std::vector<std::pair<i64, Cell> > row = t.cells(q);
  if (row.empty()) return false;
  i64 best = INF; int best_units = INT_MAX;
  for (const auto& kv : row) {
    int u = t.units_of(kv.first);
    if (kv.second.value < best || (kv.second.value == best && u < best_units)) {
      best = kv.second.value; best_units = u;
    }
  }
  bool have = false;
  std::vector<int> pick;
  for (const auto& kv : row) {
    if (kv.second.value != best || t.units_of(kv.first) != best_units) continue;
    std::vector<int> cand = backtrack(t, C, q, kv.first);
    // compare (k_q, ..., k_1): later queue positions first
    bool smaller = !have;
    if (have)
      for (int i = q - 1; i >= 0; --i) {
        int ka = C[i]->g * cand[i], kb = C[i]->g * pick[i];
        if (ka != kb) { smaller = ka < kb; break; }
      }
    if (smaller) { pick = cand; have = true; }
  }
  *value = best; *alloc = pick;
  return true;
}

// ------------------------------------------------------------- Algorithm 2
// estimate(heap, remaining): completion-heap estimate of the actions not scheduled now.
i64 estimate(const std::vector<i64>& heap_init, const std::vector<const Action*>& rest, int depth) {
  if (rest.empty()) return 0;
  i64 obj = INF;
  for (int d = 1; d <= depth; ++d) {
    if ((int)rest[0]->r.size() < d) break;
    std::priority_queue<i64, std::vector<i64>, std::greater<i64> > heap(heap_init.begin(), heap_init.end());
    i64 tmp = 0;
    for (size_t i = 0; i < rest.size(); ++i) {
      i64 T = duration(*rest[i], i == 0 ? rest[0]->r[d - 1] : rest[i]->r.front());
      i64 ts = 0;
      if (!heap.empty()) { ts = heap.top(); heap.pop(); }
      tmp = sat_add(tmp, ts + T);
      heap.push(ts + T);
    }
    if (tmp < obj) obj = tmp;
  }
  return obj;
}

struct PoolRuntime {
  PoolDesc d;
  std::vector<int> core_owner;       // CPU: action id or -1
  std::vector<uint8_t> node_busy;    // GPU: bit b = GPU b busy
  int cache_slots = 0;               // GPU: instances a GPU remembers (0: no service cache)
  std::vector<unsigned> cache_tag;   // GPU: [gpu][slot] instance tag, 0 = empty
  std::vector<i64> cache_use;        // GPU: [gpu][slot] time of last use
  int api_used = 0;                  // quota pools: tokens used in the current window
  i64 window = 0;
  int in_use = 0;                    // concurrency pools: units held
  int free_units() const {
    if (d.type == POOL_CPU) { int f = 0; for (int o : core_owner) f += o < 0; return f; }
    if (d.type == POOL_API) return d.window_us > 0 ? d.capacity - api_used : d.capacity - in_use;
    int f = 0; for (uint8_t b : node_busy) f += d.group - __builtin_popcount(b); return f;
  }
  int busy_units() const { return d.capacity - free_units(); }
};

struct Chunk { int node, start, size; };
struct Running { i64 finish; int action, pool, units; std::vector<Chunk> chunks; };
struct Grant { int action, r, units, node, off; std::vector<Chunk> chunks; bool missed = false; };

// what DPArrange needs to know about the pool: free units, or free chunk counts
struct PoolRoom { bool gpu; int free_units; int F[4]; };

// DPArrange(R_j, C): optimal duration sum and multiplicities for the task list C
bool dp_arrange(const std::vector<const Action*>& C, const PoolRoom& room, bool prune,
                i64* value, std::vector<int>* alloc) {
  DpTable t = room.gpu ? dp_gpu(C, room.F, prune) : dp_basic(C, room.free_units);
  return best_of_last_row(t, C, value, alloc);
}

// exactObj + approxObj for the first q candidates (Alg. 2, getApproximatedObjective)
i64 approx_objective(const std::vector<const Action*>& Cj, int q, const PoolRoom& room,
                     const std::vector<const Action*>& ACj, const std::vector<i64>& running_rel,
                     int depth, std::vector<int>* alloc) {
  i64 exact = 0;
  std::vector<const Action*> kept(Cj.begin(), Cj.begin() + q);
  dp_arrange(kept, room, true, &exact, alloc);
  std::vector<i64> heap(running_rel);
  for (int i = 0; i < q; ++i) heap.push_back(duration(*Cj[i], (*alloc)[i]));
  std::vector<const Action*> rest(Cj.begin() + q, Cj.end());      // evicted, in queue order,
  rest.insert(rest.end(), ACj.begin(), ACj.end());                // ahead of the others
  return sat_add(exact, estimate(heap, rest, depth));
}

// ------------------------------------------------------------- placement (R13)
// instance tag of (service, chunk size); 0 is "empty"
unsigned instance_tag(int service, int size) { return ((unsigned)service << 3 | (unsigned)log2i(size)) + 1u; }

bool chunk_caches(const PoolRuntime& pr, int node, int start, int size, unsigned tag) {
  for (int b = start; b < start + size; ++b) {
    bool has = false;
    for (int k = 0; k < pr.cache_slots; ++k) has |= pr.cache_tag[(size_t)(node * pr.d.group + b) * pr.cache_slots + k] == tag;
    if (!has) return false;
  }
  return true;
}

// R21: the instance becomes the most recently used one on every GPU of the chunk
void cache_touch(PoolRuntime& pr, int node, int start, int size, unsigned tag, i64 now) {
  for (int b = start; b < start + size; ++b) {
    unsigned* tg = &pr.cache_tag[(size_t)(node * pr.d.group + b) * pr.cache_slots];
    i64* us = &pr.cache_use[(size_t)(node * pr.d.group + b) * pr.cache_slots];
    int at = -1;
    for (int k = 0; k < pr.cache_slots && at < 0; ++k) if (tg[k] == tag) at = k;
    for (int k = 0; k < pr.cache_slots && at < 0; ++k) if (tg[k] == 0) at = k;
    if (at < 0) { at = 0; for (int k = 1; k < pr.cache_slots; ++k) if (us[k] < us[at]) at = k; }
    tg[at] = tag; us[at] = now;
  }
}

void place_gpu(PoolRuntime& pr, const std::vector<Action>& acts, std::vector<Grant>& grants,
               const std::vector<int>& which, i64 now = 0) {
  struct Req { int size, rank, rep, grant; };
  std::vector<Req> reqs;
  for (int gi : which) {
    const Action& a = acts[grants[gi].action];
    if (a.gang) reqs.push_back(Req{a.g * grants[gi].r, gi, 0, gi});
    else for (int c = 0; c < grants[gi].r; ++c) reqs.push_back(Req{a.g, gi, c, gi});
  }
  std::stable_sort(reqs.begin(), reqs.end(), [](const Req& x, const Req& y) {
    if (x.size != y.size) return x.size > y.size;
    if (x.rank != y.rank) return x.rank < y.rank;
    return x.rep < y.rep;
  });
  for (const Req& rq : reqs) {
    const Action& a = acts[grants[rq.grant].action];
    const bool cached_pool = pr.cache_slots > 0 && a.service >= 0;
    const unsigned tag = cached_pool ? instance_tag(a.service, rq.size) : 0u;
    int best_size = INT_MAX, best_node = -1, best_start = -1;
    bool best_hit = false;
    for (int node = 0; node < (int)pr.node_busy.size(); ++node) {
      // maximal free aligned blocks of this node: smallest sufficient one, a caching one first (R20)
      std::function<void(int, int)> walk = [&](int start, int size) {
        int bits = ((1 << size) - 1) << start;
        if ((pr.node_busy[node] & bits) == 0) {
          if (size < rq.size) return;
          const bool hit = cached_pool && chunk_caches(pr, node, start, rq.size, tag);
          if (size < best_size || (size == best_size && hit && !best_hit)) {
            best_size = size; best_node = node; best_start = start; best_hit = hit;
          }
          return;
        }
        if (size == 1) return;
        walk(start, size / 2); walk(start + size / 2, size / 2);
      };
      walk(0, pr.d.group);
    }
    if (best_node < 0) continue;                                   // cannot happen (R11)
    pr.node_busy[best_node] |= (uint8_t)(((1 << rq.size) - 1) << best_start);
    Grant& g = grants[rq.grant];
    g.chunks.push_back(Chunk{best_node, best_start, rq.size});
    if (rq.rep == 0) { g.node = best_node; g.off = best_start; }
    if (cached_pool) {
      if (!best_hit) g.missed = true;                              // R22
      cache_touch(pr, best_node, best_start, rq.size, tag, now);
    }
  }
}

void place_cpu(PoolRuntime& pr, std::vector<Grant>& grants, const std::vector<int>& which) {
  int D = pr.d.capacity / pr.d.group;
  for (int gi : which) {
    Grant& g = grants[gi];
    int best = -1, best_free = INT_MAX;
    for (int dmn = 0; dmn < D; ++dmn) {
      int f = 0;
      for (int c = dmn * pr.d.group; c < (dmn + 1) * pr.d.group; ++c) f += pr.core_owner[c] < 0;
      if (f >= g.units && f < best_free) { best_free = f; best = dmn; }
    }
    int need = g.units, first = -1;
    int lo = best >= 0 ? best * pr.d.group : 0, hi = best >= 0 ? (best + 1) * pr.d.group : pr.d.capacity;
    for (int c = lo; c < hi && need > 0; ++c)
      if (pr.core_owner[c] < 0) { pr.core_owner[c] = g.action; if (first < 0) first = c; --need; }
    g.node = first / pr.d.group; g.off = first;
  }
}

void place_api(PoolRuntime& pr, std::vector<Grant>& grants, const std::vector<int>& which) {
  for (int gi : which) {
    Grant& g = grants[gi];
    g.node = 0;
    if (pr.d.window_us > 0) { g.off = pr.api_used; pr.api_used += g.units; }
    else { g.off = pr.in_use; pr.in_use += g.units; }
  }
}

// ------------------------------------------------------------- Algorithm 1
// One invocation of the scheduler on waiting queue W (queue order) at time 'now'.
// Mutates the pool state by placing what it selects; returns the grants.
std::vector<Grant> schedule_round(std::vector<PoolRuntime>& pools, const std::vector<Action>& acts,
                                  const std::vector<int>& W, const std::vector<Running>& E,
                                  i64 now, int depth) {
  int k = (int)pools.size();
  // line 2: C = W[:n], n = largest prefix that fits every pool at least-required units
  std::vector<int> used(k, 0);
  std::vector<std::vector<int> > req(k, std::vector<int>(4, 0));
  std::vector<std::vector<int> > F(k, std::vector<int>(4, 0));
  std::vector<int> freeu(k, 0);
  for (int j = 0; j < k; ++j) {
    freeu[j] = pools[j].free_units();
    if (pools[j].d.type == POOL_GPU) free_block_counts(pools[j].node_busy, pools[j].d.group, F[j].data());
  }
  size_t n = 0;
  for (; n < W.size(); ++n) {
    const Action& a = acts[W[n]];
    int j = a.pool;
    if (pools[j].d.type == POOL_GPU) {
      int nn[4] = {req[j][0], req[j][1], req[j][2], req[j][3]};
      add_level(a, a.r.front(), nn, +1);
      if (!chunks_fit(nn, F[j].data())) break;
      for (int l = 0; l < 4; ++l) req[j][l] = nn[l];
    } else {
      if (used[j] + a.g * a.r.front() > freeu[j]) break;
    }
    // R24: the further amounts of the cost vector have to fit as well
    std::vector<int> extra(k, 0);
    bool fits = true;
    for (const std::pair<int, int>& c : a.side) {
      extra[c.first] += c.second;
      fits &= used[c.first] + extra[c.first] <= freeu[c.first];
    }
    if (!fits) break;
    if (pools[j].d.type != POOL_GPU) used[j] += a.g * a.r.front();
    for (int q = 0; q < k; ++q) used[q] += extra[q];
  }
  // R25: what the candidates ask of a pool beside their key resource is set aside
  std::vector<int> aside(k, 0);
  for (size_t i = 0; i < n; ++i)
    for (const std::pair<int, int>& c : acts[W[i]].side) aside[c.first] += c.second;
  std::vector<Grant> grants;
  for (int j = 0; j < k; ++j) {                                    // line 3
    std::vector<const Action*> Cj, ACj;
    std::vector<int> Cid;
    for (size_t i = 0; i < W.size(); ++i) {
      if (acts[W[i]].pool != j) continue;
      if (i < n) { Cj.push_back(&acts[W[i]]); Cid.push_back(W[i]); }
      else ACj.push_back(&acts[W[i]]);
    }
    int m = (int)Cj.size();
    std::vector<int> alloc;
    int keep = m;
    bool any_elastic = false;
    for (const Action* a : Cj) any_elastic |= a->elastic();
    if (!any_elastic) {                                            // lines 5-6
      for (const Action* a : Cj) alloc.push_back(a->r.front());
    } else {
      std::vector<i64> running_rel;
      for (const Running& e : E) if (e.pool == j) running_rel.push_back(std::max<i64>(0, e.finish - now));
      PoolRoom room;
      room.gpu = pools[j].d.type == POOL_GPU; room.free_units = freeu[j] - aside[j];
      for (int l = 0; l < 4; ++l) room.F[l] = F[j][l];
      i64 obj = approx_objective(Cj, m, room, ACj, running_rel, depth, &alloc);   // line 8
      for (int tt = 1; tt <= m - 1; ++tt) {                        // lines 9-14 (R6)
        std::vector<int> alloc2;
        i64 nobj = approx_objective(Cj, m - tt, room, ACj, running_rel, depth, &alloc2);
        if (nobj >= obj) break;
        obj = nobj; alloc = alloc2; keep = m - tt;
      }
    }
    std::vector<int> which;
    for (int i = 0; i < keep; ++i) {
      Grant g;
      g.action = Cid[i]; g.r = alloc[i]; g.units = Cj[i]->g * alloc[i]; g.node = -1; g.off = -1;
      which.push_back((int)grants.size());
      grants.push_back(g);
    }
    if (pools[j].d.type == POOL_GPU) place_gpu(pools[j], acts, grants, which, now);
    else if (pools[j].d.type == POOL_CPU) place_cpu(pools[j], grants, which);
    else place_api(pools[j], grants, which);
  }
  for (const Grant& g : grants)                                    // R26
    for (const std::pair<int, int>& c : acts[g.action].side) {
      PoolRuntime& pr = pools[c.first];
      if (pr.d.window_us > 0) pr.api_used += c.second; else pr.in_use += c.second;
    }
  return grants;
}

struct CacheIo { int slots; unsigned* tag; i64* use; };   // per scenario: [node][8][slots], in and out

std::vector<PoolRuntime> fresh_pools(const std::vector<PoolDesc>& pd, const uint8_t* gpu_busy,
                                     const CacheIo* cache = nullptr) {
  std::vector<PoolRuntime> pools(pd.size());
  int node0 = 0;
  for (size_t j = 0; j < pd.size(); ++j) {
    pools[j].d = pd[j];
    if (pd[j].type == POOL_CPU) pools[j].core_owner.assign(pd[j].capacity, -1);
    if (pd[j].type == POOL_GPU) {
      int nodes = pd[j].capacity / pd[j].group;
      pools[j].node_busy.assign(nodes, 0);
      if (gpu_busy)
        for (int v = 0; v < nodes; ++v) pools[j].node_busy[v] = gpu_busy[node0 + v] & (uint8_t)((1 << pd[j].group) - 1);
      if (cache && cache->slots > 0) {
        pools[j].cache_slots = cache->slots;
        pools[j].cache_tag.assign((size_t)nodes * pd[j].group * cache->slots, 0u);
        pools[j].cache_use.assign((size_t)nodes * pd[j].group * cache->slots, 0);
        for (int v = 0; v < nodes; ++v)
          for (int b = 0; b < pd[j].group; ++b)
            for (int k = 0; k < cache->slots; ++k) {
              const size_t src = ((size_t)(node0 + v) * 8 + b) * cache->slots + k;
              const size_t dst = ((size_t)v * pd[j].group + b) * cache->slots + k;
              pools[j].cache_tag[dst] = cache->tag[src]; pools[j].cache_use[dst] = cache->use[src];
            }
      }
      node0 += nodes;
    }
  }
  return pools;
}

bool load_actions(std::vector<Action>& acts, int n, const std::vector<PoolDesc>& pd,
                  const uint8_t* pool, const uint8_t* unit, const uint32_t* mask,
                  const i64* s, const i64* p, const i64* arrival,
                  const uint16_t* service = nullptr, const i64* restore = nullptr,
                  int n_side = 0, const uint8_t* side_pool = nullptr, const uint16_t* side_units = nullptr,
                  size_t plane = 0) {
  acts.resize(n);
  bool ok = true;
  for (int i = 0; i < n; ++i) {
    acts[i] = decode_action(pool[i], unit[i], mask[i], s[i], p[i], arrival ? arrival[i] : 0, pd);
    if (service && service[i] != 0xffff) acts[i].service = service[i];
    if (restore) acts[i].restore = clamp_param(restore[i]);
    for (int e = 0; e < n_side && side_pool && side_units; ++e) {    // R23
      const int k = side_pool[e * plane + i], c = side_units[e * plane + i];
      if (k == 0xff) continue;
      if (k >= (int)pd.size() || pd[k].type != POOL_API || k == acts[i].pool || c < 1 || c > pd[k].capacity)
        acts[i].valid = false;
      else acts[i].side.push_back(std::make_pair(k, c));
    }
    ok &= acts[i].valid;
  }
  return ok;
}

// the pools' cache state back to the caller's arrays
void store_cache(const std::vector<PoolRuntime>& pools, const CacheIo* cache) {
  if (!cache || cache->slots <= 0) return;
  int node0 = 0;
  for (const PoolRuntime& pr : pools) {
    if (pr.d.type != POOL_GPU) continue;
    const int nodes = pr.d.capacity / pr.d.group;
    for (int v = 0; v < nodes; ++v)
      for (int b = 0; b < pr.d.group; ++b)
        for (int k = 0; k < cache->slots; ++k) {
          const size_t dst = ((size_t)(node0 + v) * 8 + b) * cache->slots + k;
          const size_t src = ((size_t)v * pr.d.group + b) * cache->slots + k;
          cache->tag[dst] = pr.cache_tag[src]; cache->use[dst] = pr.cache_use[src];
        }
    node0 += nodes;
  }
}

// Trajectories pinned on arrival during a replay (R28, R29): null trajectory = none of it.
struct PinIo { const int* trajectory; const uint32_t* traj_mem; const uint8_t* traj_last; int max_traj;
               int* traj_node; i64* mem_free; uint8_t* pool_out; };

// R28 for one arriving action: true if it may join the queue (its trajectory has, or just got, a node).
bool pin_on_arrival(const PinIo& io, const std::vector<PoolDesc>& pd, Action& a, int* tn, i64* mf, size_t at) {
  int t = io.trajectory[at];
  if (t < 0 || t >= io.max_traj || pd[a.pool].type != POOL_CPU) return true;
  if (tn[t] < 0) {
    i64 need = (i64)a.g * a.r.front();
    int best = -1;
    for (int j = 0; j < (int)pd.size(); ++j) {
      if (pd[j].type != POOL_CPU || pd[j].capacity < need || mf[j] < (i64)io.traj_mem[at]) continue;
      if (best < 0 || mf[j] > mf[best]) best = j;
    }
    if (best < 0) return false;
    tn[t] = best;
    mf[best] -= io.traj_mem[at];
  }
  a.pool = tn[t];
  return true;
}

}  // namespace

// =============================================================== C entry points
extern "C" {

// Whole batched round.  Arrays are host memory, scenario-major with row stride max_actions;
// pools = n_pools x {type, capacity, group, window_us}; gpu_busy has row stride n_nodes
// (may be null); arrival may be null.  Outputs as documented for the product's result.
// service (0xffff: none), restore_us, cache_slots, cache_tag / cache_use ([scenario][node][8][slots],
// updated in place) describe the service cache of the GPU pools (Section 5.3); all may be null / 0.
// side_pool (0xff: none) / side_units, [n_side][scenario][action], are the further entries of the
// actions' cost vectors (Section 4.1, R23-R26); may be null / 0.
int oracle_schedule_batch_ext(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                          int depth, int n_nodes, const int* n_actions, const uint8_t* pool,
                          const uint8_t* unit, const uint32_t* mask, const i64* s, const i64* p,
                          const i64* arrival, const uint8_t* gpu_busy, i64 now,
                          int* alloc_units, int* place_node, int* place_off, i64* act_us,
                          i64* total_act_us, int* n_selected, int* status,
                          const uint16_t* service, const i64* restore, int cache_slots,
                          unsigned* cache_tag, i64* cache_use,
                          int n_side, const uint8_t* side_pool, const uint16_t* side_units) {
  std::vector<PoolDesc> pd(n_pools);
  for (int j = 0; j < n_pools; ++j)
    pd[j] = PoolDesc{pools_flat[4 * j], pools_flat[4 * j + 1], pools_flat[4 * j + 2], pools_flat[4 * j + 3]};
  for (int sc = 0; sc < n_scenarios; ++sc) {
    size_t base = (size_t)sc * max_actions;
    int n = n_actions[sc];
    for (int i = 0; i < max_actions; ++i) {
      alloc_units[base + i] = 0; place_node[base + i] = -1; place_off[base + i] = -1; act_us[base + i] = -1;
    }
    total_act_us[sc] = 0; n_selected[sc] = 0; status[sc] = STATUS_OK;
    std::vector<Action> acts;
    if (!load_actions(acts, n, pd, pool + base, unit + base, mask + base, s + base, p + base,
                      arrival ? arrival + base : nullptr, service ? service + base : nullptr,
                      restore ? restore + base : nullptr, n_side, side_pool ? side_pool + base : nullptr,
                      side_units ? side_units + base : nullptr, (size_t)n_scenarios * max_actions)) {
      status[sc] = STATUS_BAD_ACTION;
      continue;
    }
    const size_t cstride = (size_t)n_nodes * 8 * (cache_slots > 0 ? cache_slots : 0);
    CacheIo cio{cache_slots, cache_tag ? cache_tag + sc * cstride : nullptr, cache_use ? cache_use + sc * cstride : nullptr};
    const CacheIo* cache = (cache_slots > 0 && cache_tag && cache_use) ? &cio : nullptr;
    std::vector<PoolRuntime> pools = fresh_pools(pd, gpu_busy ? gpu_busy + (size_t)sc * n_nodes : nullptr, cache);
    std::vector<int> W(n);
    for (int i = 0; i < n; ++i) W[i] = i;
    std::vector<Running> E;
    std::vector<Grant> grants = schedule_round(pools, acts, W, E, now, depth);
    for (const Grant& g : grants) {
      const Action& a = acts[g.action];
      alloc_units[base + g.action] = g.units;
      place_node[base + g.action] = g.node;
      place_off[base + g.action] = g.off;
      i64 act = (now - a.arrival) + duration(a, g.r);              // Eq. 2: queueing + execution
      if (g.missed) act += a.restore;                              // R22: restoration precedes execution
      act_us[base + g.action] = act;
      total_act_us[sc] = sat_add(total_act_us[sc], act);
      n_selected[sc]++;
    }
    store_cache(pools, cache);
  }
  return 0;
}

int oracle_schedule_batch(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                          int depth, int n_nodes, const int* n_actions, const uint8_t* pool,
                          const uint8_t* unit, const uint32_t* mask, const i64* s, const i64* p,
                          const i64* arrival, const uint8_t* gpu_busy, i64 now,
                          int* alloc_units, int* place_node, int* place_off, i64* act_us,
                          i64* total_act_us, int* n_selected, int* status) {
  return oracle_schedule_batch_ext(n_scenarios, max_actions, n_pools, pools_flat, depth, n_nodes, n_actions, pool,
                                     unit, mask, s, p, arrival, gpu_busy, now, alloc_units, place_node, place_off,
                                     act_us, total_act_us, n_selected, status, nullptr, nullptr, 0, nullptr, nullptr, 0, nullptr, nullptr);
}

// Trace replay: rounds at now = r * round_us, r = 0 .. max_rounds-1.  Each round releases
// what has finished, admits what has arrived, runs the scheduler, starts what it selects.
// occupancy: [scenario][round][pool] units in use after the round's scheduling (zero after
// the scenario has drained); rounds_used: rounds until drained (max_rounds if never).
int oracle_replay_trace_pin(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                        int depth, int n_nodes, i64 round_us, int max_rounds, const int* n_actions,
                        const uint8_t* pool, const uint8_t* unit, const uint32_t* mask,
                        const i64* s, const i64* p, const i64* arrival, const uint8_t* gpu_busy,
                        int* alloc_units, int* place_node, int* place_off, i64* act_us,
                        i64* total_act_us, int* n_selected, int* status, int* occupancy,
                        int* rounds_used,
                        const uint16_t* service, const i64* restore, int cache_slots,
                        unsigned* cache_tag, i64* cache_use,
                        int n_side, const uint8_t* side_pool, const uint16_t* side_units, int policy,
                        const int* trajectory, const uint32_t* traj_mem, const uint8_t* traj_last, int max_traj,
                        int* traj_node, i64* node_mem_free, uint8_t* pool_out) {
  const PinIo pin{trajectory, traj_mem, traj_last, max_traj, traj_node, node_mem_free, pool_out};
  std::vector<PoolDesc> pd(n_pools);
  for (int j = 0; j < n_pools; ++j)
    pd[j] = PoolDesc{pools_flat[4 * j], pools_flat[4 * j + 1], pools_flat[4 * j + 2], pools_flat[4 * j + 3]};
  for (int sc = 0; sc < n_scenarios; ++sc) {
    size_t base = (size_t)sc * max_actions;
    int n = n_actions[sc];
    for (int i = 0; i < max_actions; ++i) {
      alloc_units[base + i] = 0; place_node[base + i] = -1; place_off[base + i] = -1; act_us[base + i] = -1;
    }
    total_act_us[sc] = 0; n_selected[sc] = 0; status[sc] = STATUS_OK; rounds_used[sc] = 0;
    if (pin.trajectory && pin.pool_out) for (int i = 0; i < max_actions; ++i) pin.pool_out[base + i] = pool[base + i];
    if (occupancy)
      std::memset(occupancy + (size_t)sc * max_rounds * n_pools, 0, sizeof(int) * (size_t)max_rounds * n_pools);
    std::vector<Action> acts;
    if (!load_actions(acts, n, pd, pool + base, unit + base, mask + base, s + base, p + base,
                      arrival ? arrival + base : nullptr, service ? service + base : nullptr,
                      restore ? restore + base : nullptr, n_side, side_pool ? side_pool + base : nullptr,
                      side_units ? side_units + base : nullptr, (size_t)n_scenarios * max_actions)) {
      status[sc] = STATUS_BAD_ACTION;
      continue;
    }
    bool sorted = true;
    for (int i = 1; i < n; ++i) sorted &= acts[i - 1].arrival <= acts[i].arrival;
    if (!sorted) { status[sc] = STATUS_UNSORTED; continue; }
    const size_t cstride = (size_t)n_nodes * 8 * (cache_slots > 0 ? cache_slots : 0);
    CacheIo cio{cache_slots, cache_tag ? cache_tag + sc * cstride : nullptr, cache_use ? cache_use + sc * cstride : nullptr};
    const CacheIo* cache = (cache_slots > 0 && cache_tag && cache_use) ? &cio : nullptr;
    std::vector<PoolRuntime> pools = fresh_pools(pd, gpu_busy ? gpu_busy + (size_t)sc * n_nodes : nullptr, cache);
    std::vector<int> W;
    std::vector<Running> E;
    int next = 0, r = 0;
    for (; r < max_rounds; ++r) {
      i64 now = (i64)r * round_us;
      for (PoolRuntime& pr : pools)                                 // R17: quota refill
        if (pr.d.type == POOL_API && pr.d.window_us > 0 && now / pr.d.window_us != pr.window) {
          pr.window = now / pr.d.window_us; pr.api_used = 0;
        }
      for (size_t e = 0; e < E.size();) {                           // release finished actions
        if (E[e].finish > now) { ++e; continue; }
        PoolRuntime& pr = pools[E[e].pool];
        if (pr.d.type == POOL_CPU) { for (int& o : pr.core_owner) if (o == E[e].action) o = -1; }
        else if (pr.d.type == POOL_GPU) {
          for (const Chunk& c : E[e].chunks) pr.node_busy[c.node] &= (uint8_t)~(((1 << c.size) - 1) << c.start);
        } else if (pr.d.window_us == 0) pr.in_use -= E[e].units;
        for (const std::pair<int, int>& c : acts[E[e].action].side)  // R26: held until the action ends
          if (pools[c.first].d.window_us == 0) pools[c.first].in_use -= c.second;
        if (pin.trajectory && pin.traj_last && pin.traj_last[base + E[e].action]) {   // R29: the trajectory is over
          const int t = pin.trajectory[base + E[e].action];
          int* tn = pin.traj_node + (size_t)sc * pin.max_traj;
          if (t >= 0 && t < pin.max_traj && tn[t] >= 0 && pd[acts[E[e].action].pool].type == POOL_CPU) {
            pin.mem_free[(size_t)sc * n_pools + tn[t]] += pin.traj_mem[base + E[e].action];
            tn[t] = -1;
          }
        }
        E.erase(E.begin() + e);
      }
      while (next < n && acts[next].arrival <= now) {               // admit arrivals
        if (pin.trajectory &&
            !pin_on_arrival(pin, pd, acts[next], pin.traj_node + (size_t)sc * pin.max_traj,
                            pin.mem_free + (size_t)sc * n_pools, base + next)) break;   // R29: waits outside the queue
        if (pin.trajectory && pin.pool_out) pin.pool_out[base + next] = (uint8_t)acts[next].pool;
        W.push_back(next++);
      }
      if (policy == 1 || policy == 2)                               // R27: the queue in the policy's order
        std::stable_sort(W.begin(), W.end(), [&](int x, int y) {
          i64 kx = duration(acts[x], acts[x].r.front()), ky = duration(acts[y], acts[y].r.front());
          return policy == 1 ? kx < ky : kx > ky;
        });
      std::vector<Grant> grants = schedule_round(pools, acts, W, E, now, depth);
      for (const Grant& g : grants) {                               // start selected actions
        const Action& a = acts[g.action];
        i64 T = duration(a, g.r);
        if (g.missed) T += a.restore;                               // R22
        E.push_back(Running{now + T, g.action, a.pool, g.units, g.chunks});
        alloc_units[base + g.action] = g.units;
        place_node[base + g.action] = g.node;
        place_off[base + g.action] = g.off;
        i64 act = (now - a.arrival) + T;
        act_us[base + g.action] = act;
        total_act_us[sc] = sat_add(total_act_us[sc], act);
        n_selected[sc]++;
        W.erase(std::find(W.begin(), W.end(), g.action));
      }
      if (occupancy)
        for (int j = 0; j < n_pools; ++j)
          occupancy[((size_t)sc * max_rounds + r) * n_pools + j] = pools[j].busy_units();
      if (next == n && W.empty() && E.empty()) { ++r; break; }
    }
    rounds_used[sc] = r;
    store_cache(pools, cache);
  }
  return 0;
}

int oracle_replay_trace_ext(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                        int depth, int n_nodes, i64 round_us, int max_rounds, const int* n_actions,
                        const uint8_t* pool, const uint8_t* unit, const uint32_t* mask,
                        const i64* s, const i64* p, const i64* arrival, const uint8_t* gpu_busy,
                        int* alloc_units, int* place_node, int* place_off, i64* act_us,
                        i64* total_act_us, int* n_selected, int* status, int* occupancy,
                        int* rounds_used,
                        const uint16_t* service, const i64* restore, int cache_slots,
                        unsigned* cache_tag, i64* cache_use,
                        int n_side, const uint8_t* side_pool, const uint16_t* side_units, int policy) {
  return oracle_replay_trace_pin(n_scenarios, max_actions, n_pools, pools_flat, depth, n_nodes, round_us, max_rounds,
                                 n_actions, pool, unit, mask, s, p, arrival, gpu_busy, alloc_units, place_node,
                                 place_off, act_us, total_act_us, n_selected, status, occupancy, rounds_used,
                                 service, restore, cache_slots, cache_tag, cache_use, n_side, side_pool, side_units,
                                 policy, nullptr, nullptr, nullptr, 0, nullptr, nullptr, nullptr);
}

int oracle_replay_trace(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                        int depth, int n_nodes, i64 round_us, int max_rounds, const int* n_actions,
                        const uint8_t* pool, const uint8_t* unit, const uint32_t* mask,
                        const i64* s, const i64* p, const i64* arrival, const uint8_t* gpu_busy,
                        int* alloc_units, int* place_node, int* place_off, i64* act_us,
                        i64* total_act_us, int* n_selected, int* status, int* occupancy,
                        int* rounds_used) {
  return oracle_replay_trace_ext(n_scenarios, max_actions, n_pools, pools_flat, depth, n_nodes, round_us, max_rounds,
                                   n_actions, pool, unit, mask, s, p, arrival, gpu_busy, alloc_units, place_node,
                                   place_off, act_us, total_act_us, n_selected, status, occupancy, rounds_used,
                                   nullptr, nullptr, 0, nullptr, nullptr, 0, nullptr, nullptr, 0);
}

// R27: permutation that sorts every scenario's queue by the policy's key (1: shortest least-level
// duration first, 2: longest first, 3: earliest arrival first; anything else: queue order), equal keys
// in queue order.  perm[sc][k] = index of the action at position k; positions >= n_actions: k itself.
int oracle_order_queue(int n_scenarios, int max_actions, int n_pools, const int* pools_flat, const int* n_actions,
                       const uint8_t* pool, const uint8_t* unit, const uint32_t* mask, const i64* s, const i64* p,
                       const i64* arrival, int policy, int* perm) {
  std::vector<PoolDesc> pd(n_pools);
  for (int j = 0; j < n_pools; ++j)
    pd[j] = PoolDesc{pools_flat[4 * j], pools_flat[4 * j + 1], pools_flat[4 * j + 2], pools_flat[4 * j + 3]};
  for (int sc = 0; sc < n_scenarios; ++sc) {
    size_t base = (size_t)sc * max_actions;
    int n = n_actions[sc];
    std::vector<i64> key(n, 0);
    for (int i = 0; i < n; ++i) {
      Action a = decode_action(pool[base + i], unit[base + i], mask[base + i], s[base + i], p[base + i],
                               arrival ? arrival[base + i] : 0, pd);
      if (policy == 1 || policy == 2) key[i] = a.valid ? duration(a, a.r.front()) : 0;
      if (policy == 2) key[i] = -key[i];
      if (policy == 3) key[i] = a.arrival;
    }
    std::vector<int> idx(n);
    for (int i = 0; i < n; ++i) idx[i] = i;
    std::stable_sort(idx.begin(), idx.end(), [&](int x, int y) { return key[x] < key[y]; });
    for (int k = 0; k < max_actions; ++k) perm[base + k] = k < n ? idx[k] : k;
  }
  return 0;
}

// One round on the queue sorted by `policy` (R27); results are indexed by the actions' own positions.
int oracle_schedule_batch_ordered(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                                  int depth, int n_nodes, const int* n_actions, const uint8_t* pool,
                                  const uint8_t* unit, const uint32_t* mask, const i64* s, const i64* p,
                                  const i64* arrival, const uint8_t* gpu_busy, i64 now, int policy,
                                  int* alloc_units, int* place_node, int* place_off, i64* act_us,
                                  i64* total_act_us, int* n_selected, int* status) {
  std::vector<PoolDesc> pd(n_pools);
  for (int j = 0; j < n_pools; ++j)
    pd[j] = PoolDesc{pools_flat[4 * j], pools_flat[4 * j + 1], pools_flat[4 * j + 2], pools_flat[4 * j + 3]};
  std::vector<int> perm((size_t)n_scenarios * max_actions);
  oracle_order_queue(n_scenarios, max_actions, n_pools, pools_flat, n_actions, pool, unit, mask, s, p, arrival,
                     policy, perm.data());
  for (int sc = 0; sc < n_scenarios; ++sc) {
    size_t base = (size_t)sc * max_actions;
    int n = n_actions[sc];
    for (int i = 0; i < max_actions; ++i) {
      alloc_units[base + i] = 0; place_node[base + i] = -1; place_off[base + i] = -1; act_us[base + i] = -1;
    }
    total_act_us[sc] = 0; n_selected[sc] = 0; status[sc] = STATUS_OK;
    std::vector<Action> acts;
    if (!load_actions(acts, n, pd, pool + base, unit + base, mask + base, s + base, p + base,
                      arrival ? arrival + base : nullptr)) {
      status[sc] = STATUS_BAD_ACTION;
      continue;
    }
    std::vector<PoolRuntime> pools = fresh_pools(pd, gpu_busy ? gpu_busy + (size_t)sc * n_nodes : nullptr);
    std::vector<int> W(perm.begin() + base, perm.begin() + base + n);
    std::vector<Running> E;
    std::vector<Grant> grants = schedule_round(pools, acts, W, E, now, depth);
    for (const Grant& g : grants) {
      const Action& a = acts[g.action];
      alloc_units[base + g.action] = g.units;
      place_node[base + g.action] = g.node;
      place_off[base + g.action] = g.off;
      i64 act = (now - a.arrival) + duration(a, g.r);
      act_us[base + g.action] = act;
      total_act_us[sc] = sat_add(total_act_us[sc], act);
      n_selected[sc]++;
    }
  }
  return 0;
}

// R28: pins the trajectories of every scenario's queue to CPU nodes (= CPU pools).  trajectory: per
// action, -1 = not tied to a trajectory (the action keeps its pool); traj_mem: memory of the whole
// trajectory, read at the action that pins it.  traj_node [scenario][max_traj] (-1: not pinned) and
// node_mem_free [scenario][pool] (entries of CPU pools) are state, in and out.  pool_out gets the
// pool column with every trajectory action moved to its node; n_admitted the length of the queue
// up to the first action whose trajectory found no node.
int oracle_pin_trajectories(int n_scenarios, int max_actions, int n_pools, const int* pools_flat,
                            const int* n_actions, const uint8_t* pool, const uint8_t* unit, const uint32_t* mask,
                            const int* trajectory, const uint32_t* traj_mem, int max_traj,
                            int* traj_node, i64* node_mem_free, uint8_t* pool_out, int* n_admitted) {
  std::vector<PoolDesc> pd(n_pools);
  for (int j = 0; j < n_pools; ++j)
    pd[j] = PoolDesc{pools_flat[4 * j], pools_flat[4 * j + 1], pools_flat[4 * j + 2], pools_flat[4 * j + 3]};
  for (int sc = 0; sc < n_scenarios; ++sc) {
    size_t base = (size_t)sc * max_actions;
    int* tn = traj_node + (size_t)sc * max_traj;
    i64* mf = node_mem_free + (size_t)sc * n_pools;
    int n = n_actions[sc], adm = n;
    for (int i = 0; i < max_actions; ++i) pool_out[base + i] = pool[base + i];
    for (int i = 0; i < n; ++i) {
      int t = trajectory[base + i];
      if (t < 0 || t >= max_traj) continue;
      if (pool[base + i] >= n_pools || pd[pool[base + i]].type != POOL_CPU) continue;   // not an action of the CPU manager
      if (tn[t] < 0) {
        // least level of the action in cores: g times its smallest multiplicity
        int g = unit[base + i] & 0x7F, rmin = 0;
        for (int r = 1; r <= 32 && !rmin; ++r) if (mask[base + i] >> (r - 1) & 1u) rmin = r;
        i64 need = (i64)g * rmin;
        int best = -1;
        for (int j = 0; j < n_pools; ++j) {
          if (pd[j].type != POOL_CPU || pd[j].capacity < need || mf[j] < (i64)traj_mem[base + i]) continue;
          if (best < 0 || mf[j] > mf[best]) best = j;
        }
        if (best < 0) { adm = i; break; }
        tn[t] = best;
        mf[best] -= traj_mem[base + i];
      }
      pool_out[base + i] = (uint8_t)tn[t];
    }
    n_admitted[sc] = adm;
  }
  return 0;
}

// ---- single pieces, exported so that tests can pin each of them on its own ----------

i64 oracle_duration(i64 s, i64 p, int r) {
  Action a; a.s = clamp_param(s); a.p = clamp_param(p);
  return duration(a, r);
}

// maximal free aligned blocks of a set of node masks: F[l] = blocks of size 2^l
void oracle_free_blocks(int n_nodes, const uint8_t* busy, int group, int* F) {
  std::vector<uint8_t> nb(busy, busy + n_nodes);
  free_block_counts(nb, group, F);
}

int oracle_chunks_fit(const int* n, const int* F) { return chunks_fit(n, F) ? 1 : 0; }

i64 oracle_encode(const int* n, const int* N) { return encode(n, N); }
void oracle_decode(i64 j, const int* N, int* n) { decode(j, N, n); }

// DPArrange on one pool: m tasks (unit byte, mask, s, p), pool descriptor, node masks for a
// GPU pool (else free units).  Writes, for every prefix q = 1..m, value[q-1] and the
// allocation in units alloc[(q-1)*m + i]; returns 0, or q if prefix q does not fit.
// prune = 0 keeps every valid DP state (slow; only to check that pruning changes nothing).
int oracle_dp_arrange(int m, const uint8_t* unit, const uint32_t* mask, const i64* s, const i64* p,
                      int type, int capacity, int group, int free_units, int n_nodes,
                      const uint8_t* busy, int prune, i64* value, int* alloc) {
  std::vector<PoolDesc> pd(1, PoolDesc{type, capacity, group, 0});
  std::vector<Action> acts(m);
  for (int i = 0; i < m; ++i) {
    acts[i] = decode_action(0, unit[i], mask[i], s[i], p[i], 0, pd);
    if (!acts[i].valid) return -1;
  }
  PoolRoom room;
  room.gpu = type == POOL_GPU; room.free_units = free_units;
  room.F[0] = room.F[1] = room.F[2] = room.F[3] = 0;
  if (room.gpu) {
    std::vector<uint8_t> nb(busy, busy + n_nodes);
    free_block_counts(nb, group, room.F);
  }
  for (int q = 1; q <= m; ++q) {
    std::vector<const Action*> C;
    for (int i = 0; i < q; ++i) C.push_back(&acts[i]);
    std::vector<int> a;
    if (!dp_arrange(C, room, prune != 0, &value[q - 1], &a)) return q;
    for (int i = 0; i < q; ++i) alloc[(size_t)(q - 1) * m + i] = acts[i].g * a[i];
  }
  return 0;
}

// estimate() of Algorithm 2 on an explicit heap and remaining list
i64 oracle_estimate(int n_heap, const i64* heap, int n_rest, const uint8_t* unit, const uint32_t* mask,
                    const i64* s, const i64* p, int depth) {
  std::vector<PoolDesc> pd(1, PoolDesc{POOL_CPU, 1 << 30, 1, 0});
  std::vector<Action> acts(n_rest);
  std::vector<const Action*> rest;
  for (int i = 0; i < n_rest; ++i) acts[i] = decode_action(0, unit[i], mask[i], s[i], p[i], 0, pd);
  for (int i = 0; i < n_rest; ++i) rest.push_back(&acts[i]);
  return estimate(std::vector<i64>(heap, heap + n_heap), rest, depth);
}

// Section 5.3 allocation of one request of m GPUs on explicit node masks (updated in place):
// rounds m up to a power of two, takes the smallest sufficient free block.  Returns 0 and
// (node, start, size), or -1 if nothing fits.
int oracle_chunk_alloc(int n_nodes, uint8_t* busy, int group, int m, int* node, int* start, int* size) {
  PoolRuntime pr;
  pr.d = PoolDesc{POOL_GPU, n_nodes * group, group, 0};
  pr.node_busy.assign(busy, busy + n_nodes);
  int sz = 1;
  while (sz < m) sz *= 2;
  std::vector<Action> acts(1);
  acts[0].g = sz; acts[0].gang = true; acts[0].r.push_back(1);
  std::vector<Grant> grants(1);
  grants[0].action = 0; grants[0].r = 1; grants[0].units = sz; grants[0].node = -1; grants[0].off = -1;
  place_gpu(pr, acts, grants, std::vector<int>(1, 0));
  if (grants[0].node < 0) return -1;
  *node = grants[0].node; *start = grants[0].off; *size = sz;
  for (int v = 0; v < n_nodes; ++v) busy[v] = pr.node_busy[v];
  return 0;
}

}  // extern "C"
