// Host side of libloki_alloc: argument checks, the planner that lays out the
// device tables and proves the arithmetic ranges, and the C-ABI entry points.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "loki_internal.h"

using namespace loki;

namespace {

typedef unsigned __int128 u128;

constexpr int64_t kMaxLatencyUs = 1LL << 40;
constexpr int64_t kMaxSloUs = 1LL << 60;
constexpr int64_t kMaxCommUs = 1LL << 50;
constexpr int kMaxSweepSlos = 64;     // SLOs per loki_alloc_solve_slos call
constexpr int64_t kMaxBatch = 1LL << 24;
constexpr int64_t kMaxCandidates = 1LL << 40;
constexpr int64_t kMaxOptionsTotal = 1LL << 21;
constexpr int64_t kMaxClassTuples = 1LL << 22;
constexpr int kMaxDevices = 64;

// Host view of a validated problem.
struct HostProblem {
  int T = 0;
  int nB = 0;
  int parent[kMaxTasks];
  int32_t fanout[kMaxTasks];
  int V[kMaxTasks];
  int voff[kMaxTasks];
  std::vector<int64_t> batch;
  std::vector<double> acc;
  std::vector<int64_t> lat;
  std::vector<int64_t> vfan;    // per-variant multiplicative factor in thousandths
  bool variant_fanout = false;  // some factor differs from 1000
  int64_t slo = 0, comm = 0, max_demand = 0;
  int32_t S = 0;
  int split = 0;
  int max_levels = 0;
  int64_t nS[kMaxTasks], O[kMaxTasks], stride[kMaxTasks];
  int64_t N = 0;
  int depth[kMaxTasks];
  int n_leaves = 0;
  int leaf_task[kMaxTasks];
  uint32_t path_mask[kMaxTasks];
  int64_t lat_limit[kMaxTasks];
  int64_t dem_max[kMaxTasks];   // largest stage demand under max_demand
};

// Halved-SLO latency limit of every leaf path: 2 * sum lat <= slo - hops * comm.
void set_leaf_limits(HostProblem& p) {
  for (int k = 0; k < p.n_leaves; ++k) {
    const int64_t budget = p.slo - (int64_t)p.depth[p.leaf_task[k]] * p.comm;
    p.lat_limit[k] = budget < 0 ? -1 : budget / 2;
  }
}

int validate_into(const loki_alloc_desc_t* d, HostProblem* hp) {
  if (d == nullptr) return LOKI_ERR_INVALID_ARG;
  if (d->n_tasks < 1 || d->n_tasks > kMaxTasks) return LOKI_ERR_INVALID_ARG;
  if (!d->parent || !d->fanout_milli || !d->n_variants || !d->batch_sizes || !d->accuracy ||
      !d->latency_us)
    return LOKI_ERR_INVALID_ARG;
  if (d->n_batches < 1 || d->n_batches > 255) return LOKI_ERR_INVALID_ARG;
  if (d->slo_us < 0 || d->slo_us > kMaxSloUs) return LOKI_ERR_INVALID_ARG;
  if (d->comm_us < 0 || d->comm_us > kMaxCommUs) return LOKI_ERR_INVALID_ARG;
  if (d->cluster_size < 0 || d->cluster_size >= (1 << 24)) return LOKI_ERR_INVALID_ARG;
  if (d->split_mode != 0 && d->split_mode != 1) return LOKI_ERR_INVALID_ARG;
  if (d->max_demand_mqps < 0) return LOKI_ERR_INVALID_ARG;
  if (d->max_levels < 1) return LOKI_ERR_INVALID_ARG;
  HostProblem& p = *hp;
  p.T = d->n_tasks;
  p.nB = d->n_batches;
  int sumV = 0;
  for (int i = 0; i < p.T; ++i) {
    if (d->n_variants[i] < 1 || d->n_variants[i] > (1 << 20)) return LOKI_ERR_INVALID_ARG;
    p.V[i] = d->n_variants[i];
    p.voff[i] = sumV;
    sumV += p.V[i];
    if (i > 0 && d->fanout_milli[i] < 1) return LOKI_ERR_INVALID_ARG;
    p.fanout[i] = i == 0 ? 1000 : d->fanout_milli[i];
  }
  // rooted tree in topological order: one root, every other task has an earlier parent
  if (d->parent[0] != -1) return LOKI_ERR_INVALID_GRAPH;
  p.parent[0] = -1;
  for (int i = 1; i < p.T; ++i) {
    if (d->parent[i] < 0 || d->parent[i] >= i) return LOKI_ERR_INVALID_GRAPH;
    p.parent[i] = d->parent[i];
  }
  for (int b = 0; b < p.nB; ++b) {
    if (d->batch_sizes[b] < 1 || d->batch_sizes[b] > kMaxBatch) return LOKI_ERR_INVALID_ARG;
    if (b > 0 && d->batch_sizes[b] <= d->batch_sizes[b - 1]) return LOKI_ERR_INVALID_ARG;
  }
  p.batch.assign(d->batch_sizes, d->batch_sizes + p.nB);
  for (int v = 0; v < sumV; ++v) {
    const double a = d->accuracy[v];
    if (!(a > 0.0) || !(a <= 1.0) || !std::isfinite(a)) return LOKI_ERR_INVALID_ARG;
    for (int b = 0; b < p.nB; ++b) {
      const int64_t l = d->latency_us[(size_t)v * p.nB + b];
      if (l < 1 || l > kMaxLatencyUs) return LOKI_ERR_INVALID_ARG;
    }
  }
  p.acc.assign(d->accuracy, d->accuracy + sumV);
  p.lat.assign(d->latency_us, d->latency_us + (size_t)sumV * p.nB);
  p.vfan.assign((size_t)sumV, 1000);
  p.variant_fanout = false;
  if (d->variant_fanout_milli != nullptr)
    for (int v = 0; v < sumV; ++v) {
      const int32_t f = d->variant_fanout_milli[v];
      if (f < 1 || f > (1 << 20)) return LOKI_ERR_INVALID_ARG;
      p.vfan[(size_t)v] = f;
      if (f != 1000) p.variant_fanout = true;
    }
  p.slo = d->slo_us;
  p.comm = d->comm_us;
  p.S = d->cluster_size;
  p.split = d->split_mode;
  p.max_demand = d->max_demand_mqps;
  p.max_levels = d->max_levels;

  // size of the search space
  u128 N = 1;
  int64_t total_opts = 0;
  for (int i = 0; i < p.T; ++i) {
    p.nS[i] = (int64_t)p.V[i] * p.nB;
    u128 Oi = (u128)p.nS[i];
    if (p.split) Oi += (u128)p.nS[i] * (u128)(p.nS[i] - 1) / 2 * 15;
    if (Oi > (u128)kMaxOptionsTotal) return LOKI_ERR_RANGE;
    p.O[i] = (int64_t)Oi;
    p.stride[i] = (int64_t)N;
    N *= Oi;
    if (N >= (u128)kMaxCandidates) return LOKI_ERR_RANGE;
    total_opts += p.O[i];
    if (total_opts > kMaxOptionsTotal) return LOKI_ERR_RANGE;
  }
  p.N = (int64_t)N;

  // tree facts: depth, leaves, path masks, halved-SLO limits per leaf
  bool is_leaf[kMaxTasks];
  uint32_t mask[kMaxTasks];
  for (int i = 0; i < p.T; ++i) {
    is_leaf[i] = true;
    p.depth[i] = i == 0 ? 1 : p.depth[p.parent[i]] + 1;
    mask[i] = (i == 0 ? 0u : mask[p.parent[i]]) | (1u << i);
  }
  for (int i = 1; i < p.T; ++i) is_leaf[p.parent[i]] = false;
  p.n_leaves = 0;
  for (int i = 0; i < p.T; ++i) {
    if (!is_leaf[i]) continue;
    const int k = p.n_leaves++;
    p.leaf_task[k] = i;
    p.path_mask[k] = mask[i];
  }
  set_leaf_limits(p);

  // overflow proof: every stage demand and every product dem * share * lat fits in int64
  int64_t max_lat = 0;
  for (int64_t l : p.lat) max_lat = std::max(max_lat, l);
  const u128 lim = (u128)1 << 62;
  p.dem_max[0] = p.max_demand;
  for (int i = 1; i < p.T; ++i) {
    const int u = p.parent[i];
    int64_t vmax = 1000;      // largest factor among the parent's variants
    for (int v = 0; v < p.V[u]; ++v) vmax = std::max(vmax, p.vfan[(size_t)(p.voff[u] + v)]);
    if (!p.variant_fanout) {
      const u128 prod = (u128)p.dem_max[u] * (u128)p.fanout[i];
      if (prod + 999 >= lim) return LOKI_ERR_RANGE;
      p.dem_max[i] = (int64_t)((prod + 999) / 1000);
    } else {
      // the kernels form demand x edge factor x (16 x variant factor) in 64 bits
      const u128 prod = (u128)p.dem_max[u] * (u128)p.fanout[i] * (u128)(16 * vmax);
      if (prod + 16000000 >= lim) return LOKI_ERR_RANGE;
      p.dem_max[i] = (int64_t)((prod + 15999999) / 16000000);
    }
  }
  for (int i = 0; i < p.T; ++i) {
    const u128 prod = (u128)p.dem_max[i] * (u128)(p.split ? 15 : 1) * (u128)max_lat;
    const u128 den = (u128)(p.split ? 16 : 1) * (u128)p.batch.back() * 1000000000ull;
    if (prod + den >= lim) return LOKI_ERR_RANGE;
  }
  return LOKI_OK;
}

// Largest double strictly below p / q (p < q): r = M * 2^-s with 2^52 <= M + 1 and
// M < 2^53.  *s_out is the scale s; p / q - r is in (0, 2^-s].
bool recip_below(uint64_t p, uint64_t q, double* out, int* s_out, bool allow_ge_one = false) {
  if (p == 0 || q == 0 || (p >= q && !allow_ge_one)) return false;
  if ((u128)p / q >= ((u128)1 << 52)) return false;
  u128 r = (u128)p % q;
  uint64_t M = (uint64_t)(p / q);     // integer part first (0 for a ratio below 1)
  int s = 0;
  while (M < (1ull << 52)) {
    r <<= 1;
    const int bit = r >= (u128)q ? 1 : 0;
    if (bit) r -= q;
    M = (M << 1) | (uint64_t)bit;
    if (++s > 200) return false;
  }
  if (r == 0) M -= 1;       // p / q is itself a 53-bit number: step one unit down
  *out = std::ldexp((double)M, -s);
  *s_out = s;
  return true;
}

uint64_t gcd_u64(uint64_t a, uint64_t b) {
  while (b) { const uint64_t t = a % b; a = b; b = t; }
  return a;
}

struct DirectPlan {
  bool ok = false;
  int jbits = 0;
  int n_parts_max = 1;
  int64_t dem_cap[kMaxTasks];
  int n_class[kMaxTasks];
  int class_off[kMaxTasks];
  std::vector<int32_t> class_first, class_count;
  std::vector<double> class_acc;
  std::vector<DirRec> members;
  int64_t member_off[kMaxTasks];
  std::vector<uint64_t> iter_prefix;
  std::vector<int32_t> class_min_lat;       // smallest member latency per class
  std::vector<unsigned char> uni_members;   // level-lane member records (kUniRecBytes1 / 2 each)
  std::vector<int32_t> lat_order;           // per class, its members' in-class indices by ascending latency
  std::vector<int32_t> join_order;          // DirProblem::join_order (empty: not tabulated)
  int32_t join_stride = 0;
  bool uniform_ok = false;                  // the largest class tuple's records fit the shared-memory stage
  int uni_stage_bytes = 0;
  int uni_max_members = 0;                  // sum over tasks of the largest class
  bool variant = false;                     // per-variant factors: only the generic and the variant kernel apply
  bool rootfirst = false;                   // the level-lane path is served by the root-first kernel
  bool tables_ok = false;                   // hoisted kernel: the largest class tuple's records fit its bound
  std::vector<double> uni_dem_r;            // [member][T]: demand ratio into child task i under the member's option
  int64_t n_ct = 0, total_iters = 0;
  int32_t lat_limit[kMaxTasks];
};

// Host image of the tables shared by all class tuples (PrefixTables): the rows and their groups.
constexpr int64_t kPrefixMaxTableBytes = 256LL << 20;
// Sweeps below this many (candidate, level) pairs keep the tables a block builds per class tuple:
// the shared tables cost one more launch (measured: C2's 2.8e7 pairs 0.032 ms against 0.023, C4's
// 1.6e9 pairs the same either way, C5's 1.8e10 pairs 1.04 ms against 4.73).
constexpr double kPrefixSharedMinPairs = 268435456.0;

struct PrefixHost {
  std::vector<int4> row_desc;
  std::vector<int32_t> row_lat;
  std::vector<uint32_t> row_digit;
  std::vector<int32_t> class_rows;
  std::vector<int32_t> pair_rows;
  std::vector<int2> groups;
  int n_outer = 0;
  bool joined = false;
};

// Lays the rows out: per class of every outer task its members in ascending latency; then the inner
// groups, a class of task 0, or (joined) a pair of classes of tasks 0 and 1 with the member pairs in
// the tabulated order of their joint latency.  An inner entry carries its rank (task 0's digit has
// weight 1, task 1's the size of task 0's class); an outer entry gets its rank from the walk.
void plan_prefix_tables(const HostProblem& p, const DirectPlan& pl, PrefixHost* out) {
  const bool joined = p.n_leaves == 1 && p.T >= 3 && !pl.join_order.empty();
  const int imin = joined ? 2 : 1;
  int n_classes = 0;
  for (int i = 0; i < p.T; ++i) n_classes += pl.n_class[i];
  out->joined = joined;
  out->class_rows.assign((size_t)n_classes, -1);
  const auto first_of = [&](int task, int cls) {
    return (size_t)pl.member_off[task] + (size_t)pl.class_first[(size_t)(pl.class_off[task] + cls)];
  };
  const auto add_class = [&](int task, int cls, bool inner) {
    const size_t first = first_of(task, cls);
    const int n = pl.class_count[(size_t)(pl.class_off[task] + cls)];
    out->class_rows[(size_t)(pl.class_off[task] + cls)] = (int32_t)out->row_desc.size();
    if (inner) out->groups.push_back(int2{(int)out->row_desc.size(), n});
    for (int k = 0; k < n; ++k) {
      const int32_t m = pl.lat_order[first + (size_t)k];
      out->row_desc.push_back(int4{(int)(first + (size_t)m), -1, inner ? m : 0, task});
      out->row_lat.push_back(pl.members[first + (size_t)m].lat);
      out->row_digit.push_back((uint32_t)m);
    }
  };
  for (int i = imin; i < p.T; ++i)
    for (int c = 0; c < pl.n_class[i]; ++c) add_class(i, c, false);
  out->n_outer = (int)out->row_desc.size();
  if (!joined) {
    for (int c = 0; c < pl.n_class[0]; ++c) add_class(0, c, true);
    return;
  }
  out->pair_rows.assign((size_t)pl.n_class[0] * (size_t)pl.n_class[1], -1);
  for (int c1 = 0; c1 < pl.n_class[1]; ++c1)
    for (int c0 = 0; c0 < pl.n_class[0]; ++c0) {
      const size_t f0 = first_of(0, c0), f1 = first_of(1, c1);
      const int n0 = pl.class_count[(size_t)(pl.class_off[0] + c0)], n1 = pl.class_count[(size_t)(pl.class_off[1] + c1)];
      const int32_t* ord = pl.join_order.data() + ((size_t)c1 * (size_t)pl.n_class[0] + (size_t)c0) * (size_t)pl.join_stride;
      out->pair_rows[(size_t)c1 * (size_t)pl.n_class[0] + (size_t)c0] = (int32_t)out->row_desc.size();
      out->groups.push_back(int2{(int)out->row_desc.size(), n0 * n1});
      for (int r = 0; r < n0 * n1; ++r) {
        const int q = ord[r];
        const int32_t m0 = pl.lat_order[f0 + (size_t)(q % n0)], m1 = pl.lat_order[f1 + (size_t)(q / n0)];
        out->row_desc.push_back(int4{(int)(f0 + (size_t)m0), (int)(f1 + (size_t)m1), m0 + m1 * n0, 0 | (1 << 8)});
        out->row_lat.push_back(pl.members[f0 + (size_t)m0].lat + pl.members[f1 + (size_t)m1].lat);
        out->row_digit.push_back(0u);
      }
    }
}

// Option tables in index order.  The task accuracy written here is recomputed on
// the device by loki_alloc_create; the host value serves the host-only self-check.
void build_options(const HostProblem& p, std::vector<OptRec>& opts, int64_t opt_off[kMaxTasks]) {
  opts.clear();
  for (int i = 0; i < p.T; ++i) {
    opt_off[i] = (int64_t)opts.size();
    const int64_t nS = p.nS[i];
    auto single = [&](int64_t o, int* v, int* bi) { *v = (int)(o / p.nB); *bi = (int)(o % p.nB); };
    for (int64_t o = 0; o < nS; ++o) {
      int v, bi;
      single(o, &v, &bi);
      OptRec r;
      std::memset(&r, 0, sizeof(r));
      r.acc = p.acc[p.voff[i] + v];
      r.lat = p.lat[(size_t)(p.voff[i] + v) * p.nB + bi];
      r.mult[0] = r.lat;
      r.den[0] = p.batch[bi] * 1000000000LL;
      r.mult[1] = 0;
      r.den[1] = 1;
      r.variant[0] = v;
      r.variant[1] = -1;
      r.batch_idx[0] = (uint8_t)bi;
      r.k = 16;
      r.parts = 1;
      r.vf16 = (uint32_t)(16 * p.vfan[(size_t)(p.voff[i] + v)]);
      opts.push_back(r);
    }
    if (!p.split) continue;
    for (int64_t o1 = 0; o1 < nS; ++o1)
      for (int64_t o2 = o1 + 1; o2 < nS; ++o2)
        for (int k = 1; k <= 15; ++k) {
          int v1, b1, v2, b2;
          single(o1, &v1, &b1);
          single(o2, &v2, &b2);
          const double A1 = p.acc[p.voff[i] + v1], A2 = p.acc[p.voff[i] + v2];
          const int64_t l1 = p.lat[(size_t)(p.voff[i] + v1) * p.nB + b1];
          const int64_t l2 = p.lat[(size_t)(p.voff[i] + v2) * p.nB + b2];
          OptRec r;
          std::memset(&r, 0, sizeof(r));
          const double share = (double)k * 0.0625;
          const double diff = A1 - A2;
          const double prod = share * diff;
          r.acc = A2 + prod;
          r.lat = std::max(l1, l2);
          r.mult[0] = (int64_t)k * l1;
          r.den[0] = 16 * p.batch[b1] * 1000000000LL;
          r.mult[1] = (int64_t)(16 - k) * l2;
          r.den[1] = 16 * p.batch[b2] * 1000000000LL;
          r.variant[0] = v1;
          r.variant[1] = v2;
          r.batch_idx[0] = (uint8_t)b1;
          r.batch_idx[1] = (uint8_t)b2;
          r.k = (uint8_t)k;
          r.parts = 2;
          r.vf16 = (uint32_t)(k * p.vfan[(size_t)(p.voff[i] + v1)] + (16 - k) * p.vfan[(size_t)(p.voff[i] + v2)]);
          opts.push_back(r);
        }
  }
}

// Decide whether the direct kernel's fixed-point arithmetic is exact for this
// problem and lay out its tables.
void plan_direct(const HostProblem& p, const std::vector<OptRec>& opts,
                 const int64_t opt_off[kMaxTasks], DirectPlan* dp) {
  dp->ok = false;
  if (!direct_supported(p.T, p.split)) return;
  dp->variant = p.variant_fanout;   // stage demands depend on the candidate: root-first level-lane kernel only
  dp->n_parts_max = p.split ? 2 : 1;
  // latencies must fit the 32-bit path sums
  int64_t lat_sum = 0;
  for (int i = 0; i < p.T; ++i) {
    int64_t m = 0;
    for (int64_t o = 0; o < p.O[i]; ++o) m = std::max(m, opts[(size_t)(opt_off[i] + o)].lat);
    lat_sum += m;
  }
  if (lat_sum >= (1LL << 31)) return;
  for (int k = 0; k < p.n_leaves; ++k)
    dp->lat_limit[k] = (int32_t)std::min<int64_t>(p.lat_limit[k], (1LL << 31) - 1);

  u128 w_max = 0;   // bound on the worker sum of any candidate under the clamped demand
  for (int i = 0; i < p.T; ++i) {
    // demand cap: from here on every part of every option needs more than S workers
    u128 cap = 0;
    uint64_t pmax = 0, qmax = 1;   // largest ratio p/q over the parts of this task
    for (int64_t o = 0; o < p.O[i]; ++o) {
      const OptRec& r = opts[(size_t)(opt_off[i] + o)];
      for (int s = 0; s < r.parts; ++s) {
        const uint64_t pp = (uint64_t)r.mult[s], qq = (uint64_t)r.den[s];
        const u128 c = (u128)(uint32_t)p.S * qq / pp + 1;
        if (c > cap) cap = c;
        if ((u128)pp * qmax > (u128)pmax * qq) { pmax = pp; qmax = qq; }
      }
    }
    const u128 lim = std::min<u128>(cap, (u128)p.dem_max[i]);
    if (lim >= ((u128)1 << 53)) return;        // stage demand must be exact as a double
    dp->dem_cap[i] = (int64_t)lim;
    if (pmax >= qmax) return;                  // ratio >= 1: not a sensible profile
    // exactness of every part, and the per-task worker bound
    u128 task_w = 0;
    for (int64_t o = 0; o < p.O[i]; ++o) {
      const OptRec& r = opts[(size_t)(opt_off[i] + o)];
      u128 w = 0;
      for (int sidx = 0; sidx < r.parts; ++sidx) {
        const uint64_t pp = (uint64_t)r.mult[sidx], qq = (uint64_t)r.den[sidx];
        const uint64_t g = gcd_u64(pp, qq);
        const u128 qred = qq / g;
        double rd;
        int sc;
        if (!recip_below(pp, qq, &rd, &sc)) return;
        // dem * (p/q - r) <= dem * 2^-s must stay below 1/q:  dem_max * q < 2^s
        if (sc < 126 && lim * qred >= ((u128)1 << sc)) return;
        w += 1 + lim * pp / qq;
      }
      if (w > task_w) task_w = w;
    }
    w_max += task_w;
  }
  if (w_max < (u128)p.S + 1) w_max = (u128)p.S + 1;

  // accuracy classes: options of a task with bit-identical task accuracy
  dp->class_first.clear(); dp->class_count.clear(); dp->class_acc.clear(); dp->members.clear();
  dp->class_min_lat.clear();
  u128 n_ct = 1;
  u128 jmax = 1;
  int64_t max_count = 1;
  for (int i = 0; i < p.T; ++i) {
    std::vector<int64_t> order((size_t)p.O[i]);
    for (int64_t o = 0; o < p.O[i]; ++o) order[(size_t)o] = o;
    auto bits = [&](int64_t o) {
      uint64_t b;
      std::memcpy(&b, &opts[(size_t)(opt_off[i] + o)].acc, 8);
      return b;
    };
    std::stable_sort(order.begin(), order.end(),
                     [&](int64_t a, int64_t b) { return bits(a) < bits(b); });
    dp->class_off[i] = (int)dp->class_first.size();
    dp->member_off[i] = (int64_t)dp->members.size();
    int n_class = 0;
    int64_t biggest = 0;
    for (size_t k = 0; k < order.size(); ++k) {
      const int64_t o = order[k];
      const OptRec& r = opts[(size_t)(opt_off[i] + o)];
      if (k == 0 || bits(o) != bits(order[k - 1])) {
        dp->class_first.push_back((int32_t)(dp->members.size() - (size_t)dp->member_off[i]));
        dp->class_count.push_back(0);
        dp->class_acc.push_back(r.acc);
        dp->class_min_lat.push_back((int32_t)r.lat);
        ++n_class;
      }
      ++dp->class_count.back();
      dp->class_min_lat.back() = std::min<int32_t>(dp->class_min_lat.back(), (int32_t)r.lat);
      biggest = std::max<int64_t>(biggest, dp->class_count.back());
      DirRec m;
      std::memset(&m, 0, sizeof(m));
      for (int sidx = 0; sidx < r.parts; ++sidx) {
        int sc;
        if (!recip_below((uint64_t)r.mult[sidx], (uint64_t)r.den[sidx], &m.r[sidx], &sc)) return;
      }
      m.lat = (int32_t)r.lat;
      m.n_real = r.parts;
      m.opt = (int32_t)o;
      dp->members.push_back(m);
    }
    dp->n_class[i] = n_class;
    n_ct *= (u128)n_class;
    jmax *= (u128)biggest;
    if (n_ct > (u128)kMaxClassTuples || jmax > ((u128)1 << 31)) return;
    max_count = std::max<int64_t>(max_count, biggest);
  }
  // the kernel splits a rank into member digits with a 32-bit reciprocal multiply,
  // exact while rank * count < 2^32
  const uint64_t iter_cands = (uint64_t)kDirectBatch;
  if ((jmax + (u128)iter_cands) * (u128)max_count >= ((u128)1 << 32)) return;
  int jbits = 1;
  while (((u128)1 << jbits) < jmax) ++jbits;
  // packed key (workers << jbits | rank) must stay below the "empty" pattern
  if (((w_max + 1) << jbits) >= (u128)0xFFFFFFFFu) return;
  dp->jbits = jbits;
  dp->n_ct = (int64_t)n_ct;

  // work items of the direct kernel per class tuple: batches of 32 columns, a column being a choice of
  // members for tasks 1 .. T-1 (with one task: a single item); class tuple index mixed-radix over the
  // class counts with task 0 least significant
  dp->iter_prefix.assign((size_t)dp->n_ct + 1, 0);
  std::vector<int> cls((size_t)p.T, 0);
  uint64_t run = 0, cands = 0;
  for (int64_t ct = 0; ct < dp->n_ct; ++ct) {
    dp->iter_prefix[(size_t)ct] = run;
    uint64_t J = 1, cols = 1;
    for (int i = 0; i < p.T; ++i) {
      const uint64_t c = (uint64_t)dp->class_count[(size_t)(dp->class_off[i] + cls[(size_t)i])];
      J *= c;
      if (i > 0) cols *= c;
    }
    run += p.T == 1 ? 1 : (cols + iter_cands - 1) / iter_cands;
    cands += J;
    for (int i = 0; i < p.T; ++i) {
      if (++cls[(size_t)i] < dp->n_class[i]) break;
      cls[(size_t)i] = 0;
    }
  }
  dp->iter_prefix[(size_t)dp->n_ct] = run;
  dp->total_iters = (int64_t)run;
  if (cands != (uint64_t)p.N) return;      // the class tuples partition the candidates
  if (run >= (1ull << 32)) return;         // the direct kernel counts batches in 32 bits
  // member records of the level-lane kernel, in the order of `members`:
  // r[parts] (double), task latency (int32), n_real << jbits (uint32), padding to 16 / 32 bytes
  {
    const size_t rec = dp->n_parts_max == 2 ? (size_t)kUniRecBytes2 : (size_t)kUniRecBytes1;
    dp->uni_members.assign(dp->members.size() * rec, 0);
    for (size_t m = 0; m < dp->members.size(); ++m) {
      unsigned char* q = dp->uni_members.data() + m * rec;
      const DirRec& src = dp->members[m];
      const uint32_t nsh = (uint32_t)src.n_real << jbits;
      std::memcpy(q, src.r, 8 * (size_t)dp->n_parts_max);
      std::memcpy(q + 8 * (size_t)dp->n_parts_max, &src.lat, 4);
      std::memcpy(q + 8 * (size_t)dp->n_parts_max + 4, &nsh, 4);
    }
    // per member and child task: the largest double r below
    //   fanout_milli[child] x (16 x option factor in thousandths) / 16e6,
    // so that the child's stage demand ceil(dem * ratio) is 1 + floor(dem * r) in one fma.  Exact
    // while dem * (ratio - r) < 1 / (reduced denominator), i.e. dem_cap[parent] * q_red < 2^s.
    dp->uni_dem_r.assign(dp->members.size() * (size_t)p.T, 0.0);
    bool dem_exact = true;
    for (int c = 1; c < p.T; ++c) {
      const int u = p.parent[c];
      for (size_t m = 0; m < (size_t)p.O[u]; ++m) {
        const DirRec& src = dp->members[(size_t)dp->member_off[u] + m];
        const uint64_t num = (uint64_t)p.fanout[c] * (uint64_t)opts[(size_t)(opt_off[u] + src.opt)].vf16;
        const uint64_t den = 16000000ull;
        const u128 qred = den / gcd_u64(num, den);
        const u128 lim = (u128)dp->dem_cap[u];
        double rd;
        int sc;
        if (!recip_below(num, den, &rd, &sc, true) || (sc < 126 && lim * qred >= ((u128)1 << sc)) ||
            lim * num / den >= ((u128)1 << 50))
          dem_exact = false;
        else
          dp->uni_dem_r[((size_t)dp->member_off[u] + m) * (size_t)p.T + (size_t)c] = rd;
      }
    }
    // per class, the in-class member indices in ascending task latency (ties: ascending index):
    // the hoisted kernel lays a class out in this order so that "fits the latency slack" is a prefix
    dp->lat_order.assign(dp->members.size(), 0);
    for (int i = 0; i < p.T; ++i)
      for (int c = 0; c < dp->n_class[i]; ++c) {
        const size_t first = (size_t)dp->member_off[i] + (size_t)dp->class_first[(size_t)(dp->class_off[i] + c)];
        const int n = dp->class_count[(size_t)(dp->class_off[i] + c)];
        std::vector<int32_t> idx((size_t)n);
        for (int k = 0; k < n; ++k) idx[(size_t)k] = k;
        std::stable_sort(idx.begin(), idx.end(), [&](int32_t a, int32_t b) {
          return dp->members[first + (size_t)a].lat < dp->members[first + (size_t)b].lat;
        });
        for (int k = 0; k < n; ++k) dp->lat_order[first + (size_t)k] = idx[(size_t)k];
      }
    // the order of the joint rows of tasks 0 and 1 depends on their classes alone: tabulated here per
    // pair of classes where that is little, so that the hoisted kernel need not rank them per class tuple
    dp->join_order.clear();
    dp->join_stride = 0;
    if (p.T >= 3) {
      int64_t big0 = 0, big1 = 0;
      for (int c = 0; c < dp->n_class[0]; ++c) big0 = std::max<int64_t>(big0, dp->class_count[(size_t)(dp->class_off[0] + c)]);
      for (int c = 0; c < dp->n_class[1]; ++c) big1 = std::max<int64_t>(big1, dp->class_count[(size_t)(dp->class_off[1] + c)]);
      const int64_t stride = big0 * big1;
      if (stride <= kHoistMaxJoinRows && stride * dp->n_class[0] * dp->n_class[1] <= (1LL << 20)) {
        dp->join_stride = (int32_t)stride;
        dp->join_order.assign((size_t)(stride * dp->n_class[0] * dp->n_class[1]), 0);
        const auto sorted_lat = [&](int task, int cls, std::vector<int32_t>* out) {
          const size_t first = (size_t)dp->member_off[task] + (size_t)dp->class_first[(size_t)(dp->class_off[task] + cls)];
          const int n = dp->class_count[(size_t)(dp->class_off[task] + cls)];
          out->resize((size_t)n);
          for (int k = 0; k < n; ++k) (*out)[(size_t)k] = dp->members[first + (size_t)dp->lat_order[first + (size_t)k]].lat;
        };
        std::vector<int32_t> l0, l1, idx;
        for (int c1 = 0; c1 < dp->n_class[1]; ++c1)
          for (int c0 = 0; c0 < dp->n_class[0]; ++c0) {
            sorted_lat(0, c0, &l0);
            sorted_lat(1, c1, &l1);
            const size_t n0 = l0.size(), n = n0 * l1.size();
            idx.resize(n);
            for (size_t q = 0; q < n; ++q) idx[q] = (int32_t)q;
            std::stable_sort(idx.begin(), idx.end(), [&](int32_t a, int32_t b) {
              return (int64_t)l0[(size_t)a % n0] + l1[(size_t)a / n0] < (int64_t)l0[(size_t)b % n0] + l1[(size_t)b / n0];
            });
            std::copy(idx.begin(), idx.end(),
                      dp->join_order.begin() + (ptrdiff_t)(((size_t)c1 * (size_t)dp->n_class[0] + (size_t)c0) * (size_t)stride));
          }
      }
    }
    // shared-memory stage of one class tuple: header + the largest class of every task
    int64_t stage = kUniformHeaderBytes;
    for (int i = 0; i < p.T; ++i) {
      int64_t biggest = 0;
      for (int c = 0; c < dp->n_class[i]; ++c)
        biggest = std::max<int64_t>(biggest, dp->class_count[(size_t)(dp->class_off[i] + c)]);
      stage += biggest * (int64_t)rec;
    }
    int64_t max_members = 0;
    for (int i = 0; i < p.T; ++i) {
      int64_t biggest = 0;
      for (int c = 0; c < dp->n_class[i]; ++c)
        biggest = std::max<int64_t>(biggest, dp->class_count[(size_t)(dp->class_off[i] + c)]);
      max_members += biggest;
    }
    dp->uni_max_members = (int)max_members;
    // the root-first kernel runs 20-24 warps per SM on its registers anyway, so its stage (records plus
    // the demand ratios) may be larger than the level-lane kernel's before residency suffers
    constexpr int64_t kVariantMaxStageBytes = 12288;
    // (without per-variant factors the ratios are the edge factors alone and the same kernel applies; it is
    // then preferred to the leaf-first level-lane kernel, which it outruns on every workload measured)
    const bool rootfirst_fits = dem_exact && stage + max_members * 8 * p.T <= kVariantMaxStageBytes;
    dp->uniform_ok = rootfirst_fits;
    dp->rootfirst = rootfirst_fits;
    dp->tables_ok = stage <= kUniformMaxStageBytes;     // member records small enough for the hoisted kernel's staging
    dp->uni_stage_bytes = (int)((stage + 15) / 16 * 16);
  }
  dp->ok = true;
}

// Solves that use the shared constant-memory demand tile are ordered on the
// device through one event per device.
std::mutex g_tile_mutex;
cudaEvent_t g_tile_event[kMaxDevices];
bool g_tile_event_ready[kMaxDevices];

}  // namespace

struct loki_alloc {
  HostProblem hp;
  DevProblem dev;
  DirProblem dir;
  DirectPlan plan;
  int device = 0;
  int n_sms = 0;
  int path_auto = LOKI_PATH_GENERIC;
  int path_current = LOKI_PATH_GENERIC;
  int path_last = 0;                   // kernel the last solve used (resolves LOKI_PATH_FASTEST)
  int tile_last = 0;                   // demand levels per scoring tile in the last solve
  int n_blocks_generic = 0;
  int n_blocks_direct = 0;             // blocks of the direct kernel on its shortest tiles (the most it launches)
  std::vector<int> direct_occ;         // [level groups of the tile] resident blocks per SM
  int direct_tile_max = 0;             // most levels per launch of the direct kernel: whole groups within kDirectMaxTile
  uint32_t direct_n_units = 1;
  std::vector<uint32_t> direct_unit_start;   // [n_units + 1] first batch of every work unit
  uint32_t* d_unit_start = nullptr;
  int direct_tile_last = 0;            // tile of the last direct solve (for the executed-work count)
  int direct_tiles_last = 0;
  bool hoist_ok = false;               // at least the 32-level tile of the hoisted kernel fits
  bool hoist_tile_ok[3] = {false, false, false};   // tiles of 32, 64 and 128 levels
  HoistLayout hoist_lay[3];
  HoistLayout hoist_lay_flat[3];       // the same without the join of tasks 0 and 1 (what LOKI_PATH_PREFIX takes on a tree)
  int n_blocks_hoisted[3] = {0, 0, 0};
  int n_blocks_flat[3] = {0, 0, 0};    // blocks of the layout without the join (hoist_lay_flat)
  int n_blocks_uniform[3] = {0, 0, 0};   // tiles of 32, 64 and 128 levels
  int n_launches_last = 0;
  int64_t scratch_bytes = 0, table_bytes = 0;
  int padded_levels = 0;
  int64_t partial_keys = 0;            // capacity of d_partial
  // device memory
  OptRec* d_opts = nullptr;
  int64_t* d_dem64 = nullptr;
  int32_t* d_status = nullptr;
  double* d_demf = nullptr;
  int64_t* d_dem_cap = nullptr;
  Key* d_partial = nullptr;
  Key* d_final = nullptr;
  Key* d_zero_key = nullptr;
  int32_t* d_class_first = nullptr;
  int32_t* d_class_count = nullptr;
  double* d_class_acc = nullptr;
  DirRec* d_members = nullptr;
  uint64_t* d_iter_prefix = nullptr;
  uint64_t* d_ct_acc = nullptr;
  uint64_t* d_ct_sorted_acc = nullptr;
  uint32_t* d_ct_sorted_idx = nullptr;
  uint32_t* d_ct_rank = nullptr;
  uint32_t* d_debug_flags = nullptr;   // status words of the checked build (zero in the release build)
  int32_t* d_slo_limits = nullptr;     // [kMaxSweepSlos][kMaxTasks] per-leaf latency limits of an SLO sweep
  uint32_t* d_counters = nullptr;      // [0..1] rows scored by the direct kernel (64 bits), [2 + t] unit counter of tile t
  int n_counters = 0;
  double* d_uni_dem_r = nullptr;
  unsigned char* d_uni_members = nullptr;
  int32_t* d_class_min_lat = nullptr;
  int32_t* d_lat_order = nullptr;
  int32_t* d_join_order = nullptr;
  // tables shared by all class tuples (LOKI_PATH_PREFIX)
  bool ptab_ok = false;
  PrefixTables ptab{};
  int ptab_blocks[3] = {0, 0, 0};      // resident blocks of the walk, by tile size
  int4* d_pt_desc = nullptr;
  int32_t* d_pt_lat = nullptr;
  uint32_t* d_pt_digit = nullptr;
  int32_t* d_pt_class_rows = nullptr;
  int32_t* d_pt_pair_rows = nullptr;
  int2* d_pt_groups = nullptr;
  uint32_t* d_pt_tab = nullptr;
  int64_t* d_demand_stage = nullptr;
  loki_config_t* d_out_stage = nullptr;
  std::vector<void*> owned;
  // optional timing of the scoring launches (loki_alloc_set_timing)
  bool timing = false;
  std::vector<cudaEvent_t> ev;     // begin/end pairs, one per scoring launch
  int ev_used = 0;
};

namespace {

template <typename Tp>
int dev_alloc(loki_alloc* h, Tp** ptr, size_t count, int64_t* account) {
  const size_t bytes = std::max<size_t>(count, 1) * sizeof(Tp);
  void* q = nullptr;
  const cudaError_t e = cudaMalloc(&q, bytes);
  if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return LOKI_ERR_NOMEM; }
  if (e != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  h->owned.push_back(q);
  *ptr = static_cast<Tp*>(q);
  *account += (int64_t)bytes;
  return LOKI_OK;
}

template <typename Tp>
int dev_upload(loki_alloc* h, Tp** ptr, const std::vector<Tp>& v, int64_t* account) {
  const int rc = dev_alloc(h, ptr, v.size(), account);
  if (rc != LOKI_OK) return rc;
  if (!v.empty() &&
      cudaMemcpy(*ptr, v.data(), v.size() * sizeof(Tp), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  return LOKI_OK;
}

void free_all(loki_alloc* h) {
  for (void* q : h->owned) cudaFree(q);
  h->owned.clear();
  for (cudaEvent_t e : h->ev) cudaEventDestroy(e);
  h->ev.clear();
}

// Brackets one scoring launch with an event pair when timing is on.
struct ScoreTimer {
  loki_alloc* h;
  cudaStream_t st;
  int slot;
  ScoreTimer(loki_alloc* h_, cudaStream_t st_) : h(h_), st(st_), slot(-1) {
    if (!h->timing) return;
    while ((int)h->ev.size() < h->ev_used + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return; }
      h->ev.push_back(e);
    }
    slot = h->ev_used;
    h->ev_used += 2;
    cudaEventRecord(h->ev[(size_t)slot], st);
  }
  ~ScoreTimer() {
    if (slot >= 0) cudaEventRecord(h->ev[(size_t)slot + 1], st);
  }
};

// LOKI_PATH_AUTO (and its older name LOKI_PATH_FASTEST) for a sweep of n_levels: the kernel this
// library's measurements say is quickest.  The hoisted kernel (with prefix minima) wherever its class tables fit the
// shared-memory bound, except short sweeps (at most 16 levels) of big candidate spaces, where the
// table build is not amortised and the direct kernel wins; where the tables do not fit, the
// root-first level-lane kernel on sweeps of several tiles, else the direct kernel; the generic
// kernel where the exactness conditions of the others fail.  Per-variant factors: the root-first
// kernel, else the generic one.
// The hoisted kernel's layout for tiles of 32 << v levels, with (LOKI_PATH_PREFIX) or without the
// prefix minima of the inner rows.  One task has no outer digit to look a prefix up for.
HoistLayout hoist_layout(const loki_alloc* h, int v, bool prefix) {
  if (!prefix || h->hp.T == 1) return h->hoist_lay[v];
  // joined tasks on a tree walk their rows one by one where a path bypasses task 1: the prefix
  // minima of task 0's rows under a loop over task 1 serve such problems instead
  HoistLayout lay = h->hoist_lay[v].join_rows > 0 && h->hp.n_leaves > 1 ? h->hoist_lay_flat[v] : h->hoist_lay[v];
  lay.pmin_mode = 1;
  return lay;
}

int resolve_path(const loki_alloc* h, int n_levels) {
  if (h->path_current != LOKI_PATH_FASTEST && h->path_current != LOKI_PATH_AUTO) return h->path_current;
  if (!h->plan.ok || h->plan.variant) return h->path_auto;
  const bool fits = h->hoist_ok && h->hoist_lay[0].smem_bytes <= kHoistMaxSmemBytes;
  const bool short_and_big = h->hp.N >= (1LL << 20) && n_levels <= 16;
  if (fits && !short_and_big) return h->hp.T > 1 ? LOKI_PATH_PREFIX : LOKI_PATH_HOISTED;
  if (!fits && h->plan.rootfirst && n_levels >= 256) return LOKI_PATH_UNIFORM;
  return h->path_auto;
}

// Every exit of the direct branch records the event that orders users of the shared
// constant-memory demand tile, also when a launch in between failed.
struct TileEventGuard {
  cudaEvent_t ev;
  cudaStream_t st;
  ~TileEventGuard() { cudaEventRecord(ev, st); }
};

// d_out == nullptr: the plans are not decoded, only the reduced keys written to h->d_final.
int enqueue_solve(loki_alloc* h, const int64_t* d_demand, int n_levels, cudaStream_t st,
                  loki_config_t* d_out, int path, const Key* zero_key) {
  int launches = 0;
  const bool shared_tables = h->ptab_ok && (path == LOKI_PATH_SHARED ||
      (path == LOKI_PATH_PREFIX && (double)h->hp.N * (double)n_levels >= kPrefixSharedMinPairs));
  const bool hoisted = path == LOKI_PATH_HOISTED || path == LOKI_PATH_PREFIX || path == LOKI_PATH_SHARED;
  const bool uniform = path == LOKI_PATH_UNIFORM;
  const bool direct = path == LOKI_PATH_DIRECT || hoisted || uniform;   // all use the clamped demand tiles
  const int uni_v = n_levels <= 32 ? 0 : 1;     // the root-first kernel takes tiles of 32 or 64 levels
  int hoist_v = n_levels <= 32 ? 0 : n_levels <= 64 ? 1 : 2;   // the largest tile up to that size whose table fits
  while (hoist_v > 0 && !h->hoist_tile_ok[hoist_v]) --hoist_v;
  const bool counted = path == LOKI_PATH_DIRECT;      // the direct kernel deals its work through counters
  int tile = uniform ? 32 << uni_v : hoisted ? 32 << hoist_v : 0;
  if (counted) {
    // tiles as even as the sweep allows, each whole level groups and a last group that may be shorter
    const int tiles = (n_levels + h->direct_tile_max - 1) / h->direct_tile_max;
    tile = direct_tile_levels(h->hp.T, (n_levels + tiles - 1) / tiles);
  }
  h->tile_last = direct ? tile : kGenericLevelGroup;
  const int n_tiles = direct ? (n_levels + tile - 1) / tile : 1;
  // K0 serves the generic kernel (stage demands and status per level) and the direct kernel (its demand
  // tiles, work counters zeroed); the level-lane kernels and the finishing kernels derive what they need
  // from the root demands themselves
  if (!direct || counted) {
    if (launch_prepare_levels(h->dev, d_demand, n_levels, h->d_dem64, h->d_status, h->d_dem_cap,
                              counted ? h->d_demf : nullptr, counted ? -tile : tile, st,
                              counted ? h->d_counters : nullptr,
                              counted ? std::min(h->n_counters, 2 + n_tiles) : 0) != cudaSuccess)
      return LOKI_ERR_CUDA;
    ++launches;
  }
  if (!direct) {
    {
      ScoreTimer timer(h, st);
      if (launch_generic_score(h->dev, h->d_dem64, h->d_status, n_levels, h->n_blocks_generic,
                               h->d_partial, st) != cudaSuccess)
        return LOKI_ERR_CUDA;
    }
    if (launch_finish(h->dev, h->d_partial, h->n_blocks_generic, 0, 0, n_levels, d_demand,
                      zero_key, h->d_final, d_out, st) != cudaSuccess)
      return LOKI_ERR_CUDA;
    launches += 2;
  } else if (shared_tables) {
    // tables shared by all class tuples: built once for the whole sweep, then walked, a warp per
    // class tuple; blocks per tile so that about twice the resident warps are in flight over all tiles
    const int v = n_levels <= 32 ? 0 : n_levels <= 64 ? 1 : 2;
    tile = 32 << v;
    h->tile_last = tile;
    const int tiles = (n_levels + tile - 1) / tile;
    int64_t nb = std::max<int64_t>(16, 2 * (int64_t)h->ptab_blocks[v] / tiles);
    nb = std::min<int64_t>(nb, h->ptab_blocks[v]);
    nb = std::min<int64_t>(nb, (h->dir.n_ct + kPrefixWarps - 1) / kPrefixWarps);
    nb = std::max<int64_t>(1, std::min<int64_t>(nb, h->partial_keys / ((int64_t)kPrefixWarps * tile)));
    const int n_parts = (int)nb * kPrefixWarps;
    const int64_t tile_keys = (int64_t)n_parts * tile;
    const int per_launch = (int)std::max<int64_t>(1, std::min<int64_t>(tiles, h->partial_keys / tile_keys));
    for (int t = 0; t < tiles; t += per_launch) {
      const int tiles_here = std::min(per_launch, tiles - t);
      const int levels_here = std::min(tiles_here * tile, n_levels - t * tile);
      {
        ScoreTimer timer(h, st);
        if (t == 0) {
          if (launch_prefix_build(h->dir, h->ptab, LevelSpan{d_demand, n_levels, 0}, tile, tiles, st) != cudaSuccess)
            return LOKI_ERR_CUDA;
          ++launches;
        }
        if (launch_prefix_walk(h->dir, h->ptab, LevelSpan{d_demand, n_levels, t * tile}, tile, t, tiles_here, (int)nb,
                               h->d_partial, st) != cudaSuccess)
          return LOKI_ERR_CUDA;
      }
      if (launch_finish(h->dev, h->d_partial, n_parts, tile, t * tile, levels_here, d_demand, zero_key,
                        h->d_final, d_out, st) != cudaSuccess)
        return LOKI_ERR_CUDA;
      launches += 2;
    }
  } else if (uniform || hoisted) {
    // level-lane kernels: several level tiles per launch (grid.y), as many as the scratch holds
    const HoistLayout lay = hoist_layout(h, hoist_v, path == LOKI_PATH_PREFIX || path == LOKI_PATH_SHARED);
    const int nb = uniform ? h->n_blocks_uniform[uni_v]
                 : lay.join_rows == h->hoist_lay[hoist_v].join_rows ? h->n_blocks_hoisted[hoist_v] : h->n_blocks_flat[hoist_v];
    const int n_parts = uniform ? nb : nb * lay.warps;     // partial keys per level: one per warp
    const int64_t tile_keys = (int64_t)n_parts * tile;
    const int per_launch = (int)std::max<int64_t>(1, std::min<int64_t>(n_tiles, h->partial_keys / tile_keys));
    for (int t = 0; t < n_tiles; t += per_launch) {
      const int tiles_here = std::min(per_launch, n_tiles - t);
      const int levels_here = std::min(tiles_here * tile, n_levels - t * tile);
      const LevelSpan span{d_demand, n_levels, t * tile};
      {
        ScoreTimer timer(h, st);
        const cudaError_t e = uniform
            ? launch_variant_score(h->dir, span, tile, nb, h->d_partial, st, tiles_here)
            : launch_hoisted_score(h->dir, lay, span, tile, nb, h->d_partial, st, false, tiles_here);
        if (e != cudaSuccess) return LOKI_ERR_CUDA;
      }
      if (launch_finish(h->dev, h->d_partial, n_parts, tile, t * tile, levels_here, d_demand, zero_key,
                        h->d_final, d_out, st) != cudaSuccess)
        return LOKI_ERR_CUDA;
      launches += 2;
    }
  } else {
    const int n_groups = (tile - 1) / direct_group_levels(h->hp.T) + 1;
    const int nb = (int)std::min<int64_t>(h->n_blocks_direct, (int64_t)h->n_sms * h->direct_occ[(size_t)n_groups]);
    std::lock_guard<std::mutex> lock(g_tile_mutex);
    const int dv = h->device;
    if (!g_tile_event_ready[dv]) {
      if (cudaEventCreateWithFlags(&g_tile_event[dv], cudaEventDisableTiming) != cudaSuccess)
        return LOKI_ERR_CUDA;
      g_tile_event_ready[dv] = true;
    } else if (cudaStreamWaitEvent(st, g_tile_event[dv], 0) != cudaSuccess) {
      return LOKI_ERR_CUDA;
    }
    TileEventGuard guard{g_tile_event[dv], st};
    h->direct_tile_last = tile;
    h->direct_tiles_last = n_tiles;
    for (int t = 0; t < n_tiles; ++t) {
      const int here = std::min(tile, n_levels - t * tile);
      const int tile_doubles = n_groups * direct_group_stride(h->hp.T);
      const double* dem = h->d_demf + (size_t)t * tile_doubles;
      if (direct_upload_tile(dem, tile_doubles, st) != cudaSuccess) return LOKI_ERR_CUDA;
      {
        ScoreTimer timer(h, st);
        if (launch_direct_score(h->dir, tile, nb, h->d_partial, h->d_counters + 2 + t,
                                reinterpret_cast<unsigned long long*>(h->d_counters), h->direct_n_units,
                                st) != cudaSuccess)
          return LOKI_ERR_CUDA;
      }
      if (launch_direct_finish(h->dir, h->dev, h->d_partial, nb, t * tile, here, dem, d_demand, zero_key,
                               h->d_final, d_out, st) != cudaSuccess)
        return LOKI_ERR_CUDA;
      launches += 3;
    }
  }
  h->n_launches_last = launches;
  return LOKI_OK;
}

// Enqueues, on `st`, the computation of the demand-free answer of zero-demand levels under the
// handle's current latency limits and its copy into *dst (device).  With zero demand no option needs
// a worker, so the answer is the most accurate latency-feasible candidate with the lowest index: the
// hoisted kernel's walk with rank-only table entries where its tables fit, else one generic pass
// with D = 0.  Uses the handle's scratch like a solve.
int enqueue_zero_key(loki_alloc* h, cudaStream_t st, Key* dst, int* launches) {
  if (cudaMemsetAsync(h->d_demand_stage, 0, sizeof(int64_t), st) != cudaSuccess) return LOKI_ERR_CUDA;
  if (h->plan.ok && h->hoist_ok) {
    const int tile = 32;
    if (launch_hoisted_score(h->dir, h->hoist_lay[0], LevelSpan{h->d_demand_stage, 1, 0}, tile,
                             h->n_blocks_hoisted[0], h->d_partial, st, true) != cudaSuccess ||
        launch_finish(h->dev, h->d_partial, h->n_blocks_hoisted[0] * h->hoist_lay[0].warps, 0, 0, 1,
                      h->d_demand_stage, nullptr, h->d_final, nullptr, st) != cudaSuccess)
      return LOKI_ERR_CUDA;
    if (launches) *launches += 3;
  } else {
    const bool timing = h->timing;
    h->timing = false;
    const int rc = enqueue_solve(h, h->d_demand_stage, 1, st, nullptr, LOKI_PATH_GENERIC, nullptr);
    h->timing = timing;
    if (rc != LOKI_OK) return rc;
    if (launches) *launches += h->n_launches_last + 1;
  }
  if (cudaMemcpyAsync(dst, h->d_final, sizeof(Key), cudaMemcpyDeviceToDevice, st) != cudaSuccess) return LOKI_ERR_CUDA;
  if (launches) *launches += 1;
  return LOKI_OK;
}

// One demand sweep under n_slos latency SLOs with the hoisted kernel, the SLOs as a second
// batched axis of the same launches (grid.z of the scoring kernel, grid.y of the finishing
// kernel): the SLO enters the walk only as the slack it starts from, so the worker tables are
// shared.  Enqueues: the per-SLO limits (one copy), the demand-free answers of all SLOs (level
// kernel, one scoring launch, one finishing launch), the level kernel of the sweep, and per
// batch of (SLOs x level tiles) that the partial-key scratch holds one scoring and one finishing
// launch -- a single pair for sweeps of small problems.
int enqueue_slo_sweep_hoisted(loki_alloc* h, const int64_t* d_demand, int n_levels, const int64_t* slo_us,
                              int n_slos, cudaStream_t st, loki_config_t* d_out) {
  const HostProblem& hp = h->hp;
  std::vector<int32_t> lim((size_t)n_slos * kMaxTasks, 0);
  for (int s = 0; s < n_slos; ++s)
    for (int k = 0; k < hp.n_leaves; ++k) {
      const int64_t budget = slo_us[s] - (int64_t)hp.depth[hp.leaf_task[k]] * hp.comm;
      lim[(size_t)s * kMaxTasks + (size_t)k] = budget < 0 ? -1 : (int32_t)std::min<int64_t>(budget / 2, (1LL << 31) - 1);
    }
  int launches = 0;
  // pageable source: the copy has left the host buffer when the call returns
  if (cudaMemcpyAsync(h->d_slo_limits, lim.data(), lim.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return LOKI_ERR_CUDA;
  ++launches;
  Key* const zero_keys = h->d_zero_key + 1;
  // ---- the demand-free answer of every SLO (zero-demand levels take it) ----
  {
    const int tile = 32, nb = h->n_blocks_hoisted[0], n_parts = nb * h->hoist_lay[0].warps;
    if (cudaMemsetAsync(h->d_demand_stage, 0, sizeof(int64_t), st) != cudaSuccess) return LOKI_ERR_CUDA;
    ++launches;
    const int64_t slo_keys = (int64_t)n_parts * tile;
    const int per = (int)std::max<int64_t>(1, std::min<int64_t>(n_slos, h->partial_keys / slo_keys));
    for (int s0 = 0; s0 < n_slos; s0 += per) {
      const int here = std::min(per, n_slos - s0);
      if (launch_hoisted_score(h->dir, h->hoist_lay[0], LevelSpan{h->d_demand_stage, 1, 0}, tile, nb, h->d_partial, st,
                               true, 1, here, h->d_slo_limits + (size_t)s0 * kMaxTasks) != cudaSuccess ||
          launch_finish(h->dev, h->d_partial, n_parts, 0, 0, 1, h->d_demand_stage, nullptr, zero_keys + s0, nullptr,
                        st, here, slo_keys, 1) != cudaSuccess)
        return LOKI_ERR_CUDA;
      launches += 2;
    }
  }
  // ---- the sweep ----
  int hoist_v = n_levels <= 32 ? 0 : n_levels <= 64 ? 1 : 2;
  while (hoist_v > 0 && !h->hoist_tile_ok[hoist_v]) --hoist_v;
  const HoistLayout lay = hoist_layout(h, hoist_v, h->path_last != LOKI_PATH_HOISTED);
  const int tile = 32 << hoist_v;
  const int nb = lay.join_rows == h->hoist_lay[hoist_v].join_rows ? h->n_blocks_hoisted[hoist_v] : h->n_blocks_flat[hoist_v];
  const int n_parts = nb * lay.warps;
  h->tile_last = tile;
  const int n_tiles = (n_levels + tile - 1) / tile;
  const int64_t tile_keys = (int64_t)n_parts * tile;
  // as many (SLO, tile) pairs per launch as the scratch holds: whole sweeps of several SLOs where
  // a sweep fits, else one SLO and a run of tiles
  const int64_t pairs = std::max<int64_t>(1, h->partial_keys / tile_keys);
  const int slos_per = (int)std::max<int64_t>(1, std::min<int64_t>(n_slos, pairs / n_tiles));
  const int tiles_per = pairs >= n_tiles ? n_tiles : (int)pairs;
  for (int s0 = 0; s0 < n_slos; s0 += slos_per) {
    const int slos_here = std::min(slos_per, n_slos - s0);
    for (int t = 0; t < n_tiles; t += tiles_per) {
      const int tiles_here = std::min(tiles_per, n_tiles - t);
      const int levels_here = std::min(tiles_here * tile, n_levels - t * tile);
      const LevelSpan span{d_demand, n_levels, t * tile};
      {
        ScoreTimer timer(h, st);
        if (launch_hoisted_score(h->dir, lay, span, tile, nb, h->d_partial, st, false, tiles_here,
                                 slos_here, h->d_slo_limits + (size_t)s0 * kMaxTasks) != cudaSuccess)
          return LOKI_ERR_CUDA;
      }
      if (launch_finish(h->dev, h->d_partial, n_parts, tile, t * tile, levels_here, d_demand, zero_keys + s0,
                        nullptr, d_out + (size_t)s0 * n_levels, st, slos_here,
                        (int64_t)tiles_here * tile_keys, n_levels) != cudaSuccess)
        return LOKI_ERR_CUDA;
      launches += 2;
    }
  }
  h->n_launches_last = launches;
  return LOKI_OK;
}

// The handle's own demand-free answer: on the default stream, then a synchronise.
int compute_zero_key(loki_alloc* h) {
  const int rc = enqueue_zero_key(h, 0, h->d_zero_key, nullptr);
  if (rc != LOKI_OK) { cudaGetLastError(); return rc; }
  if (cudaStreamSynchronize(0) != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  return LOKI_OK;
}

}  // namespace

namespace loki {
bool handle_view(const loki_alloc_t* h, HandleView* out) {
  if (!h || !out) return false;
  out->dev = h->dev;
  out->device = h->device;
  out->n_sms = h->n_sms;
  out->n_tasks = h->hp.T;
  out->n_batches = h->hp.nB;
  return true;
}
}  // namespace loki

extern "C" {

int loki_alloc_validate(const loki_alloc_desc_t* desc) {
  HostProblem* hp = new (std::nothrow) HostProblem;
  if (!hp) return LOKI_ERR_NOMEM;
  int rc;
  try {
    rc = validate_into(desc, hp);
  } catch (const std::bad_alloc&) {
    rc = LOKI_ERR_NOMEM;
  }
  delete hp;
  return rc;
}

int loki_alloc_plan_selfcheck(const loki_alloc_desc_t* desc, int32_t* direct_ok,
                              int64_t* n_checked, int64_t* n_mismatch) {
  if (!direct_ok || !n_checked || !n_mismatch) return LOKI_ERR_INVALID_ARG;
  *direct_ok = 0; *n_checked = 0; *n_mismatch = 0;
  try {
    HostProblem hp;
    const int rc = validate_into(desc, &hp);
    if (rc != LOKI_OK) return rc;
    std::vector<OptRec> opts;
    int64_t opt_off[kMaxTasks];
    build_options(hp, opts, opt_off);
    DirectPlan pl;
    plan_direct(hp, opts, opt_off, &pl);
    if (!pl.ok) return LOKI_OK;
    *direct_ok = pl.variant ? 0 : 1;   // with per-variant factors the same fma serves the root-first kernel
    // replay the kernel's fma-round-down arithmetic with integers against exact division
    for (int i = 0; i < hp.T; ++i) {
      const uint64_t lim = (uint64_t)pl.dem_cap[i];
      const int64_t m_begin = pl.member_off[i];
      const int64_t m_end = i + 1 < hp.T ? pl.member_off[i + 1] : (int64_t)pl.members.size();
      for (int64_t m = m_begin; m < m_end; ++m) {
        const DirRec& rec = pl.members[(size_t)m];
        const OptRec& o = opts[(size_t)(opt_off[i] + rec.opt)];
        for (int sidx = 0; sidx < o.parts; ++sidx) {
          const uint64_t pp = (uint64_t)o.mult[sidx], qq = (uint64_t)o.den[sidx];
          // the stored double as M * 2^-sc with M a 53-bit integer
          int ex = 0;
          const double fr = std::frexp(rec.r[sidx], &ex);
          const uint64_t M = (uint64_t)std::ldexp(fr, 53);
          const int sc = 53 - ex;
          auto check = [&](uint64_t dem) {
            if (dem < 1 || dem > lim) return;
            // fma.rm(dem, r, integer) adds floor(dem * r) = floor(dem * M / 2^sc)
            const u128 prod = (u128)dem * M;
            const uint64_t w = 1 + (sc >= 128 ? 0 : (uint64_t)(prod >> sc));
            const u128 num = (u128)dem * pp;
            const uint64_t want = (uint64_t)((num + qq - 1) / qq);
            ++*n_checked;
            if (w != want) ++*n_mismatch;
          };
          check(1); check(2); check(lim); check(lim - 1); check(lim / 2); check(lim / 3 + 1);
          // demands on both sides of the points where the ceiling steps
          for (uint64_t w = 1; w <= 40; ++w) {
            const uint64_t edge = (uint64_t)((u128)w * qq / pp);
            check(edge - 1); check(edge); check(edge + 1);
          }
          const uint64_t wl = (uint64_t)((u128)lim * pp / qq);
          for (uint64_t w = wl > 3 ? wl - 3 : 1; w <= wl; ++w) {
            const uint64_t edge = (uint64_t)((u128)w * qq / pp);
            check(edge - 1); check(edge); check(edge + 1);
          }
        }
      }
    }
    // per-variant factors: the root-first kernel derives a child's stage demand with the same fma
    // form; replay it for every (child task, parent option) against exact division
    if (pl.rootfirst)
      for (int c = 1; c < hp.T; ++c) {
        const int u = hp.parent[c];
        const uint64_t lim = (uint64_t)pl.dem_cap[u];
        for (int64_t m = 0; m < hp.O[u]; ++m) {
          const DirRec& rec = pl.members[(size_t)(pl.member_off[u] + m)];
          const uint64_t pp = (uint64_t)hp.fanout[c] * (uint64_t)opts[(size_t)(opt_off[u] + rec.opt)].vf16;
          const uint64_t qq = 16000000ull;
          int ex = 0;
          const double fr = std::frexp(pl.uni_dem_r[(size_t)(pl.member_off[u] + m) * (size_t)hp.T + (size_t)c], &ex);
          const uint64_t M = (uint64_t)std::ldexp(fr, 53);
          const int sc = 53 - ex;
          auto check = [&](uint64_t dem) {
            if (dem < 1 || dem > lim) return;
            const u128 prod = (u128)dem * M;
            const uint64_t got = 1 + (sc >= 128 ? 0 : (uint64_t)(prod >> sc));
            const uint64_t want = (uint64_t)(((u128)dem * pp + qq - 1) / qq);
            ++*n_checked;
            if (got != want) ++*n_mismatch;
          };
          check(1); check(2); check(lim); check(lim - 1); check(lim / 2); check(lim / 3 + 1);
          for (uint64_t w = 1; w <= 40; ++w) {
            const uint64_t edge = (uint64_t)((u128)w * qq / pp);
            check(edge - 1); check(edge); check(edge + 1);
          }
          const uint64_t wl = (uint64_t)((u128)lim * pp / qq);
          for (uint64_t w = wl > 3 ? wl - 3 : 1; w <= wl; ++w) {
            const uint64_t edge = (uint64_t)((u128)w * qq / pp);
            check(edge - 1); check(edge); check(edge + 1);
          }
        }
      }
  } catch (const std::bad_alloc&) {
    return LOKI_ERR_NOMEM;
  }
  return LOKI_OK;
}

int loki_alloc_create(const loki_alloc_desc_t* desc, loki_alloc_t** out) {
  if (out == nullptr) return LOKI_ERR_INVALID_ARG;
  loki_alloc* h = new (std::nothrow) loki_alloc;
  if (!h) return LOKI_ERR_NOMEM;
  int rc = LOKI_OK;
  try {
    rc = validate_into(desc, &h->hp);
    if (rc != LOKI_OK) { delete h; return rc; }
    const HostProblem& p = h->hp;
    if (cudaGetDevice(&h->device) != cudaSuccess || h->device < 0 || h->device >= kMaxDevices) {
      cudaGetLastError();
      delete h;
      return LOKI_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, h->device) != cudaSuccess) {
      cudaGetLastError();
      delete h;
      return LOKI_ERR_CUDA;
    }
    h->n_sms = prop.multiProcessorCount;
    // the allocation-free entry point's fixed array is bound to this device now, while allocating is allowed
    if ((rc = static_scratch_prepare(h->device)) != LOKI_OK) { delete h; return rc; }

    std::vector<OptRec> opts;
    int64_t opt_off[kMaxTasks];
    build_options(p, opts, opt_off);

    auto fail = [&](int code) { free_all(h); delete h; return code; };
    if ((rc = dev_upload(h, &h->d_opts, opts, &h->table_bytes)) != LOKI_OK) return fail(rc);
    // task accuracies of all options are computed on the device (split mean in
    // three rounded operations) and read back for the class construction
    {
      double* d_var_acc = nullptr;
      if ((rc = dev_upload(h, &d_var_acc, p.acc, &h->table_bytes)) != LOKI_OK) return fail(rc);
      for (int i = 0; i < p.T; ++i)
        if (launch_option_accuracy(h->d_opts + opt_off[i], p.O[i], d_var_acc + p.voff[i], 0) !=
            cudaSuccess) {
          cudaGetLastError();
          return fail(LOKI_ERR_CUDA);
        }
      if (cudaMemcpy(opts.data(), h->d_opts, opts.size() * sizeof(OptRec),
                     cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return fail(LOKI_ERR_CUDA);
      }
    }
    plan_direct(p, opts, opt_off, &h->plan);

    DevProblem& d = h->dev;
    std::memset(&d, 0, sizeof(d));
    d.T = p.T; d.n_leaves = p.n_leaves; d.split = p.split; d.S = p.S; d.N = p.N;
    d.opts = h->d_opts; d.max_demand_mqps = p.max_demand;
    d.variant_fanout = p.variant_fanout ? 1 : 0;
    d.n_opts = (int64_t)opts.size();
    for (int i = 0; i < p.T; ++i) {
      d.parent[i] = p.parent[i]; d.fanout_milli[i] = p.fanout[i];
      d.O[i] = p.O[i]; d.stride[i] = p.stride[i]; d.opt_off[i] = opt_off[i];
    }
    for (int k = 0; k < p.n_leaves; ++k) {
      d.leaf_task[k] = p.leaf_task[k]; d.path_mask[k] = p.path_mask[k]; d.lat_limit[k] = p.lat_limit[k];
    }

    // scoring grid sizes
    h->n_blocks_generic = std::max(1, h->n_sms * 2);
    // level arrays are padded to whole tiles of every kernel (the direct kernel's: up to kDirectMaxTile)
    // (a direct tile is rounded up to whole groups of at most 16 levels, and there is one tile per 240 levels or more)
    h->padded_levels = (p.max_levels + p.max_levels / 15 + 16 + kDirectMaxTile - 1) / kDirectMaxTile * kDirectMaxTile;
    size_t partial_keys = (size_t)h->n_blocks_generic * (size_t)h->padded_levels;
    if (h->plan.ok) {
      const DirectPlan& pl = h->plan;
      // direct kernel: one warp per block, as many as stay resident; work is dealt in units of
      // column batches through a device counter
      {
        const int G = direct_group_levels(p.T);
        h->direct_tile_max = kDirectMaxTile / G * G;
        // resident blocks per SM by the number of level groups of a tile (the per-level minima take
        // shared memory, so a short tile may leave room for one block more than the longest)
        const int max_groups = h->direct_tile_max / G;
        h->direct_occ.assign((size_t)max_groups + 1, 0);
        for (int g = 1; g <= max_groups; ++g) {
          h->direct_occ[(size_t)g] = direct_max_blocks_per_sm(p.T, pl.n_parts_max, g);
          if (h->direct_occ[(size_t)g] < 1) { cudaGetLastError(); return fail(LOKI_ERR_CUDA); }
        }
        const int64_t resident = (int64_t)h->n_sms * h->direct_occ[1];
        const int64_t iters = std::max<int64_t>(1, pl.total_iters);
        // guided schedule: a unit is a share 1 / (share x warps) of the work still to deal, so the units
        // start long (few partly filled stages) and end short (the launch ends evenly).  Work is counted
        // in steps: a column batch of a class tuple costs one step per member of task 0's class.
        {
          const double share = 4.0;                // measured best of 2 .. 8 over the named workloads
          std::vector<int> cls((size_t)p.T, 0);
          std::vector<uint32_t> ct_batches((size_t)pl.n_ct), ct_steps((size_t)pl.n_ct);
          double total_cost = 0.0;
          for (int64_t ct = 0; ct < pl.n_ct; ++ct) {
            uint64_t cols = 1;
            for (int i = 1; i < p.T; ++i) cols *= (uint64_t)pl.class_count[(size_t)(pl.class_off[i] + cls[(size_t)i])];
            const uint64_t c0 = (uint64_t)pl.class_count[(size_t)(pl.class_off[0] + cls[0])];
            ct_batches[(size_t)ct] = (uint32_t)(p.T == 1 ? 1 : (cols + kDirectBatch - 1) / kDirectBatch);
            ct_steps[(size_t)ct] = (uint32_t)(p.T == 1 ? (c0 + 31) / 32 : c0);
            total_cost += (double)ct_batches[(size_t)ct] * (double)ct_steps[(size_t)ct];
            for (int i = 0; i < p.T; ++i) {
              if (++cls[(size_t)i] < pl.n_class[i]) break;
              cls[(size_t)i] = 0;
            }
          }
          const double min_cost = 2.0 * total_cost / (double)iters;      // about two average batches
          h->direct_unit_start.clear();
          double remaining = total_cost;
          int64_t at = 0, ct = 0;
          uint32_t used = 0;                       // batches of class tuple `ct` already dealt
          while (at < iters) {
            h->direct_unit_start.push_back((uint32_t)at);
            const double target = std::max(min_cost, remaining / (share * (double)resident));
            double got = 0.0;
            while (ct < pl.n_ct && got < target) {
              const uint32_t left = ct_batches[(size_t)ct] - used;
              const double per = (double)ct_steps[(size_t)ct];
              uint32_t take = (uint32_t)std::min<double>((double)left, std::ceil((target - got) / per));
              if (take == 0) take = 1;
              got += per * take;
              at += take;
              used += take;
              if (used == ct_batches[(size_t)ct]) { ++ct; used = 0; }
            }
            remaining -= got;
          }
          h->direct_unit_start.push_back((uint32_t)iters);
        }
        h->direct_n_units = (uint32_t)(h->direct_unit_start.size() - 1);
        h->n_blocks_direct = (int)std::max<int64_t>(1, std::min<int64_t>(resident, h->direct_n_units));
        partial_keys = std::max(partial_keys, (size_t)h->n_blocks_direct * (size_t)h->direct_tile_max);
      }
      // level-lane kernel: one warp per block, as many as stay resident
      if (pl.uniform_ok) {
        DirProblem shape;
        std::memset(&shape, 0, sizeof(shape));
        shape.T = p.T; shape.n_parts_max = pl.n_parts_max; shape.n_leaves = p.n_leaves;
        shape.uni_stage_bytes = pl.uni_stage_bytes;
        for (int k = 0; k < p.n_leaves; ++k) shape.path_mask[k] = p.path_mask[k];
        shape.uni_max_members = pl.uni_max_members;
        for (int v = 0; v < 2; ++v) {
          const int tile = 32 << v;
          const int occ = variant_max_blocks_per_sm(shape, tile);
          if (occ < 1) { cudaGetLastError(); return fail(LOKI_ERR_CUDA); }
          int64_t nb = (int64_t)h->n_sms * occ;
          nb = std::min<int64_t>(nb, std::max<int64_t>(1, p.N / 128));
          h->n_blocks_uniform[v] = (int)nb;
          partial_keys = std::max(partial_keys, (size_t)nb * (size_t)tile);
        }
      }
      // hoisted kernel: per-class-tuple worker tables in shared memory, shared by the warps of a block
      h->hoist_ok = false;
      if (pl.tables_ok && !pl.variant) {
        int64_t members = 0, big[kMaxTasks];
        for (int i = 0; i < p.T; ++i) {
          int64_t biggest = 0;
          for (int c = 0; c < pl.n_class[i]; ++c)
            biggest = std::max<int64_t>(biggest, pl.class_count[(size_t)(pl.class_off[i] + c)]);
          members += biggest;
          big[i] = biggest;
        }
        // three or more tasks with small innermost classes: walk tasks 0 and 1 as one loop
        const int64_t join_rows = (p.T >= 3 && big[0] * big[1] <= kHoistMaxJoinRows) ? big[0] * big[1] : 0;
        DirProblem shape;
        std::memset(&shape, 0, sizeof(shape));
        shape.T = p.T; shape.n_parts_max = pl.n_parts_max; shape.n_leaves = p.n_leaves;
        for (int k = 0; k < p.n_leaves; ++k) shape.path_mask[k] = p.path_mask[k];
        const int64_t smallest = kUniformHeaderBytes + (members * 4 + 15) / 16 * 16 + members * 32 * 4;
        const int64_t join_ints = (join_rows * 4 * 4 + 15) / 16 * 16;
        // big classes: better few resident warps than no hoisted path at all
        const int64_t bound = smallest <= kHoistMaxSmemBytes ? kHoistMaxSmemBytes : kHoistLastResortSmemBytes;
        for (int v = 0; v < 3; ++v) {
          const int tile = 32 << v;
          HoistLayout& lay = h->hoist_lay[v];
          const int64_t base = kUniformHeaderBytes + (members * 4 + 15) / 16 * 16 + members * tile * 4;
          if (base > bound) continue;
          // the joint table is taken only where it still fits the bound
          // joined: tasks 0 and 1 keep no table rows of their own, only their member records
          const int64_t joined = big[0] + big[1];
          const int64_t rec_bytes = pl.n_parts_max == 2 ? kUniRecBytes2 : kUniRecBytes1;
          const int64_t with_join = kUniformHeaderBytes + (members * 4 + 15) / 16 * 16 + (members - joined) * tile * 4 +
                                    join_ints + joined * rec_bytes + join_rows * tile * 4;
          const bool join = join_rows > 0 && with_join <= kHoistMaxSmemBytes;
          lay.smem_bytes = (int32_t)(join ? with_join : base);
          lay.max_members = (int32_t)members;
          lay.join_rows = join ? (int32_t)join_rows : 0;
          lay.tab_members = (int32_t)(join ? members - joined : members);
          lay.join_members = (int32_t)(join ? joined : 0);
          lay.pmin_mode = 0;
          // warps per block: they share the table and split the class tuple's candidates (walk_share).
          // Measured over the named workloads with 2 .. 8 warps: few warps for small tables (less waiting
          // at the class-tuple barrier: C4 0.245 ms with 2 against 0.280 with 5), more where the table is
          // big and blocks per SM are few (C5's 49 KB: 5.45 ms with 8, 5.66 with 6, 6.12 with 4) --
          // about one warp per 8 KB of table, all eight above 40 KB
          const auto warps_for = [](int64_t smem) {
            return smem > 40 * 1024 ? kHoistMaxWarps
                                    : (int)std::min<int64_t>(kHoistMaxWarps, std::max<int64_t>(2, (smem + 4096) / 8192));
          };
          lay.warps = warps_for(lay.smem_bytes);
          const int occ = hoisted_max_blocks_per_sm(shape, lay, tile);
          if (occ < 1) { cudaGetLastError(); continue; }
          int64_t nb = (int64_t)h->n_sms * occ;
          nb = std::min<int64_t>(nb, std::max<int64_t>(1, pl.n_ct));      // a block takes whole class tuples
          h->n_blocks_hoisted[v] = (int)nb;
          h->hoist_tile_ok[v] = true;
          partial_keys = std::max(partial_keys, (size_t)nb * (size_t)lay.warps * (size_t)tile);
          // the layout without the join, with its own grid (its table is smaller, more blocks stay
          // resident; the query also admits its shared memory to that instantiation)
          HoistLayout& flat = h->hoist_lay_flat[v];
          flat = lay;
          h->n_blocks_flat[v] = (int)nb;
          if (join) {
            flat.smem_bytes = (int32_t)base;
            flat.join_rows = 0;
            flat.tab_members = (int32_t)members;
            flat.join_members = 0;
            flat.warps = warps_for(flat.smem_bytes);
            const int occ_flat = hoisted_max_blocks_per_sm(shape, flat, tile);
            if (occ_flat < 1) {
              cudaGetLastError();
              flat = lay;
            } else {
              h->n_blocks_flat[v] = (int)std::min<int64_t>((int64_t)h->n_sms * occ_flat, std::max<int64_t>(1, pl.n_ct));
              partial_keys = std::max(partial_keys, (size_t)h->n_blocks_flat[v] * (size_t)flat.warps * (size_t)tile);
            }
          }
        }
        h->hoist_ok = h->hoist_tile_ok[0];
      }
    }

    const size_t ML = (size_t)h->padded_levels;
    if ((rc = dev_alloc(h, &h->d_dem64, ML * kMaxTasks, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_status, ML, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_demf, ML * kMaxTasks, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    // room for several level tiles of the level-lane kernels in one launch, up to kMaxPartialKeys
    {
      size_t batched = partial_keys;
      for (int v = 0; v < 3; ++v) {
        const int tile = 32 << v;
        const size_t tiles = ((size_t)h->padded_levels + tile - 1) / tile;
        const size_t nb = (size_t)std::max(h->n_blocks_uniform[v],
                                           h->hoist_tile_ok[v] ? std::max(h->n_blocks_hoisted[v] * h->hoist_lay[v].warps,
                                                                          h->n_blocks_flat[v] * h->hoist_lay_flat[v].warps) : 0);
        // the hoisted kernel also takes SLO sweeps as a batched axis: room for 16 SLOs of a whole sweep where that is little
        const size_t slos = h->hoist_tile_ok[v] ? 16 : 1;
        batched = std::max(batched, std::min<size_t>(slos * tiles * nb * tile, (size_t)kMaxPartialKeys));
      }
      partial_keys = std::max(partial_keys, batched);
    }
    h->partial_keys = (int64_t)partial_keys;
    if ((rc = dev_alloc(h, &h->d_partial, partial_keys, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_debug_flags, (size_t)kDebugWords, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if (cudaMemset(h->d_debug_flags, 0, sizeof(uint32_t) * kDebugWords) != cudaSuccess) { cudaGetLastError(); return fail(LOKI_ERR_CUDA); }
    d.partial_keys = h->partial_keys;
    d.debug_flags = h->d_debug_flags;
    if ((rc = dev_alloc(h, &h->d_final, ML, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_zero_key, 1 + kMaxSweepSlos, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_demand_stage, ML, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_out_stage, ML, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    if ((rc = dev_alloc(h, &h->d_slo_limits, (size_t)kMaxSweepSlos * kMaxTasks, &h->scratch_bytes)) != LOKI_OK) return fail(rc);
    h->n_counters = 2 + (int)ML;       // the direct kernel's tiles hold at least one level each
    if ((rc = dev_alloc(h, &h->d_counters, (size_t)h->n_counters, &h->scratch_bytes)) != LOKI_OK) return fail(rc);

    if (h->plan.ok) {
      DirectPlan& pl = h->plan;
      std::vector<int64_t> cap(pl.dem_cap, pl.dem_cap + kMaxTasks);
      if ((rc = dev_upload(h, &h->d_dem_cap, cap, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_class_first, pl.class_first, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_class_count, pl.class_count, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_class_acc, pl.class_acc, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_members, pl.members, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_iter_prefix, pl.iter_prefix, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_uni_members, pl.uni_members, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_class_min_lat, pl.class_min_lat, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_lat_order, pl.lat_order, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if ((rc = dev_upload(h, &h->d_uni_dem_r, pl.uni_dem_r, &h->table_bytes)) != LOKI_OK) return fail(rc);
      if (!pl.join_order.empty() &&
          (rc = dev_upload(h, &h->d_join_order, pl.join_order, &h->table_bytes)) != LOKI_OK) return fail(rc);
      DirProblem& q = h->dir;
      std::memset(&q, 0, sizeof(q));
      q.T = p.T; q.n_leaves = p.n_leaves; q.S = p.S; q.jbits = pl.jbits; q.n_parts_max = pl.n_parts_max;
      q.N = p.N; q.n_ct = pl.n_ct; q.total_iters = pl.total_iters;
      for (int i = 0; i < p.T; ++i) {
        q.n_class[i] = pl.n_class[i]; q.class_off[i] = pl.class_off[i];
        q.parent[i] = p.parent[i]; q.stride[i] = p.stride[i]; q.member_off[i] = pl.member_off[i];
      }
      for (int k = 0; k < p.n_leaves; ++k) {
        q.leaf_task[k] = p.leaf_task[k]; q.path_mask[k] = p.path_mask[k]; q.lat_limit[k] = pl.lat_limit[k];
      }
      q.class_first = h->d_class_first; q.class_count = h->d_class_count; q.class_acc = h->d_class_acc;
      q.members = h->d_members; q.iter_prefix = h->d_iter_prefix;
      q.uni_members = h->d_uni_members; q.class_min_lat = h->d_class_min_lat;
      q.lat_order = h->d_lat_order;
      q.join_order = h->d_join_order;
      q.join_stride = pl.join_stride;
      q.uni_dem_r = h->d_uni_dem_r; q.dem_cap = h->d_dem_cap; q.uni_max_members = pl.uni_max_members;
      for (int i = 0; i < p.T; ++i) q.fanout_milli[i] = p.fanout[i];
      q.uni_stage_bytes = pl.uni_stage_bytes;
      q.max_demand_mqps = p.max_demand;
      if ((rc = dev_upload(h, &h->d_unit_start, h->direct_unit_start, &h->table_bytes)) != LOKI_OK) return fail(rc);
      q.unit_start = h->d_unit_start;
      q.n_classes = (int32_t)pl.class_count.size();
      q.n_members = (int32_t)pl.members.size();
      q.partial_keys = h->partial_keys;
      q.debug_flags = h->d_debug_flags;
      {
        int64_t nb_max = 1;
        for (int v = 0; v < 3; ++v)
          nb_max = std::max<int64_t>(nb_max, std::max(h->n_blocks_uniform[v], std::max(h->n_blocks_hoisted[v], h->n_blocks_flat[v])));
        const int64_t want = (kUniformUnitsPerWarp * nb_max + pl.n_ct - 1) / pl.n_ct;
        q.uni_slices = (int32_t)std::min<int64_t>(kUniformMaxSlices, std::max<int64_t>(1, want));
      }
      // end-to-end accuracy of every class tuple, computed on the device (a2), and the same
      // sorted by accuracy bits: the direct path's finishing kernel looks up the class tuples
      // that share a winning accuracy
      {
        if ((rc = dev_alloc(h, &h->d_ct_acc, (size_t)pl.n_ct, &h->table_bytes)) != LOKI_OK) return fail(rc);
        q.ct_acc = h->d_ct_acc;
        std::vector<uint64_t> acc((size_t)pl.n_ct);
        if (launch_class_tuple_accuracy(q, h->d_ct_acc, 0) != cudaSuccess ||
            cudaMemcpy(acc.data(), h->d_ct_acc, acc.size() * sizeof(uint64_t), cudaMemcpyDeviceToHost) != cudaSuccess) {
          cudaGetLastError();
          return fail(LOKI_ERR_CUDA);
        }
        std::vector<uint32_t> order((size_t)pl.n_ct);
        for (size_t k = 0; k < order.size(); ++k) order[k] = (uint32_t)k;
        std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
          return acc[a] < acc[b] || (acc[a] == acc[b] && a < b);
        });
        std::vector<uint64_t> sorted_acc(order.size());
        for (size_t k = 0; k < order.size(); ++k) sorted_acc[k] = acc[order[k]];
        if ((rc = dev_upload(h, &h->d_ct_sorted_acc, sorted_acc, &h->table_bytes)) != LOKI_OK) return fail(rc);
        if ((rc = dev_upload(h, &h->d_ct_sorted_idx, order, &h->table_bytes)) != LOKI_OK) return fail(rc);
        std::vector<uint32_t> rank(order.size());
        for (size_t k = 0; k < order.size(); ++k) rank[order[k]] = (uint32_t)k;
        if ((rc = dev_upload(h, &h->d_ct_rank, rank, &h->table_bytes)) != LOKI_OK) return fail(rc);
        q.ct_sorted_acc = h->d_ct_sorted_acc;
        q.ct_sorted_idx = h->d_ct_sorted_idx;
        q.ct_rank = h->d_ct_rank;
      }
      // tables shared by all class tuples, for LOKI_PATH_PREFIX: rows and groups now, the entries at
      // every solve.  Two tasks or more, one fan-out factor per edge, and tables of all level tiles
      // of the longest sweep within kPrefixMaxTableBytes.
      h->ptab_ok = false;
      if (!pl.variant && p.T > 1) {
        PrefixHost ph;
        plan_prefix_tables(p, pl, &ph);
        const int64_t levels128 = ((int64_t)p.max_levels + 127) / 128 * 128;
        const int64_t bytes = (int64_t)ph.row_desc.size() * levels128 * 4;
        if (!ph.row_desc.empty() && bytes <= kPrefixMaxTableBytes) {
          if ((rc = dev_upload(h, &h->d_pt_desc, ph.row_desc, &h->table_bytes)) != LOKI_OK) return fail(rc);
          if ((rc = dev_upload(h, &h->d_pt_lat, ph.row_lat, &h->table_bytes)) != LOKI_OK) return fail(rc);
          if ((rc = dev_upload(h, &h->d_pt_digit, ph.row_digit, &h->table_bytes)) != LOKI_OK) return fail(rc);
          if ((rc = dev_upload(h, &h->d_pt_class_rows, ph.class_rows, &h->table_bytes)) != LOKI_OK) return fail(rc);
          if (!ph.pair_rows.empty() &&
              (rc = dev_upload(h, &h->d_pt_pair_rows, ph.pair_rows, &h->table_bytes)) != LOKI_OK) return fail(rc);
          if ((rc = dev_upload(h, &h->d_pt_groups, ph.groups, &h->table_bytes)) != LOKI_OK) return fail(rc);
          if ((rc = dev_alloc(h, &h->d_pt_tab, (size_t)(bytes / 4), &h->scratch_bytes)) != LOKI_OK) return fail(rc);
          PrefixTables& t = h->ptab;
          t.row_desc = h->d_pt_desc; t.row_lat = h->d_pt_lat; t.row_digit = h->d_pt_digit;
          t.class_rows = h->d_pt_class_rows; t.pair_rows = h->d_pt_pair_rows; t.groups = h->d_pt_groups;
          t.tab = h->d_pt_tab;
          t.n_rows = (int32_t)ph.row_desc.size(); t.n_outer = ph.n_outer;
          t.n_groups = (int32_t)ph.groups.size(); t.joined = ph.joined ? 1 : 0;
          bool all = true;
          for (int v = 0; v < 3; ++v) {
            const int occ = prefix_walk_max_blocks_per_sm(q, t, 32 << v);
            if (occ < 1) { cudaGetLastError(); all = false; break; }
            h->ptab_blocks[v] = h->n_sms * occ;
          }
          h->ptab_ok = all;
        }
      }
      // the host copies of the big tables are no longer needed
      std::vector<DirRec>().swap(pl.members);
      std::vector<uint64_t>().swap(pl.iter_prefix);
      std::vector<unsigned char>().swap(pl.uni_members);
    }
    h->path_auto = !h->plan.ok ? LOKI_PATH_GENERIC
                   : !h->plan.variant ? LOKI_PATH_DIRECT
                   : h->plan.uniform_ok ? LOKI_PATH_UNIFORM : LOKI_PATH_GENERIC;
    h->path_current = LOKI_PATH_AUTO;

    rc = compute_zero_key(h);
    if (rc != LOKI_OK) return fail(rc);
    h->n_launches_last = 0;
  } catch (const std::bad_alloc&) {
    free_all(h);
    delete h;
    return LOKI_ERR_NOMEM;
  }
  *out = h;
  return LOKI_OK;
}

int loki_alloc_solve(loki_alloc_t* h, const int64_t* d_demand_mqps, int32_t n_levels,
                     void* cuda_stream, loki_config_t* d_out) {
  if (!h || !d_demand_mqps || !d_out) return LOKI_ERR_INVALID_ARG;
  if (n_levels < 1 || n_levels > h->hp.max_levels) return LOKI_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  if (dev != h->device) return LOKI_ERR_INVALID_ARG;
  h->path_last = resolve_path(h, n_levels);
  h->ev_used = 0;
  const int rc = enqueue_solve(h, d_demand_mqps, n_levels, static_cast<cudaStream_t>(cuda_stream),
                               d_out, h->path_last, h->d_zero_key);
  if (rc == LOKI_ERR_CUDA) cudaGetLastError();
  return rc;
}

int loki_alloc_solve_slos(loki_alloc_t* h, const int64_t* d_demand_mqps, int32_t n_levels,
                          const int64_t* slo_us, int32_t n_slos, void* cuda_stream,
                          loki_config_t* d_out) {
  if (!h || !d_demand_mqps || !d_out || !slo_us) return LOKI_ERR_INVALID_ARG;
  if (n_levels < 1 || n_levels > h->hp.max_levels) return LOKI_ERR_INVALID_ARG;
  if (n_slos < 1) return LOKI_ERR_INVALID_ARG;
  if (n_slos > kMaxSweepSlos) return LOKI_ERR_RANGE;
  for (int s = 0; s < n_slos; ++s)
    if (slo_us[s] < 0 || slo_us[s] > kMaxSloUs) return LOKI_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  if (dev != h->device) return LOKI_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  h->ev_used = 0;          // the timers of all launches accumulate
  const int sweep_path = resolve_path(h, n_levels);
  if ((sweep_path == LOKI_PATH_HOISTED || sweep_path == LOKI_PATH_PREFIX || sweep_path == LOKI_PATH_SHARED) &&
      h->plan.ok && h->hoist_ok) {
    // the SLOs as a second batched axis of the hoisted kernel's launches
    h->path_last = sweep_path;
    const int rc = enqueue_slo_sweep_hoisted(h, d_demand_mqps, n_levels, slo_us, n_slos, st, d_out);
    if (rc == LOKI_ERR_CUDA) cudaGetLastError();
    return rc;
  }
  // The other kernels take the per-path latency limits from their launch parameters:
  // swap them per SLO, put the handle's own back at the end.
  HostProblem saved = h->hp;
  const bool timing = h->timing;
  int rc = LOKI_OK;
  int launches = 0;
  for (int s = 0; s < n_slos && rc == LOKI_OK; ++s) {
    h->hp.slo = slo_us[s];
    set_leaf_limits(h->hp);
    for (int k = 0; k < h->hp.n_leaves; ++k) {
      h->dev.lat_limit[k] = h->hp.lat_limit[k];
      h->dir.lat_limit[k] = (int32_t)std::min<int64_t>(h->hp.lat_limit[k], (1LL << 31) - 1);
    }
    // the demand-free answer of zero-demand levels under this SLO, on the caller's stream,
    // kept in this SLO's slot
    Key* zero = h->d_zero_key + 1 + s;
    rc = enqueue_zero_key(h, st, zero, &launches);
    if (rc != LOKI_OK) break;
    h->path_last = resolve_path(h, n_levels);
    rc = enqueue_solve(h, d_demand_mqps, n_levels, st, d_out + (size_t)s * n_levels, h->path_last, zero);
    launches += h->n_launches_last;
  }
  h->timing = timing;
  h->hp = saved;
  for (int k = 0; k < h->hp.n_leaves; ++k) {
    h->dev.lat_limit[k] = h->hp.lat_limit[k];
    h->dir.lat_limit[k] = h->plan.lat_limit[k];
  }
  h->n_launches_last = launches;
  if (rc == LOKI_ERR_CUDA) cudaGetLastError();
  return rc;
}

int loki_alloc_solve_host(loki_alloc_t* h, const int64_t* h_demand_mqps, int32_t n_levels,
                          void* cuda_stream, loki_config_t* h_out) {
  if (!h || !h_demand_mqps || !h_out) return LOKI_ERR_INVALID_ARG;
  if (n_levels < 1 || n_levels > h->hp.max_levels) return LOKI_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(h->d_demand_stage, h_demand_mqps, sizeof(int64_t) * (size_t)n_levels,
                      cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  const int rc = loki_alloc_solve(h, h->d_demand_stage, n_levels, cuda_stream, h->d_out_stage);
  if (rc != LOKI_OK) return rc;
  if (cudaMemcpyAsync(h_out, h->d_out_stage, sizeof(loki_config_t) * (size_t)n_levels,
                      cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  h->n_launches_last += 2;
  return LOKI_OK;
}

int loki_alloc_destroy(loki_alloc_t* h) {
  if (!h) return LOKI_OK;
  cudaDeviceSynchronize();
  free_all(h);
  delete h;
  return LOKI_OK;
}

int loki_alloc_set_path(loki_alloc_t* h, int32_t path) {
  if (!h) return LOKI_ERR_INVALID_ARG;
  if (path == LOKI_PATH_AUTO || path == LOKI_PATH_FASTEST) { h->path_current = path; return LOKI_OK; }   // resolved per solve
  if (path == LOKI_PATH_GENERIC) { h->path_current = path; return LOKI_OK; }
  if (path == LOKI_PATH_DIRECT || path == LOKI_PATH_UNIFORM) {
    if (!h->plan.ok || (path == LOKI_PATH_UNIFORM && !h->plan.uniform_ok)) return LOKI_ERR_RANGE;
    if (path == LOKI_PATH_DIRECT && h->plan.variant) return LOKI_ERR_RANGE;
    h->path_current = path;
    return LOKI_OK;
  }
  if (path == LOKI_PATH_SHARED) {
    if (!h->plan.ok || !h->ptab_ok) return LOKI_ERR_RANGE;
    h->path_current = path;
    return LOKI_OK;
  }
  if (path == LOKI_PATH_HOISTED || path == LOKI_PATH_PREFIX) {
    if (!h->plan.ok || !h->hoist_ok) return LOKI_ERR_RANGE;
    h->path_current = path;
    return LOKI_OK;
  }
  return LOKI_ERR_INVALID_ARG;
}

int loki_alloc_set_slo(loki_alloc_t* h, int64_t slo_us, int64_t comm_us) {
  if (!h) return LOKI_ERR_INVALID_ARG;
  if (slo_us < 0 || slo_us > kMaxSloUs || comm_us < 0 || comm_us > kMaxCommUs) return LOKI_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  if (dev != h->device) return LOKI_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  h->hp.slo = slo_us;
  h->hp.comm = comm_us;
  set_leaf_limits(h->hp);
  for (int k = 0; k < h->hp.n_leaves; ++k) {
    h->dev.lat_limit[k] = h->hp.lat_limit[k];
    h->plan.lat_limit[k] = (int32_t)std::min<int64_t>(h->hp.lat_limit[k], (1LL << 31) - 1);
    h->dir.lat_limit[k] = h->plan.lat_limit[k];
  }
  return compute_zero_key(h);
}

int loki_alloc_set_timing(loki_alloc_t* h, int32_t enable) {
  if (!h) return LOKI_ERR_INVALID_ARG;
  h->timing = enable != 0;
  return LOKI_OK;
}

int loki_alloc_last_score_ms(loki_alloc_t* h, float* total_ms, int32_t* n_launches) {
  if (!h || !total_ms || !n_launches) return LOKI_ERR_INVALID_ARG;
  *total_ms = 0.0f;
  *n_launches = 0;
  for (int s = 0; s + 1 < h->ev_used; s += 2) {
    float ms = 0.0f;
    if (cudaEventSynchronize(h->ev[(size_t)s + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, h->ev[(size_t)s], h->ev[(size_t)s + 1]) != cudaSuccess) {
      cudaGetLastError();
      return LOKI_ERR_CUDA;
    }
    *total_ms += ms;
    ++*n_launches;
  }
  return LOKI_OK;
}

int loki_alloc_last_fma_count(loki_alloc_t* h, int64_t* executed) {
  if (!h || !executed) return LOKI_ERR_INVALID_ARG;
  *executed = 0;
  if (h->path_last != LOKI_PATH_DIRECT || h->d_counters == nullptr) return LOKI_OK;
  unsigned long long rows = 0;
  if (cudaMemcpy(&rows, h->d_counters, sizeof(rows), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  // a scored row is 32 candidates against every level of the tile, one fma per option part
  *executed = (int64_t)rows * 32 * h->direct_tile_last * h->hp.T * h->plan.n_parts_max;
  return LOKI_OK;
}

int loki_alloc_debug_status(const loki_alloc_t* h, int32_t* checked_build, uint32_t* site_mask,
                            uint32_t* n_violations) {
  if (!h || !checked_build || !site_mask || !n_violations) return LOKI_ERR_INVALID_ARG;
#ifdef LOKI_DEBUG
  *checked_build = 1;
#else
  *checked_build = 0;
#endif
  uint32_t words[kDebugWords] = {0, 0, 0, 0};
  if (h->d_debug_flags != nullptr &&
      cudaMemcpy(words, h->d_debug_flags, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  *site_mask = words[0];
  *n_violations = words[1];
  return LOKI_OK;
}

int loki_alloc_num_candidates(const loki_alloc_t* h, int64_t* out) {
  if (!h || !out) return LOKI_ERR_INVALID_ARG;
  *out = h->hp.N;
  return LOKI_OK;
}

int loki_alloc_get_info(const loki_alloc_t* h, loki_alloc_info_t* out) {
  if (!h || !out) return LOKI_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  out->n_candidates = h->hp.N;
  out->path_auto = h->path_auto;
  out->path_current = h->path_current;
  out->path_last = h->path_last;
  out->uniform_ok = h->plan.ok && h->plan.uniform_ok ? 1 : 0;
  out->level_tile_last = h->tile_last;
  out->direct_ok = h->plan.ok && !h->plan.variant ? 1 : 0;
  out->direct_level_tile = h->direct_tile_max;
  out->n_blocks = h->path_current == LOKI_PATH_UNIFORM ? h->n_blocks_uniform[1]
                  : h->path_current == LOKI_PATH_DIRECT ? h->n_blocks_direct
                  : h->path_current == LOKI_PATH_SHARED ? h->ptab_blocks[1]
                  : h->path_current == LOKI_PATH_HOISTED || h->path_current == LOKI_PATH_PREFIX ? h->n_blocks_hoisted[1]
                  : h->n_blocks_generic;
  out->hoisted_ok = h->plan.ok && h->hoist_ok ? 1 : 0;
  out->n_launches_last = h->n_launches_last;
  out->scratch_bytes = h->scratch_bytes;
  out->table_bytes = h->table_bytes;
  return LOKI_OK;
}

const char* loki_alloc_strerror(int code) {
  switch (code) {
    case LOKI_OK: return "ok";
    case LOKI_ERR_INVALID_ARG: return "invalid argument";
    case LOKI_ERR_INVALID_GRAPH: return "pipeline is not a rooted tree in topological order";
    case LOKI_ERR_RANGE: return "value range or search space too large";
    case LOKI_ERR_CUDA: return "CUDA call failed";
    case LOKI_ERR_NOMEM: return "out of memory";
    default: return "unknown error";
  }
}

int32_t loki_alloc_config_size(void) { return (int32_t)sizeof(loki_config_t); }

}  // extern "C"
