// CPU oracle for the allocation search.  TEST INFRASTRUCTURE ONLY: nothing on
// the product path may call, link or import this file; it shares no code,
// header, table or constant with the CUDA library.
//
// What it computes (Loki, HPDC '24; Section 4.1 "MILPs for hardware and
// accuracy scaling"): for every demand level D it enumerates, in ascending
// candidate index, every candidate allocation plan -- per task one (variant,
// batch size) option, or in split mode a pair of distinct options with a k/16
// traffic split -- and keeps the plan with the highest end-to-end accuracy
// that satisfies the paper's constraints, ties broken by fewer workers and
// then by lower candidate index:
//
//   * accuracy of a root-to-leaf path = product of the task accuracies on it,
//     pipeline accuracy = mean over leaves (Section 2.1 "Inference pipelines";
//     Section 4.1 "Modeling the system accuracy", objective Eq. 12);
//   * latency: for every root-to-leaf path 2 * sum lat <= SLO - hops * comm
//     (Eqs. 6-7, the halved SLO of "Meeting the latency SLO", and the
//     "Communication latency" paragraph of Section 4.2);
//   * stage demand: root demand times the multiplicative factors above the task
//     (Eq. 1): on every edge the parent's stage demand is multiplied by the edge's
//     factor and by the factor r(i,k) of the parent's chosen variant (the
//     k/16-weighted mean of the two in a split option; Algorithm 1 multiplies
//     "multFactor" by "branchRatio" the same way), rounded up per edge in
//     milli-queries/s;
//   * workers: smallest integer x with demand <= x * q where q = b / lat is
//     the profiled throughput (Eq. 2 with Eq. 5), i.e.
//     ceil(demand_mqps * lat_us / (b * 1e9));
//   * cluster: sum of workers <= S (Eq. 3);
//   * objective: Eq. 8-11 (fewest workers at maximum accuracy) and Eq. 12
//     (maximum accuracy) folded into one lexicographic order.
//
// It is the plain definition written out: no pruning, no tables of
// precomputed worker counts, plain '/' and '%', doubles with contraction
// disabled (compile with -ffp-contract=off).  Per-candidate quantities that
// do not depend on the demand (decode, accuracy, latency test) are evaluated
// once per candidate and the demand levels are the inner loop; threads split
// the candidate range into contiguous chunks and are merged in index order.
//
// Parity status: pinned by hand-worked examples (tests/golden), an
// independent pure-Python brute force, closed forms and invariants.  The
// *quality* of the allocation relative to the paper's MILP optimum (which may
// mix more than two variants per task with real-valued traffic ratios) is
// "parity unpinned": no MILP solver or profile data is available.
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <thread>
#include <vector>

namespace {

constexpr int kMaxTasks = 8;

struct Problem {
  int T = 0;
  int parent[kMaxTasks];
  int64_t fanout_milli[kMaxTasks];
  int V[kMaxTasks];
  int voff[kMaxTasks];  // offset of task's first variant in the flat tables
  int nB = 0;
  std::vector<int64_t> batch;
  std::vector<double> acc;       // [sumV]
  std::vector<int64_t> lat;      // [sumV][nB]
  std::vector<int64_t> vfan;     // [sumV] per-variant multiplicative factor r(i,k) in thousandths
  int64_t slo_us = 0, comm_us = 0;
  int64_t S = 0;
  int split = 0;
  int64_t nS[kMaxTasks];   // single options per task
  int64_t O[kMaxTasks];    // options per task
  int64_t N = 0;           // candidates
  int depth[kMaxTasks];    // tasks on the path root..i
  bool is_leaf[kMaxTasks];
  int n_leaves = 0;
};

// One option of a task, decoded: one or two (variant, batch index) parts.
struct Option {
  int parts;        // 1 or 2
  int v[2], bi[2];
  int k;            // 16 for a single option, else share (in 16ths) of part 0
};

// Split-mode numbering: options 0..nS-1 are the single options o = v*nB + bi.
// Above that, o' = o - nS, pair rank r = o' / 15, k = o' % 15 + 1; pairs
// (o1 < o2) are ranked lexicographically.
Option decode_option(const Problem& p, int task, int64_t o) {
  Option op;
  const int64_t nS = p.nS[task];
  if (o < nS) {
    op.parts = 1;
    op.v[0] = (int)(o / p.nB);
    op.bi[0] = (int)(o % p.nB);
    op.v[1] = op.bi[1] = -1;
    op.k = 16;
    return op;
  }
  const int64_t rest = o - nS;
  int64_t r = rest / 15;
  op.k = (int)(rest % 15) + 1;
  int64_t o1 = 0;
  while (r >= nS - 1 - o1) {   // row o1 holds the pairs (o1, o1+1 .. nS-1)
    r -= nS - 1 - o1;
    ++o1;
  }
  const int64_t o2 = o1 + 1 + r;
  op.parts = 2;
  op.v[0] = (int)(o1 / p.nB);
  op.bi[0] = (int)(o1 % p.nB);
  op.v[1] = (int)(o2 / p.nB);
  op.bi[1] = (int)(o2 % p.nB);
  return op;
}

inline int64_t ceil_div_i128(unsigned __int128 num, int64_t den) {
  const unsigned __int128 d = (unsigned __int128)den;
  if (num <= (unsigned __int128)INT64_MAX) {
    const int64_t n = (int64_t)num;
    return n / den + (n % den != 0 ? 1 : 0);
  }
  return (int64_t)(num / d) + ((num % d) != 0 ? 1 : 0);
}

struct Best {
  int64_t cand = -1;
  double acc = 0.0;
  int64_t workers = 0;
};

// true if (acc, W, c) beats b in the order: accuracy down, workers up, index up
inline bool better(double acc, int64_t W, int64_t c, const Best& b) {
  if (b.cand < 0) return true;
  if (acc != b.acc) return acc > b.acc;
  if (W != b.workers) return W < b.workers;
  return c < b.cand;
}

struct LevelInfo {
  int status;                   // 0 usable, 2 bad demand
  int64_t dem[kMaxTasks];       // stage demand in mQPS
};

void scan_range(const Problem& p, const std::vector<LevelInfo>& lv, int64_t c_begin,
                int64_t c_end, std::vector<Best>& best) {
  const int T = p.T;
  const int M = (int)lv.size();
  for (int64_t c = c_begin; c < c_end; ++c) {
    // decode: task 0 is the least significant digit
    Option op[kMaxTasks];
    int64_t rem = c;
    for (int i = 0; i < T; ++i) {
      op[i] = decode_option(p, i, rem % p.O[i]);
      rem /= p.O[i];
    }
    // task accuracy and task latency
    double a[kMaxTasks];
    int64_t L[kMaxTasks];
    for (int i = 0; i < T; ++i) {
      const int f = p.voff[i];
      if (op[i].parts == 1) {
        a[i] = p.acc[f + op[i].v[0]];
        L[i] = p.lat[(size_t)(f + op[i].v[0]) * p.nB + op[i].bi[0]];
      } else {
        const double A1 = p.acc[f + op[i].v[0]];
        const double A2 = p.acc[f + op[i].v[1]];
        const double share = (double)op[i].k * 0.0625;     // exact
        const double diff = A1 - A2;
        const double prod = share * diff;
        a[i] = A2 + prod;
        const int64_t l1 = p.lat[(size_t)(f + op[i].v[0]) * p.nB + op[i].bi[0]];
        const int64_t l2 = p.lat[(size_t)(f + op[i].v[1]) * p.nB + op[i].bi[1]];
        L[i] = l1 > l2 ? l1 : l2;     // both parts carry traffic (1 <= k <= 15)
      }
    }
    // path accuracy products in task order, then the mean over leaves
    double pp[kMaxTasks];
    int64_t pl[kMaxTasks];
    pp[0] = a[0];
    pl[0] = L[0];
    for (int i = 1; i < T; ++i) {
      const double up = pp[p.parent[i]];
      pp[i] = up * a[i];
      pl[i] = pl[p.parent[i]] + L[i];
    }
    double sum = 0.0;
    bool first = true;
    bool lat_ok = true;
    for (int i = 0; i < T; ++i) {
      if (!p.is_leaf[i]) continue;
      if (first) { sum = pp[i]; first = false; } else { sum = sum + pp[i]; }
      if (2 * pl[i] > p.slo_us - (int64_t)p.depth[i] * p.comm_us) lat_ok = false;
    }
    const double acc = sum / (double)p.n_leaves;
    if (!lat_ok) continue;

    // sixteenths-weighted multiplicative factor of each task's chosen option
    int64_t vf16[kMaxTasks];
    for (int i = 0; i < T; ++i) {
      const int f = p.voff[i];
      vf16[i] = op[i].parts == 1 ? 16 * p.vfan[f + op[i].v[0]]
                                 : op[i].k * p.vfan[f + op[i].v[0]] + (16 - op[i].k) * p.vfan[f + op[i].v[1]];
    }
    for (int m = 0; m < M; ++m) {
      if (lv[m].status != 0) continue;
      // stage demand (Eq. 1): ceiling on every edge
      int64_t demv[kMaxTasks];
      demv[0] = lv[m].dem[0];
      for (int i = 1; i < T; ++i) {
        const int u = p.parent[i];
        const unsigned __int128 num = (unsigned __int128)demv[u] * (unsigned __int128)p.fanout_milli[i] *
                                      (unsigned __int128)vf16[u];
        demv[i] = ceil_div_i128(num, 16000000LL);
      }
      int64_t W = 0;
      for (int i = 0; i < T; ++i) {
        const int f = p.voff[i];
        const unsigned __int128 dem = (unsigned __int128)demv[i];
        if (op[i].parts == 1) {
          const int64_t lat = p.lat[(size_t)(f + op[i].v[0]) * p.nB + op[i].bi[0]];
          const int64_t den = p.batch[op[i].bi[0]] * 1000000000LL;
          W += ceil_div_i128(dem * (unsigned __int128)lat, den);
        } else {
          for (int s = 0; s < 2; ++s) {
            const int64_t lat = p.lat[(size_t)(f + op[i].v[s]) * p.nB + op[i].bi[s]];
            const int64_t share = s == 0 ? op[i].k : 16 - op[i].k;
            const int64_t den = 16 * p.batch[op[i].bi[s]] * 1000000000LL;
            W += ceil_div_i128(dem * (unsigned __int128)share * (unsigned __int128)lat, den);
          }
        }
      }
      if (W > p.S) continue;
      if (better(acc, W, c, best[m])) {
        best[m].cand = c;
        best[m].acc = acc;
        best[m].workers = W;
      }
    }
  }
}

}  // namespace

extern "C" {

// Per-level result of the oracle (its own layout; not the library's struct).
struct loki_oracle_result {
  int64_t cand_index;      // -1 if no feasible candidate
  double accuracy;         // 0.0 if infeasible
  int64_t total_workers;   // 0 if infeasible
  int32_t status;          // 0 feasible, 1 infeasible, 2 bad demand
  int32_t pad;
  int32_t variant[kMaxTasks][2];
  int32_t batch[kMaxTasks][2];
  int64_t workers[kMaxTasks][2];
  int32_t split_k[kMaxTasks];
  int64_t latency_budget_us[kMaxTasks];
  int64_t stage_demand_mqps[kMaxTasks];
};

int loki_oracle_result_size(void) { return (int)sizeof(loki_oracle_result); }

// Returns 0 on success, -1 on malformed input.  All pointers are host memory.
// max_demand_mqps: levels with demand < 0 or > this bound get status 2.
// Only candidates with cand_begin <= index < cand_end take part (cand_end < 0
// means "to the end"); the full search is the range [0, N).
// variant_fanout_milli: [sum n_variants] r(i,k) in thousandths, or NULL for 1000 everywhere.
int loki_oracle_solve_range(int n_tasks, const int32_t* parent, const int32_t* fanout_milli,
                      const int32_t* n_variants, int n_batches, const int32_t* batch_sizes,
                      const double* accuracy, const int64_t* latency_us,
                      const int32_t* variant_fanout_milli, int64_t slo_us,
                      int64_t comm_us, int32_t cluster_size, int32_t split_mode,
                      int64_t max_demand_mqps, const int64_t* demand_mqps, int n_levels,
                      int n_threads, int64_t cand_begin, int64_t cand_end,
                      loki_oracle_result* out) {
  if (n_tasks < 1 || n_tasks > kMaxTasks || n_batches < 1 || n_levels < 0) return -1;
  Problem p;
  p.T = n_tasks;
  p.nB = n_batches;
  p.batch.assign(batch_sizes, batch_sizes + n_batches);
  int sumV = 0;
  for (int i = 0; i < n_tasks; ++i) {
    if (n_variants[i] < 1) return -1;
    if (i == 0 ? parent[i] != -1 : (parent[i] < 0 || parent[i] >= i)) return -1;
    p.parent[i] = parent[i];
    p.fanout_milli[i] = fanout_milli[i];
    p.V[i] = n_variants[i];
    p.voff[i] = sumV;
    sumV += n_variants[i];
  }
  p.acc.assign(accuracy, accuracy + sumV);
  p.lat.assign(latency_us, latency_us + (size_t)sumV * n_batches);
  p.vfan.assign((size_t)sumV, 1000);
  if (variant_fanout_milli != nullptr)
    for (int v = 0; v < sumV; ++v) {
      if (variant_fanout_milli[v] < 1) return -1;
      p.vfan[(size_t)v] = variant_fanout_milli[v];
    }
  p.slo_us = slo_us;
  p.comm_us = comm_us;
  p.S = cluster_size;
  p.split = split_mode;
  p.N = 1;
  for (int i = 0; i < n_tasks; ++i) {
    p.nS[i] = (int64_t)p.V[i] * p.nB;
    p.O[i] = split_mode ? p.nS[i] + (p.nS[i] * (p.nS[i] - 1) / 2) * 15 : p.nS[i];
    p.N *= p.O[i];
    p.is_leaf[i] = true;
    p.depth[i] = i == 0 ? 1 : p.depth[p.parent[i]] + 1;
  }
  for (int i = 1; i < n_tasks; ++i) p.is_leaf[p.parent[i]] = false;
  p.n_leaves = 0;
  for (int i = 0; i < n_tasks; ++i) p.n_leaves += p.is_leaf[i] ? 1 : 0;

  // per level: status and the root demand (stage demands depend on the candidate)
  std::vector<LevelInfo> lv((size_t)n_levels);
  for (int m = 0; m < n_levels; ++m) {
    const int64_t D = demand_mqps[m];
    lv[m].status = (D < 0 || D > max_demand_mqps) ? 2 : 0;
    if (lv[m].status != 0) { std::memset(lv[m].dem, 0, sizeof(lv[m].dem)); continue; }
    std::memset(lv[m].dem, 0, sizeof(lv[m].dem));
    lv[m].dem[0] = D;
  }

  if (cand_end < 0 || cand_end > p.N) cand_end = p.N;
  if (cand_begin < 0) cand_begin = 0;
  if (cand_begin > cand_end) cand_begin = cand_end;
  const int64_t span = cand_end - cand_begin;
  if (n_threads < 1) n_threads = 1;
  if ((int64_t)n_threads > span) n_threads = span > 0 ? (int)span : 1;
  std::vector<std::vector<Best>> part((size_t)n_threads, std::vector<Best>((size_t)n_levels));
  {
    std::vector<std::thread> th;
    for (int t = 0; t < n_threads; ++t) {
      const int64_t b = cand_begin + span / n_threads * t + (t < span % n_threads ? t : span % n_threads);
      const int64_t e = b + span / n_threads + (t < span % n_threads ? 1 : 0);
      if (n_threads == 1) {
        scan_range(p, lv, b, e, part[0]);
      } else {
        th.emplace_back([&, t, b, e] { scan_range(p, lv, b, e, part[(size_t)t]); });
      }
    }
    for (auto& x : th) x.join();
  }
  // merge the chunks in ascending candidate order with the same comparison
  std::vector<Best> best((size_t)n_levels);
  for (int t = 0; t < n_threads; ++t)
    for (int m = 0; m < n_levels; ++m) {
      const Best& b = part[(size_t)t][(size_t)m];
      if (b.cand >= 0 && better(b.acc, b.workers, b.cand, best[(size_t)m])) best[(size_t)m] = b;
    }

  for (int m = 0; m < n_levels; ++m) {
    loki_oracle_result& r = out[m];
    std::memset(&r, 0, sizeof(r));
    for (int i = 0; i < kMaxTasks; ++i) {
      r.variant[i][0] = r.variant[i][1] = -1;
      r.batch[i][0] = r.batch[i][1] = 0;
      r.split_k[i] = 0;
    }
    if (lv[m].status != 0) { r.cand_index = -1; r.status = 2; continue; }
    const Best& b = best[(size_t)m];
    if (b.cand < 0) { r.cand_index = -1; r.status = 1; continue; }
    r.cand_index = b.cand;
    r.accuracy = b.acc;
    r.total_workers = b.workers;
    r.status = 0;
    // decode the winner, then its stage demands (Eq. 1) and per-part workers
    Option wop[kMaxTasks];
    int64_t rem = b.cand;
    for (int i = 0; i < n_tasks; ++i) {
      wop[i] = decode_option(p, i, rem % p.O[i]);
      rem /= p.O[i];
    }
    r.stage_demand_mqps[0] = lv[m].dem[0];
    for (int i = 1; i < n_tasks; ++i) {
      const int u = p.parent[i];
      const int fu = p.voff[u];
      const int64_t vf16 = wop[u].parts == 1 ? 16 * p.vfan[fu + wop[u].v[0]]
                                             : wop[u].k * p.vfan[fu + wop[u].v[0]] +
                                                   (16 - wop[u].k) * p.vfan[fu + wop[u].v[1]];
      r.stage_demand_mqps[i] = ceil_div_i128((unsigned __int128)r.stage_demand_mqps[u] *
                                                 (unsigned __int128)p.fanout_milli[i] * (unsigned __int128)vf16,
                                             16000000LL);
    }
    for (int i = 0; i < n_tasks; ++i) {
      const Option& op = wop[i];
      const int f = p.voff[i];
      r.split_k[i] = op.k;
      int64_t budget = 0;
      for (int s = 0; s < op.parts; ++s) {
        const int64_t lat = p.lat[(size_t)(f + op.v[s]) * p.nB + op.bi[s]];
        r.variant[i][s] = op.v[s];
        r.batch[i][s] = (int32_t)p.batch[op.bi[s]];
        const unsigned __int128 dem = (unsigned __int128)r.stage_demand_mqps[i];
        if (op.parts == 1) {
          r.workers[i][s] = ceil_div_i128(dem * (unsigned __int128)lat, p.batch[op.bi[s]] * 1000000000LL);
        } else {
          const int64_t share = s == 0 ? op.k : 16 - op.k;
          r.workers[i][s] = ceil_div_i128(dem * (unsigned __int128)share * (unsigned __int128)lat,
                                          16 * p.batch[op.bi[s]] * 1000000000LL);
        }
        if (lat > budget) budget = lat;
      }
      r.latency_budget_us[i] = budget;   // Section 4.2 "Latency budgets for tasks"
    }
  }
  return 0;
}

int loki_oracle_solve(int n_tasks, const int32_t* parent, const int32_t* fanout_milli,
                      const int32_t* n_variants, int n_batches, const int32_t* batch_sizes,
                      const double* accuracy, const int64_t* latency_us,
                      const int32_t* variant_fanout_milli, int64_t slo_us,
                      int64_t comm_us, int32_t cluster_size, int32_t split_mode,
                      int64_t max_demand_mqps, const int64_t* demand_mqps, int n_levels,
                      int n_threads, loki_oracle_result* out) {
  return loki_oracle_solve_range(n_tasks, parent, fanout_milli, n_variants, n_batches, batch_sizes,
                                 accuracy, latency_us, variant_fanout_milli, slo_us, comm_us, cluster_size,
                                 split_mode, max_demand_mqps, demand_mqps, n_levels, n_threads, 0, -1, out);
}

}  // extern "C"
