// loki_alloc_route: the Load Balancer's request routing (MostAccurateFirst,
// Algorithm 1 of Section 5.1) for a batch of demand levels, one thread per level.
// It consumes the plans loki_alloc_solve wrote for those levels and produces,
// per level, the routing tables of the Frontend and of every worker, and per
// worker its capacity, the requests routed to it and its leftover capacity (the
// list handed to upstream workers for opportunistic rerouting, Section 5.2).
//
// The greedy of one level is sequential -- a child worker's remaining capacity
// depends on everything routed before -- and short (a few hundred steps), so the
// parallel axis is the demand sweep: one warp per level, lane 0 walks the greedy
// with the level's worker table in shared memory (every step reads what the step
// before wrote), then all lanes copy the table out.  Plans with more workers
// than fit in shared memory are walked directly in the output buffer.  Arithmetic is IEEE double with explicitly
// rounded operations (no fused multiply-add), in the order Algorithm 1 states:
//   capacity  = (batch * 1e6) / lat_us                    (Eq. 5, queries/s)
//   outgoing  = (incoming * multFactor) * branchRatio
//   routed    = min(outgoing, capacity);  probability = routed / totalChildDemand
#include "loki_internal.h"

using namespace loki;

namespace {

struct RouteProblem {
  DevProblem dev;
  int32_t n_batches;
  int32_t max_workers;
  int32_t max_entries;
  int32_t pad;
};

// Algorithm 1 for level l; W is the level's worker table (shared or global memory).
__device__ void route_level(const RouteProblem& rp, const int64_t* __restrict__ demand,
                            const loki_config_t* __restrict__ plans, int l,
                            loki_route_header_t* __restrict__ hdr, loki_route_worker_t* W,
                            loki_route_entry_t* __restrict__ entries) {
  const DevProblem& p = rp.dev;
  const int T = p.T;
  loki_route_entry_t* E = entries + (size_t)l * rp.max_entries;
  loki_route_header_t h;
  h.status = LOKI_ROUTE_OK;
  h.n_workers = 0;
  h.n_entries = 0;
  h.reserved = 0;
  h.unrouted_qps = 0.0;
  const loki_config_t& plan = plans[l];
  if (plan.status != LOKI_LEVEL_FEASIBLE) {
    h.status = LOKI_ROUTE_NO_PLAN;
    hdr[l] = h;
    return;
  }

  // ---- the plan's workers, per task in non-increasing single-model accuracy ----
  int t_begin[kMaxTasks], t_end[kMaxTasks], open_from[kMaxTasks];
  int n = 0;
  bool overflow = false;
  for (int i = 0; i < T; ++i) {
    t_begin[i] = n;
    const int ng = plan.split_k[i] == 16 ? 1 : 2;
    int order[2] = {0, 1};
    if (ng == 2) {
      const OptRec* o0 = p.opts + p.opt_off[i] + (int64_t)plan.variant[i][0] * rp.n_batches;
      const OptRec* o1 = p.opts + p.opt_off[i] + (int64_t)plan.variant[i][1] * rp.n_batches;
      if (o1->acc > o0->acc) { order[0] = 1; order[1] = 0; }   // equal accuracies keep the plan's order
    }
    for (int g = 0; g < ng; ++g) {
      const int s = order[g];
      const int v = plan.variant[i][s], b = plan.batch[i][s], cnt = plan.workers[i][s];
      int64_t lat = 0;
      for (int bi = 0; bi < rp.n_batches; ++bi) {
        const OptRec* rec = p.opts + p.opt_off[i] + (int64_t)v * rp.n_batches + bi;
        if (rec->den[0] == (int64_t)b * 1000000000LL) lat = rec->lat;
      }
      const double cap = lat > 0 ? __ddiv_rn(__dmul_rn((double)b, 1e6), (double)lat) : 0.0;
      for (int k = 0; k < cnt; ++k) {
        if (n < rp.max_workers) {
          loki_route_worker_t x;
          x.task = i; x.variant = v; x.batch = b; x.reserved = 0;
          x.capacity_qps = cap; x.incoming_qps = 0.0; x.leftover_qps = cap;
          W[n] = x;
          ++n;
        } else {
          overflow = true;
        }
      }
    }
    t_end[i] = n;
    open_from[i] = t_begin[i];
  }
  h.n_workers = n;
  if (overflow) {
    h.status = LOKI_ROUTE_TABLE_FULL;
    hdr[l] = h;
    return;
  }

  int n_e = 0;
  double unrouted = 0.0;
  // Routes `outgoing` requests of source worker `src` to the workers of `child`.
  // Workers before open_from[child] are saturated (capacity 0): the algorithm's
  // "capacity > 0" test skips them, the cursor only avoids re-reading them.
  auto fill = [&](int src, int child, double outgoing) {
    const double total = outgoing;
    for (int cw = open_from[child]; cw < t_end[child] && outgoing > 0.0; ++cw) {
      const double rem = W[cw].leftover_qps;
      if (rem > 0.0) {
        const double routed = outgoing < rem ? outgoing : rem;
        if (n_e < rp.max_entries) {
          loki_route_entry_t e;
          e.src_worker = src; e.dst_worker = cw; e.probability = __ddiv_rn(routed, total);
          E[n_e] = e;
        } else {
          h.status = LOKI_ROUTE_TABLE_FULL;
        }
        ++n_e;
        outgoing = __dsub_rn(outgoing, routed);
        const double left = __dsub_rn(rem, routed);
        W[cw].leftover_qps = left;
        W[cw].incoming_qps = __dadd_rn(W[cw].incoming_qps, routed);
        if (!(left > 0.0) && cw == open_from[child]) open_from[child] = cw + 1;
      } else if (cw == open_from[child]) {
        open_from[child] = cw + 1;
      }
    }
    if (outgoing > 0.0) unrouted = __dadd_rn(unrouted, outgoing);
  };

  fill(-1, 0, __ddiv_rn((double)demand[l], 1000.0));          // the Frontend's table
  for (int i = 0; i < T; ++i) {
    for (int u = t_begin[i]; u < t_end[i]; ++u) {
      const double inc = W[u].incoming_qps;
      const OptRec* rec = p.opts + p.opt_off[i] + (int64_t)W[u].variant * rp.n_batches;
      const double mult = __ddiv_rn((double)(rec->vf16 / 16u), 1000.0);
      for (int c = i + 1; c < T; ++c) {
        if (p.parent[c] != i) continue;
        const double branch = __ddiv_rn((double)p.fanout_milli[c], 1000.0);
        fill(u, c, __dmul_rn(__dmul_rn(inc, mult), branch));
      }
    }
  }
  h.n_entries = n_e < rp.max_entries ? n_e : rp.max_entries;
  h.unrouted_qps = unrouted;
  hdr[l] = h;
}

// One warp per level.  IN_SHARED: the worker table lives in dynamic shared memory while
// lane 0 walks, and is copied to the output by the whole warp afterwards.
template <bool IN_SHARED>
__global__ void __launch_bounds__(32)
route_kernel(const RouteProblem rp, const int64_t* __restrict__ demand,
             const loki_config_t* __restrict__ plans, int n_levels,
             loki_route_header_t* __restrict__ hdr, loki_route_worker_t* __restrict__ workers,
             loki_route_entry_t* __restrict__ entries) {
  extern __shared__ __align__(16) unsigned char s_route[];
  const int l = blockIdx.x;
  if (l >= n_levels) return;
  loki_route_worker_t* out = workers + (size_t)l * rp.max_workers;
  loki_route_worker_t* W = IN_SHARED ? reinterpret_cast<loki_route_worker_t*>(s_route) : out;
  if (threadIdx.x == 0) route_level(rp, demand, plans, l, hdr, W, entries);
  if (IN_SHARED) {
    __syncwarp();
    __threadfence_block();
    const int n = hdr[l].n_workers < rp.max_workers ? hdr[l].n_workers : rp.max_workers;
    for (int k = threadIdx.x; k < n; k += 32) out[k] = W[k];
  }
}

constexpr size_t kRouteSharedLimit = 96 * 1024;

}  // namespace

extern "C" int loki_alloc_route(const loki_alloc_t* h, const int64_t* d_demand_mqps,
                                const loki_config_t* d_plans, int32_t n_levels, int32_t max_workers,
                                int32_t max_entries, void* cuda_stream, loki_route_header_t* d_headers,
                                loki_route_worker_t* d_workers, loki_route_entry_t* d_entries) {
  if (!h || !d_demand_mqps || !d_plans || !d_headers || !d_workers || !d_entries) return LOKI_ERR_INVALID_ARG;
  if (n_levels < 1 || max_workers < 1 || max_entries < 1) return LOKI_ERR_INVALID_ARG;
  HandleView v;
  if (!handle_view(h, &v)) return LOKI_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  if (dev != v.device) return LOKI_ERR_INVALID_ARG;
  RouteProblem rp;
  rp.dev = v.dev;
  rp.n_batches = v.n_batches;
  rp.max_workers = max_workers;
  rp.max_entries = max_entries;
  rp.pad = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t table = (size_t)max_workers * sizeof(loki_route_worker_t);
  if (table <= kRouteSharedLimit) {
    if (table > 48 * 1024 &&
        cudaFuncSetAttribute(route_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)table) != cudaSuccess) {
      cudaGetLastError();
      return LOKI_ERR_CUDA;
    }
    route_kernel<true><<<n_levels, 32, table, st>>>(rp, d_demand_mqps, d_plans, n_levels, d_headers, d_workers,
                                                     d_entries);
  } else {
    route_kernel<false><<<n_levels, 32, 0, st>>>(rp, d_demand_mqps, d_plans, n_levels, d_headers, d_workers,
                                                  d_entries);
  }
  if (cudaGetLastError() != cudaSuccess) return LOKI_ERR_CUDA;
  return LOKI_OK;
}
