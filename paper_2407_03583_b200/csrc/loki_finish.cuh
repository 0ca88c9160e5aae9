// Device code shared by the finishing kernels of libloki_alloc (a9 + a10): the
// block-wide maximum over the partial keys of one demand level, and the decode of
// the winning key into the level's plan.  Included by the translation units that
// define a finishing kernel.
#ifndef LOKI_FINISH_CUH_
#define LOKI_FINISH_CUH_

#include "loki_internal.h"

namespace loki {

constexpr int kFinishThreads = 128;          // block of the finishing kernel
constexpr int kDirectFinishThreads = 512;    // ... of the direct path's, which also re-scores a class tuple per level
constexpr uint64_t kIndexMask = (1ull << 40) - 1;   // low part of Key::tail: N - 1 - candidate index

__device__ __forceinline__ int64_t finish_ceil_div(int64_t num, int64_t den) {
  // num >= 0, den > 0, num + den does not overflow (proved at create time)
  const uint64_t q = (uint64_t)num / (uint64_t)den;
  return (int64_t)(q + ((uint64_t)num - q * (uint64_t)den != 0 ? 1 : 0));
}

// Maximum over partial[pidx * partial_stride + column], pidx < n_parts, by all
// THREADS threads of the block; every thread returns the result.  Keys are
// totally ordered, so the maximum is the same bits whatever the order of the comparisons.
template <int THREADS>
__device__ __forceinline__ Key block_max_key(const Key* __restrict__ partial, int n_parts,
                                             int partial_stride, int column) {
  Key k{0ull, 0ull};
  for (int pidx = threadIdx.x; pidx < n_parts; pidx += THREADS) {
    const Key o = partial[(size_t)pidx * partial_stride + column];
    if (key_less(k, o)) k = o;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    Key o;
    o.acc_bits = __shfl_xor_sync(0xFFFFFFFFu, k.acc_bits, off);
    o.tail = __shfl_xor_sync(0xFFFFFFFFu, k.tail, off);
    if (key_less(k, o)) k = o;
  }
  __shared__ Key s_warp_key[THREADS / 32];
  if ((threadIdx.x & 31) == 0) s_warp_key[threadIdx.x >> 5] = k;
  __syncthreads();
  k = s_warp_key[0];
#pragma unroll
  for (int w = 1; w < THREADS / 32; ++w)
    if (key_less(k, s_warp_key[w])) k = s_warp_key[w];
  return k;
}

// a10: the plan of level l, whose demand is D, from its winning key (one thread).  Stage demands
// (a4: Eq. 1, ceiling on every edge) and workers are re-derived with plain integer division, and the
// worker sum must agree with the key's.
__device__ inline void decode_level(const DevProblem& p, const Key k, const int64_t D, int l,
                                    loki_config_t* __restrict__ out) {
  loki_config_t r;
  r.cand_index = -1;
  r.accuracy = 0.0;
  r.total_workers = 0;
  for (int i = 0; i < kMaxTasks; ++i) {
    r.variant[i][0] = r.variant[i][1] = -1;
    r.batch[i][0] = r.batch[i][1] = 0;
    r.workers[i][0] = r.workers[i][1] = 0;
    r.split_k[i] = 0;
    r.latency_budget_us[i] = 0;
  }
  if (D < 0 || D > p.max_demand_mqps) {
    r.status = LOKI_LEVEL_BAD_DEMAND;
  } else if (k.acc_bits == 0ull && k.tail == 0ull) {
    r.status = LOKI_LEVEL_INFEASIBLE;
  } else {
    const int64_t c = p.N - 1 - (int64_t)(k.tail & kIndexMask);
    if (c < 0 || c >= p.N) {
      r.status = LOKI_LEVEL_INTERNAL_ERROR;     // a key without a candidate behind it
    } else {
      r.status = LOKI_LEVEL_FEASIBLE;
      r.cand_index = c;
      r.accuracy = __longlong_as_double((long long)k.acc_bits);
      uint64_t rem = (uint64_t)c;
      int64_t W = 0;
      int64_t demv[kMaxTasks];
      uint32_t vf16[kMaxTasks];
      for (int i = 0; i < p.T; ++i) {
        const uint64_t Oi = (uint64_t)p.O[i];
        const uint64_t q = rem / Oi;
        const OptRec* rec = p.opts + LOKI_IDX(p.opt_off[i] + (rem - q * Oi), p.n_opts, kSiteOption, p.debug_flags);
        rem = q;
        int64_t d = D;
        if (i > 0)
          d = p.variant_fanout
                  ? finish_ceil_div(demv[p.parent[i]] * (int64_t)p.fanout_milli[i] * (int64_t)vf16[p.parent[i]], 16000000)
                  : finish_ceil_div(demv[p.parent[i]] * (int64_t)p.fanout_milli[i], 1000);
        demv[i] = d;
        vf16[i] = rec->vf16;
        r.split_k[i] = rec->k;
        r.latency_budget_us[i] = rec->lat;          // Sec. 4.2 "Latency budgets for tasks"
        for (int s = 0; s < rec->parts; ++s) {
          const int64_t w = finish_ceil_div(d * rec->mult[s], rec->den[s]);
          r.variant[i][s] = rec->variant[s];
          r.batch[i][s] = (int32_t)(rec->den[s] / (rec->parts == 2 ? 16000000000LL : 1000000000LL));
          r.workers[i][s] = (int32_t)w;
          W += w;
        }
      }
      r.total_workers = (int32_t)W;
      // the key's worker count must agree with the recomputation from the plan
      if (W != p.S - (int64_t)(k.tail >> 40)) r.status = LOKI_LEVEL_INTERNAL_ERROR;
    }
  }
  out[l] = r;
}

}  // namespace loki

#endif  // LOKI_FINISH_CUH_
