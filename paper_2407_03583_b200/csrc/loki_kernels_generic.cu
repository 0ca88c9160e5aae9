// Set-up, level preparation, the generic scoring kernel and the finishing kernel
// (cross-block reduction + winner decode) of libloki_alloc.  Hand-written CUDA for sm_100a.
//
// The generic scoring kernel evaluates the definition directly in 64-bit
// integers (quotients estimated in floating point, corrected to the exact integer);
// it accepts every problem loki_alloc_create accepts and is the reference point for
// the faster kernels.  The winner decode uses plain division and cross-checks the key.
#include "loki_finish.cuh"

namespace loki {

namespace {

__device__ __forceinline__ int64_t ceil_div_pos(int64_t num, int64_t den) {
  // num >= 0, den > 0, num + den does not overflow (proved at create time)
  const uint64_t q = (uint64_t)num / (uint64_t)den;
  return (int64_t)(q + ((uint64_t)num - q * (uint64_t)den != 0 ? 1 : 0));
}

// The same ceiling with the quotient estimated in floating point and corrected in integers:
// exact for every num in [0, 2^63) and den in (0, 2^59) -- the loops run until the remainder
// is in [0, den), whatever the estimate was.  The divisors here are at least 1e9, so the
// quotient is below 2^34, the estimate is off by less than one, and the loops run at most once.
// inv_den is any double close to 1 / den.
__device__ __forceinline__ int64_t ceil_div_est(int64_t num, int64_t den, double inv_den) {
  uint64_t q = __double2ull_rz(__dmul_rn((double)num, inv_den));
  int64_t r = (int64_t)((uint64_t)num - q * (uint64_t)den);
  while (r < 0) { --q; r += den; }
  while (r >= den) { ++q; r -= den; }
  return (int64_t)q + (r != 0 ? 1 : 0);
}

// ---- set-up: task accuracy of every option, one thread per option ------------
// Split options: a = A2 + (k/16) * (A1 - A2) in three rounded operations (k/16 is
// exact), which returns A exactly when both parts use the same variant.
__global__ void option_accuracy_kernel(OptRec* __restrict__ opts, int64_t n,
                                       const double* __restrict__ variant_acc) {
  const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= n) return;
  OptRec& r = opts[o];
  if (r.parts == 1) {
    r.acc = variant_acc[r.variant[0]];
  } else {
    const double A1 = variant_acc[r.variant[0]], A2 = variant_acc[r.variant[1]];
    const double share = __dmul_rn((double)r.k, 0.0625);
    r.acc = __dadd_rn(A2, __dmul_rn(share, __dsub_rn(A1, A2)));
  }
}

// ---- K0: per level status and stage demand (Eq. 1, ceiling on every edge) ----
__global__ void prepare_levels_kernel(DevProblem p, const int64_t* __restrict__ demand,
                                      int n_levels, int n_padded, int64_t* __restrict__ dem64,
                                      int32_t* __restrict__ status,
                                      const int64_t* __restrict__ dem_cap,
                                      double* __restrict__ demf, int tile,
                                      uint32_t* __restrict__ zero_words, int n_zero_words) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  // the solve's work counters start from zero (the scoring launches follow on the same stream)
  for (int z = l; z < n_zero_words; z += gridDim.x * blockDim.x) zero_words[z] = 0u;
  if (l >= n_padded) return;
  int64_t dem[kMaxTasks];
#pragma unroll
  for (int i = 0; i < kMaxTasks; ++i) dem[i] = 0;
  int32_t st = LOKI_LEVEL_BAD_DEMAND;
  if (l < n_levels) {
    const int64_t D = demand[l];
    if (D >= 0 && D <= p.max_demand_mqps) {
      st = LOKI_LEVEL_FEASIBLE;
      dem[0] = D;
#pragma unroll
      for (int i = 1; i < kMaxTasks; ++i) {
        if (i < p.T) {
          int64_t up = 0;
#pragma unroll
          for (int j = 0; j < kMaxTasks - 1; ++j)
            if (j == p.parent[i]) up = dem[j];
          dem[i] = ceil_div_pos(up * (int64_t)p.fanout_milli[i], 1000);
        }
      }
    }
    status[l] = st;
  }
#pragma unroll
  for (int i = 0; i < kMaxTasks; ++i) {
    if (i < p.T) {
      const int64_t d = st == LOKI_LEVEL_FEASIBLE ? dem[i] : 0;
      if (l < n_levels) dem64[(size_t)l * kMaxTasks + i] = d;
      if (demf != nullptr) {
        // direct path: clamp to the per-task cap above which every option of the
        // task already needs more than S workers (keeps the level infeasible and
        // the packed key inside 32 bits); exact as a double (cap < 2^53);
        // tile-major layout [tile][level pair][task][2], or (tile < 0) the direct kernel's groups
        const int64_t cap = dem_cap[i];
        const int tl = tile < 0 ? -tile : tile;
        const int ll = l % tl;
        size_t at;
        if (tile < 0)
          at = (size_t)(l / tl) * (size_t)((tl + direct_group_levels(p.T) - 1) / direct_group_levels(p.T) * direct_group_stride(p.T)) +
               (size_t)direct_dem_offset(p.T, ll, i);
        else
          at = (size_t)(l / tl) * tl * p.T + ((size_t)(ll >> 1) * p.T + i) * 2 + (ll & 1);
        demf[at] = (double)(d > cap ? cap : d);
      }
    }
  }
}

// ---- K1 (generic): thread <-> candidate, kGenericLevelGroup levels per decode ----
// Templated on the number of tasks so that the per-task arrays live in registers.
template <int T>
__global__ void __launch_bounds__(kGenericThreads)
generic_score_kernel(const __grid_constant__ DevProblem p, const int64_t* __restrict__ dem64,
                     const int32_t* __restrict__ status, int n_levels, Key* __restrict__ partial) {
  constexpr int LG = kGenericLevelGroup;
  const int l0 = blockIdx.y * LG;
  __shared__ int64_t s_dem[LG][kMaxTasks];
  __shared__ int s_live[LG];
  __shared__ Key s_red[LG][kGenericThreads / 32];
  if (threadIdx.x < LG * kMaxTasks) {
    const int g = threadIdx.x / kMaxTasks, i = threadIdx.x % kMaxTasks;
    const int l = l0 + g;
    s_dem[g][i] = (l < n_levels && i < T) ? dem64[(size_t)l * kMaxTasks + i] : 0;
    if (i == 0) s_live[g] = (l < n_levels && status[l] == LOKI_LEVEL_FEASIBLE) ? 1 : 0;
  }
  __syncthreads();
  bool any_live = false;
  for (int g = 0; g < LG; ++g) any_live |= s_live[g] != 0;

  double b_acc[LG];
  int64_t b_w[LG], b_c[LG];
#pragma unroll
  for (int g = 0; g < LG; ++g) { b_acc[g] = 0.0; b_w[g] = 0; b_c[g] = -1; }

  if (any_live) {
    const int64_t chunk = (p.N + gridDim.x - 1) / gridDim.x;
    const int64_t cb = chunk * blockIdx.x;
    const int64_t ce = cb + chunk < p.N ? cb + chunk : p.N;
    for (int64_t c = cb + threadIdx.x; c < ce; c += kGenericThreads) {
      // a1: mixed-radix decode, task 0 least significant
      const OptRec* rec[kMaxTasks];
      if (p.N <= 0xFFFFFFFFLL) {
        uint32_t rem = (uint32_t)c;
#pragma unroll
        for (int i = 0; i < T; ++i) {
          const uint32_t Oi = (uint32_t)p.O[i];
          const uint32_t q = rem / Oi;
          rec[i] = p.opts + LOKI_IDX(p.opt_off[i] + (rem - q * Oi), p.n_opts, kSiteOption, p.debug_flags);
          rem = q;
        }
      } else {
        uint64_t rem = (uint64_t)c;
#pragma unroll
        for (int i = 0; i < T; ++i) {
          const uint64_t Oi = (uint64_t)p.O[i];
          const uint64_t q = rem / Oi;
          rec[i] = p.opts + LOKI_IDX(p.opt_off[i] + (rem - q * Oi), p.n_opts, kSiteOption, p.debug_flags);
          rem = q;
        }
      }
      // a2/a3: path accuracy products in task order, path latency per leaf
      double pp[kMaxTasks];
      int64_t lat[kMaxTasks];
#pragma unroll
      for (int i = 0; i < T; ++i) {
        const double a = rec[i]->acc;
        lat[i] = rec[i]->lat;
        double up = 1.0;                       // pp[parent[i]], picked without dynamic indexing
#pragma unroll
        for (int j = 0; j < T; ++j)
          if (j < i && j == p.parent[i]) up = pp[j];
        pp[i] = i == 0 ? a : __dmul_rn(up, a);
      }
      double sum = 0.0;
      bool lat_ok = true;
      for (int k = 0; k < p.n_leaves; ++k) {
        double v = 0.0;
#pragma unroll
        for (int j = 0; j < T; ++j)
          if (j == p.leaf_task[k]) v = pp[j];
        sum = k == 0 ? v : __dadd_rn(sum, v);
        int64_t pl = 0;
#pragma unroll
        for (int i = 0; i < T; ++i)
          if ((p.path_mask[k] >> i) & 1u) pl += lat[i];
        lat_ok &= pl <= p.lat_limit[k];
      }
      if (!lat_ok) continue;
      const double acc = __ddiv_rn(sum, (double)p.n_leaves);
      // reciprocals of this candidate's divisors, shared by the levels of the group
      double inv[kMaxTasks][2];
#pragma unroll
      for (int i = 0; i < T; ++i) {
        inv[i][0] = __drcp_rn((double)rec[i]->den[0]);
        inv[i][1] = __drcp_rn((double)rec[i]->den[1]);
      }
      // a5-a7: workers, cluster bound, running argmax per level
#pragma unroll
      for (int g = 0; g < LG; ++g) {
        if (!s_live[g]) continue;
        int64_t W = 0;
        int64_t demv[kMaxTasks];
#pragma unroll
        for (int i = 0; i < T; ++i) {
          int64_t d = s_dem[g][i];
          if (p.variant_fanout && i > 0) {
            // a4 with per-variant factors: parent demand x edge factor x the
            // share-weighted factor of the parent's chosen option (in sixteenths)
            int64_t dem_up = 0, vf_up = 0;
#pragma unroll
            for (int j = 0; j < T; ++j)
              if (j < i && j == p.parent[i]) { dem_up = demv[j]; vf_up = (int64_t)rec[j]->vf16; }
            d = ceil_div_pos(dem_up * (int64_t)p.fanout_milli[i] * vf_up, 16000000);
          }
          demv[i] = d;
          W += ceil_div_est(d * rec[i]->mult[0], rec[i]->den[0], inv[i][0]);
          if (rec[i]->parts == 2) W += ceil_div_est(d * rec[i]->mult[1], rec[i]->den[1], inv[i][1]);
        }
        if (W > p.S) continue;
        if (b_c[g] < 0 || acc > b_acc[g] || (acc == b_acc[g] && W < b_w[g])) {
          b_acc[g] = acc; b_w[g] = W; b_c[g] = c;   // c ascends within a thread: ties keep the earlier
        }
      }
    }
  }
  // a8: block argmax per level (warp shuffles, then shared memory across warps)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int g = 0; g < LG; ++g) {
    Key k;
    k.acc_bits = b_c[g] < 0 ? 0ull : (uint64_t)__double_as_longlong(b_acc[g]);
    k.tail = b_c[g] < 0 ? 0ull
                        : (((uint64_t)(p.S - b_w[g])) << 40) | (uint64_t)(p.N - 1 - b_c[g]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      Key o;
      o.acc_bits = __shfl_xor_sync(0xFFFFFFFFu, k.acc_bits, off);
      o.tail = __shfl_xor_sync(0xFFFFFFFFu, k.tail, off);
      if (key_less(k, o)) k = o;
    }
    if (lane == 0) s_red[g][warp] = k;
  }
  __syncthreads();
  if (threadIdx.x < LG) {
    const int g = threadIdx.x;
    Key k = s_red[g][0];
    for (int w = 1; w < kGenericThreads / 32; ++w)
      if (key_less(k, s_red[g][w])) k = s_red[g][w];
    const int l = l0 + g;
    if (l < n_levels)   // [level][block]
      partial[LOKI_IDX((size_t)l * gridDim.x + blockIdx.x, p.partial_keys, kSitePartial, p.debug_flags)] = k;
  }
}

// ---- K2 + K3: deterministic cross-block reduction and winner decode, one block per level ----
// Keys carry the candidate index, so they are totally ordered and the maximum is
// the same bits whatever the order of the comparisons.  `partial` is [level][n_parts]: a level's
// keys lie in a row.  tile_levels > 0: it holds several level tiles back to back, each
// [tile_levels][n_parts]; level `local` is row local % tile_levels of tile local / tile_levels.
// grid.y: latency SLOs of a sweep solved in one scoring launch.  SLO s reads the keys at
// partial + s * slo_keys, takes zero_key[s] for zero-demand levels, and writes final_key and out
// at + s * slo_levels (the plans of SLO s follow those of SLO s - 1).
__global__ void __launch_bounds__(kFinishThreads)
finish_kernel(const __grid_constant__ DevProblem p, const Key* __restrict__ partial, int n_parts,
              int tile_levels, int level_begin, int n_levels_here,
              const int64_t* __restrict__ demand, const Key* __restrict__ zero_key,
              Key* __restrict__ final_key, loki_config_t* __restrict__ out,
              long long slo_keys, int slo_levels) {
  const int local = blockIdx.x;
  if (local >= n_levels_here) return;
  const int slo = blockIdx.y;
  partial += (size_t)slo * (size_t)slo_keys;
  if (zero_key != nullptr) zero_key += slo;
  if (final_key != nullptr) final_key += (size_t)slo * (size_t)slo_levels;
  if (out != nullptr) out += (size_t)slo * (size_t)slo_levels;
  const int within = tile_levels > 0 ? local % tile_levels : local;
  if (tile_levels > 0) partial += (size_t)(local / tile_levels) * (size_t)tile_levels * (size_t)n_parts;
#ifdef LOKI_DEBUG
  {
    const size_t tile_off = tile_levels > 0 ? (size_t)(local / tile_levels) * (size_t)tile_levels * (size_t)n_parts : 0;
    (void)LOKI_IDX((size_t)blockIdx.y * (size_t)slo_keys + tile_off + (size_t)within * n_parts + n_parts - 1,
                   p.partial_keys, kSitePartial, p.debug_flags);
  }
#endif
  Key k = block_max_key<kFinishThreads>(partial + (size_t)within * n_parts, n_parts, 1, 0);
  if (threadIdx.x == 0) {
    const int l = level_begin + local;
    // a zero-demand level needs no workers whatever the plan: its answer is the
    // demand-free one computed once at create time
    if (zero_key != nullptr && demand[l] == 0) k = *zero_key;
    if (final_key != nullptr) final_key[l] = k;
    if (out != nullptr) decode_level(p, k, demand[l], l, out);
  }
}

}  // namespace

cudaError_t launch_option_accuracy(OptRec* d_opts, int64_t n, const double* d_variant_acc,
                                   cudaStream_t st) {
  option_accuracy_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(d_opts, n, d_variant_acc);
  return cudaGetLastError();
}

cudaError_t launch_prepare_levels(const DevProblem& p, const int64_t* d_demand, int n_levels,
                                  int64_t* d_dem64, int32_t* d_status, const int64_t* d_dem_cap,
                                  double* d_demf, int tile, cudaStream_t st, uint32_t* d_zero_words,
                                  int n_zero_words) {
  if (tile == 0) tile = 1;
  const int tl = tile < 0 ? -tile : tile;
  int n_padded = n_levels;
  if (d_demf != nullptr) n_padded = (n_levels + tl - 1) / tl * tl;
  prepare_levels_kernel<<<(n_padded + 127) / 128, 128, 0, st>>>(p, d_demand, n_levels, n_padded,
                                                                d_dem64, d_status, d_dem_cap,
                                                                d_demf, tile, d_zero_words, n_zero_words);
  return cudaGetLastError();
}

cudaError_t launch_generic_score(const DevProblem& p, const int64_t* d_dem64, const int32_t* d_status,
                                 int n_levels, int n_blocks_x, Key* d_partial, cudaStream_t st) {
  dim3 grid((unsigned)n_blocks_x, (unsigned)((n_levels + kGenericLevelGroup - 1) / kGenericLevelGroup));
  switch (p.T) {
#define LOKI_GENERIC_CASE(N)                                                                        \
    case N:                                                                                         \
      generic_score_kernel<N><<<grid, kGenericThreads, 0, st>>>(p, d_dem64, d_status, n_levels,     \
                                                                d_partial);                        \
      break;
    LOKI_GENERIC_CASE(1) LOKI_GENERIC_CASE(2) LOKI_GENERIC_CASE(3) LOKI_GENERIC_CASE(4)
    LOKI_GENERIC_CASE(5) LOKI_GENERIC_CASE(6) LOKI_GENERIC_CASE(7) LOKI_GENERIC_CASE(8)
#undef LOKI_GENERIC_CASE
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_finish(const DevProblem& p, const Key* d_partial, int n_parts, int tile_levels,
                          int level_begin, int n_levels_here, const int64_t* d_demand, const Key* d_zero_key,
                          Key* d_final, loki_config_t* d_out, cudaStream_t st, int n_slos, long long slo_keys,
                          int slo_levels) {
  if (n_slos < 1 || n_slos > 65535) return cudaErrorInvalidValue;
  finish_kernel<<<dim3(n_levels_here, n_slos), kFinishThreads, 0, st>>>(p, d_partial, n_parts, tile_levels,
                                                                        level_begin, n_levels_here, d_demand,
                                                                        d_zero_key, d_final, d_out, slo_keys,
                                                                        slo_levels);
  return cudaGetLastError();
}

}  // namespace loki
