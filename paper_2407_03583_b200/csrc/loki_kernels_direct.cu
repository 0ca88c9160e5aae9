// The direct scoring kernel of libloki_alloc: every (candidate, demand level)
// pair of a latency-feasible candidate is scored with the full per-task worker
// arithmetic.  Hand-written CUDA for sm_100a; bound by the FP64 pipe (one fused
// multiply-add per option part and pair), not by memory.
//
// Workers (Eq. 2 with Eq. 5 of the paper): ceil(dem * p / q) with p / q =
// share * lat / (16 * batch * 1e9) is evaluated as 1 + floor(dem * r), r the
// largest double strictly below p / q.  One fma rounded toward minus infinity,
// fma.rm(dem, r, acc) with acc an integer-valued double in [2^52, 2^53), returns
// acc + floor(dem * r) exactly: the product is formed without rounding and the
// result's unit in the last place is 1.  Chaining the fmas of all parts sums the
// floors in the low mantissa word.  dem * r is below the true value by e with
// 0 < e <= dem * 2^-s (r = M * 2^-s, M a 53-bit integer), and the host has
// checked dem_max * q < 2^s, so e < 1/q and the floor lands exactly one below
// the ceiling for every dem >= 1.
//
// Mapping.  Candidates are grouped into class tuples: per task, options with
// bit-identical task accuracy form a class, so all candidates of a class tuple
// have the same end-to-end accuracy and compete on workers alone.  One warp per
// block.  A warp takes work units (runs of 32-candidate batches) from a counter;
// for every batch it decodes one candidate per lane, applies the latency bound of
// Eqs. 6-7, and packs the constants of the candidates that pass into rows of a
// shared-memory stage (a row holds 32 candidates, one per lane).  When the stage is
// full, or the class tuple ends, the rows are scored against the demand levels of
// the tile, G levels at a time: the group's G x T stage demands are read from
// constant memory at a warp-uniform address and are loop-invariant operands of the
// loop over the staged rows (at most 30 doubles, which is what the compiler keeps
// in uniform registers: an fma with a uniform source issues at the FP64 pipe's full
// rate, with three register sources at two thirds of it).  Per pair the loop costs
// the fmas of the option parts and one unsigned minimum: the key of the running
// best is the worker sum alone.  After a group's loop the warp's minimum per level
// goes to a small shared array; at the end of the class tuple it is merged into a
// lane-distributed running best that carries the accuracy.  Which of the candidates
// with the winning worker sum has the lowest index is decided after the cross-block
// reduction, by the finishing kernel, which re-scores the class tuples with the
// winning accuracy for that one level (a few thousand candidates per level).
//
// Because every staged candidate passed the latency bound, the fmas executed are
// those of latency-feasible pairs (plus the copies that pad a ragged last row and
// the levels that pad the tile to whole groups).
#include "loki_finish.cuh"


// Demand operands of the current tile, group by group (direct_dem_offset).
__constant__ __align__(16) double loki_direct_dem[loki::kDirectMaxTile * loki::kMaxTasks];

namespace loki {

namespace {

// Doubles staged per candidate: one per option part, plus (split options) the start
// value of the accumulator, which carries the number of real parts.
__host__ __device__ constexpr int stage_doubles(int T, int NP) { return T * NP + (NP == 2 ? 1 : 0); }

// Value equal in all lanes, made so for the compiler: a warp reduction's result
// lives in a uniform register, so control flow that depends on it is uniform.
__device__ __forceinline__ uint32_t uniform(uint32_t x) { return __reduce_max_sync(0xFFFFFFFFu, x); }

// One pass over the staged rows for a group of GL levels (a5-a7): the group's GL x T stage demands
// come from constant memory at a warp-uniform address and stay resident as operands of the loop over
// the rows; the warp's fewest workers per level go to wmin[0 .. GL).
template <int T, int NP, int GL>
__device__ __forceinline__ void score_group(const double* s_stage, const double* dem_group, uint32_t* wmin,
                                            uint32_t n_rows, int lane) {
  constexpr int SD = stage_doubles(T, NP);
  const double2* dp = reinterpret_cast<const double2*>(dem_group);
  double dem[GL * T + 1];
#pragma unroll
  for (int e = 0; e < (GL * T + 1) / 2; ++e) {
    const double2 v = dp[e];
    dem[2 * e] = v.x;
    dem[2 * e + 1] = v.y;
  }
  uint32_t b[GL];
#pragma unroll
  for (int g = 0; g < GL; ++g) b[g] = kEmpty;
  const uint32_t n_pairs = n_rows >> 1;               // rows are scored two at a time, an odd last one alone
  uint32_t off = (uint32_t)lane;
#pragma unroll 1
  for (uint32_t k = 0; k < n_pairs; ++k, off += 2u * (uint32_t)(SD * 32)) {
    double ra[SD], rb[SD];
#pragma unroll
    for (int q = 0; q < SD; ++q) { ra[q] = s_stage[off + q * 32]; rb[q] = s_stage[off + (SD + q) * 32]; }
#pragma unroll
    for (int g = 0; g < GL; ++g) {
      // every single option has one real part: the "1 +" of its ceiling is in the start value
      double acc_a = NP == 2 ? ra[SD - 1] : kMagic + (double)T;
      double acc_b = NP == 2 ? rb[SD - 1] : kMagic + (double)T;
#pragma unroll
      for (int q = 0; q < T * NP; ++q) {
        acc_a = __fma_rd(dem[g * T + q / NP], ra[q], acc_a);
        acc_b = __fma_rd(dem[g * T + q / NP], rb[q], acc_b);
      }
      b[g] = __vimin3_u32(b[g], (uint32_t)__double2loint(acc_a), (uint32_t)__double2loint(acc_b));
    }
  }
  if (n_rows & 1u) {
    double ra[SD];
#pragma unroll
    for (int q = 0; q < SD; ++q) ra[q] = s_stage[off + q * 32];
#pragma unroll
    for (int g = 0; g < GL; ++g) {
      double acc_a = NP == 2 ? ra[SD - 1] : kMagic + (double)T;
#pragma unroll
      for (int i = 0; i < T; ++i)
#pragma unroll
        for (int s = 0; s < NP; ++s) acc_a = __fma_rd(dem[g * T + i], ra[i * NP + s], acc_a);
      b[g] = min(b[g], (uint32_t)__double2loint(acc_a));
    }
  }
  // one shared-memory atomic of all lanes per level: cheaper than a warp reduction followed by a
  // read, a minimum and a write
#pragma unroll
  for (int g = 0; g < GL; ++g) atomicMin(wmin + g, b[g]);
}

// Resident blocks per SM the compiler is asked to leave registers for.  Four single-option tasks
// would otherwise take 162 registers (12 blocks per SM: a quarter slower on a four-task tree);
// the other instantiations are left alone: the five-task one fits 128 registers by itself and
// runs a third slower with the bound, whose only effect there is a different schedule.
__host__ __device__ constexpr int direct_min_blocks(int T, int NP) { return T == 4 && NP == 1 ? 16 : 0; }      // 0: no request

// n_groups groups of levels are scored: G = direct_group_levels(T) each, the last one last_gl.
template <int T, int NP>
__global__ void __launch_bounds__(32, direct_min_blocks(T, NP))
direct_score_kernel(const __grid_constant__ DirProblem p, Key* __restrict__ partial,
                    uint32_t* __restrict__ unit_counter, unsigned long long* __restrict__ rows_scored,
                    int stage_rows, int n_groups, int last_gl, uint32_t n_units) {
  using Rec = UniRec<NP>;
  constexpr int SD = stage_doubles(T, NP);
  constexpr int G = direct_group_levels(T);
  constexpr int NB = kDirectMaxTile / 32;     // running-best slots per lane
  const int lane = threadIdx.x;
  const int tile_lv = (n_groups - 1) * G + last_gl;     // levels scored
  extern __shared__ __align__(16) double s_stage[];                              // [stage_rows][SD][32]
  uint32_t* const s_wmin = reinterpret_cast<uint32_t*>(s_stage + (size_t)stage_rows * SD * 32);   // [tile_lv]
#ifdef LOKI_DEBUG
  if (lane == 0 && (size_t)stage_rows * SD * 32 * sizeof(double) + (size_t)tile_lv * sizeof(uint32_t) > loki_dynamic_smem_bytes())
    (void)LOKI_IDX(-1, 0, kSiteSharedLayout, p.debug_flags);
#endif
  for (int l = lane; l < tile_lv; l += 32) s_wmin[l] = kEmpty;
  __syncwarp();

  uint64_t rb_acc[NB];                        // level b * 32 + lane: best (accuracy, workers) so far ...
  uint32_t rb_w[NB], rb_ct[NB];               // ... and a class tuple that attains it
#pragma unroll
  for (int b = 0; b < NB; ++b) { rb_acc[b] = 0; rb_w[b] = 0; rb_ct[b] = 0; }

  const Rec* const recs = reinterpret_cast<const Rec*>(p.uni_members);
  const uint32_t jbits = (uint32_t)p.jbits;
  const uint32_t stage_cap = (uint32_t)(stage_rows - 1) * 32u;   // a step is staged while at most this many wait
  uint32_t staged = 0;                        // candidates waiting in the stage (uniform)

  for (;;) {
    uint32_t u = 0;
    if (lane == 0) u = atomicAdd(unit_counter, 1u);
    u = uniform(u);
    if (u >= n_units) break;
    uint32_t it = uniform(p.unit_start[u]);
    const uint32_t it_end = uniform(p.unit_start[u + 1]);
    // class tuple holding column batch `it`: largest ct with prefix[ct] <= it
    uint32_t ct;
    {
      uint32_t lo = 0, hi = (uint32_t)p.n_ct;     // invariant: prefix[lo] <= it < prefix[hi]
      while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (p.iter_prefix[mid] <= (uint64_t)it) lo = mid; else hi = mid;
      }
      ct = uniform(lo);
    }
    while (it < it_end) {
      // ---- class tuple set-up.  A column is a choice of members for tasks 1 .. T-1; the members
      //      of task 0 are walked step by step, so a column is decoded once for all of them.
      //      (One task: the "columns" are the lanes, a step is 32 members.) ----
      uint32_t cnt[T], inv[T], mem_base[T];
      uint32_t n_cols = 1;
      int32_t min_lat0;
      {
        uint32_t r = ct;
#pragma unroll
        for (int i = 0; i < T; ++i) {
          const uint32_t nc = (uint32_t)p.n_class[i];
          const uint32_t cls = r % nc;
          r /= nc;
          const int idx = (int)LOKI_IDX(p.class_off[i] + (int)cls, p.n_classes, kSiteClass, p.debug_flags);
          cnt[i] = (uint32_t)p.class_count[idx];
          inv[i] = 0xFFFFFFFFu / cnt[i] + 1u;     // x / cnt == umulhi(x, inv) while x * cnt < 2^32
          mem_base[i] = (uint32_t)p.member_off[i] + (uint32_t)p.class_first[idx];
          if (i > 0) n_cols *= cnt[i];
          if (i == 0) min_lat0 = p.class_min_lat[idx];
        }
      }
      const uint32_t n_steps = uniform(T == 1 ? (cnt[0] + 31u) >> 5 : cnt[0]);
      (void)LOKI_IDX(ct, p.n_ct, kSiteClassTuple, p.debug_flags);
      const uint64_t acc_bits = p.ct_acc[ct];     // a2: path products and leaf mean, computed at create
      const uint32_t ct_first = (uint32_t)p.iter_prefix[ct];
      const uint32_t ct_iters = (uint32_t)p.iter_prefix[ct + 1] - ct_first;
      uint32_t cb = uniform(it - ct_first);       // column batch within the class tuple
      const uint32_t cb_end = uniform(ct_iters - cb < it_end - it ? ct_iters : cb + (it_end - it));
      it += cb_end - cb;

      uint32_t step = 0;
      double col_vals[SD];                        // this lane's column: constants of tasks 1 .. T-1
      uint32_t col_nsh = 0;
      int32_t slack = -1;                         // what the column leaves of the tightest latency bound
      bool col_valid = false;
      while (cb < cb_end) {
        // ---- a1 + a3: stage the candidates within the latency bound, one step of task 0 at a time ----
        while (staged <= stage_cap && cb < cb_end) {
          if (step == 0) {
            const uint32_t col = cb * 32u + (uint32_t)lane;
            col_valid = T == 1 ? true : col < n_cols;
            int32_t lat[T];
            lat[0] = 0;
            col_nsh = 0;
            uint32_t r = col_valid ? col : 0u;
#pragma unroll
            for (int i = 1; i < T; ++i) {
              const uint32_t q = __umulhi(r, inv[i]);
              const uint32_t dgt = r - q * cnt[i];
              r = q;
              const Rec rec = recs[LOKI_IDX(mem_base[i] + dgt, p.n_members, kSiteMember, p.debug_flags)];
              col_vals[i * NP] = rec.r[0];
              if (NP == 2) col_vals[i * NP + NP - 1] = rec.r[NP - 1];
              lat[i] = rec.lat;
              col_nsh += rec.nsh;
            }
            slack = 0x7FFFFFFF;
            for (int k = 0; k < p.n_leaves; ++k) {
              int32_t pl = 0;
#pragma unroll
              for (int i = 1; i < T; ++i)
                if ((p.path_mask[k] >> i) & 1u) pl += lat[i];
              slack = min(slack, p.lat_limit[k] - pl);      // the root is on every path
            }
            // a column batch none of whose columns leaves room for task 0's fastest member is skipped
            if (__ballot_sync(0xFFFFFFFFu, col_valid && slack >= min_lat0) == 0u) { ++cb; continue; }
          }
          const uint32_t d0 = T == 1 ? step * 32u + (uint32_t)lane : step;
          const bool in_class = T == 1 ? d0 < cnt[0] : true;
          const Rec rec0 = recs[LOKI_IDX(mem_base[0] + (in_class ? d0 : 0u), p.n_members, kSiteMember, p.debug_flags)];
          const bool alive = col_valid && in_class && rec0.lat <= slack;
          const uint32_t mask = __ballot_sync(0xFFFFFFFFu, alive);
          if (alive) {
            const uint32_t pos = (uint32_t)LOKI_IDX(staged + (uint32_t)__popc(mask & ((1u << lane) - 1u)),
                                                    (uint32_t)stage_rows * 32u, kSiteDirectStage, p.debug_flags);
            double* dst = s_stage + (pos >> 5) * (uint32_t)(SD * 32) + (pos & 31u);
            dst[0] = rec0.r[0];
            if (NP == 2) dst[32] = rec0.r[NP - 1];
#pragma unroll
            for (int q = NP; q < T * NP; ++q) dst[q * 32] = col_vals[q];
            // split options: the start value carries the number of real parts (exact: a small integer onto ulp 1)
            if (NP == 2) dst[(SD - 1) * 32] = kMagic + (double)((col_nsh + rec0.nsh) >> jbits);
          }
          staged += (uint32_t)__popc(mask);
          if (++step == n_steps) { step = 0; ++cb; }
        }
        if (staged == 0) continue;
        // ---- a5-a7: score the staged rows against every level of the tile ----
        // whole rows only while the class tuple goes on: the candidates of a partly filled last
        // row wait for the next pass
        const bool last_pass = cb >= cb_end;
        const uint32_t rem = staged & 31u;
        const uint32_t n_rows = last_pass ? (staged + 31u) >> 5 : staged >> 5;
        __syncwarp();
        if (last_pass && rem != 0 && (uint32_t)lane >= rem) {
          // ragged last row: the free lanes take a copy of the row's first candidate
          // (a copy cannot change a minimum)
          double* row = s_stage + (n_rows - 1) * (uint32_t)(SD * 32);
#pragma unroll
          for (int q = 0; q < SD; ++q) row[q * 32 + lane] = row[q * 32];
        }
        __syncwarp();
        if (lane == 0) atomicAdd(rows_scored, (unsigned long long)n_rows);
#pragma unroll 1
        for (int lg = 0; lg < n_groups; ++lg) {
          const double* dem = loki_direct_dem + LOKI_IDX(lg * direct_group_stride(T), kDirectMaxTile * kMaxTasks - direct_group_stride(T) + 1,
                                                         kSiteDemandTile, p.debug_flags);
          uint32_t* wmin = s_wmin + LOKI_IDX(lg * G, tile_lv, kSiteDirectWmin, p.debug_flags);
          if (lg + 1 < n_groups || last_gl == G) score_group<T, NP, G>(s_stage, dem, wmin, n_rows, lane);
          else if (last_gl == direct_short_group(T, 1)) score_group<T, NP, direct_short_group(T, 1)>(s_stage, dem, wmin, n_rows, lane);
          else score_group<T, NP, direct_short_group(T, 2)>(s_stage, dem, wmin, n_rows, lane);
        }
        __syncwarp();
        if (!last_pass && rem != 0) {
          // the waiting candidates move to the first row
          if ((uint32_t)lane < rem) {
            const double* row = s_stage + n_rows * (uint32_t)(SD * 32);
#pragma unroll
            for (int q = 0; q < SD; ++q) s_stage[q * 32 + lane] = row[q * 32 + lane];
          }
          __syncwarp();
          staged = rem;
        } else {
          staged = 0;
        }
      }

      // ---- end of this warp's share of the class tuple: merge its fewest workers per level
      //      into the running best (a6: cluster bound) ----
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        const int l = b * 32 + lane;
        if (l >= tile_lv) continue;
        const uint32_t W = s_wmin[l];
        s_wmin[l] = kEmpty;
        if (W > (uint32_t)p.S) continue;        // also the empty pattern
        if (acc_bits > rb_acc[b] || (acc_bits == rb_acc[b] && W < rb_w[b])) { rb_acc[b] = acc_bits; rb_w[b] = W; rb_ct[b] = ct; }
      }
      __syncwarp();
      ct = ct + 1;
    }
  }

  // ---- a8: one partial key per (warp, level): accuracy, then workers; the index part names a
  //      class tuple that attains them (any one: the finishing kernel finds the others with the
  //      same accuracy and puts the winning candidate's index there) ----
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const int l = b * 32 + lane;
    if (l < tile_lv) {
      Key k{0ull, 0ull};
      if (rb_acc[b] != 0) {
        k.acc_bits = rb_acc[b];
        k.tail = ((uint64_t)((uint32_t)p.S - rb_w[b]) << 40) | (uint64_t)rb_ct[b];
      }
      // [level][block]: the finishing kernel reads a level's keys in a row
      partial[LOKI_IDX((size_t)l * gridDim.x + blockIdx.x, p.partial_keys, kSitePartial, p.debug_flags)] = k;
    }
  }
}

// a2 for every class tuple: path products in task order and the mean over the leaves
// (no fused multiply-add), one thread per class tuple.
__global__ void class_tuple_accuracy_kernel(DirProblem p, uint64_t* __restrict__ ct_acc) {
  const int64_t ct = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (ct >= p.n_ct) return;
  double pp[kMaxTasks];
  uint64_t r = (uint64_t)ct;
  for (int i = 0; i < p.T; ++i) {
    const uint32_t nc = (uint32_t)p.n_class[i];
    const double a = p.class_acc[p.class_off[i] + (int)(r % nc)];
    r /= nc;
    pp[i] = i == 0 ? a : __dmul_rn(pp[p.parent[i]], a);
  }
  double sum = pp[p.leaf_task[0]];
  for (int k = 1; k < p.n_leaves; ++k) sum = __dadd_rn(sum, pp[p.leaf_task[k]]);
  ct_acc[ct] = (uint64_t)__double_as_longlong(__ddiv_rn(sum, (double)p.n_leaves));
}

// Lowest candidate index among the candidates of class tuple `ct` that pass the latency
// bound and need exactly `W` workers at the demands `dem` (one level): the direct kernel's
// own arithmetic, candidate by candidate.  Called by all threads of a block; the block-wide
// result goes to *s_min (shared, initialised by the caller).
template <int T>
__device__ void lowest_index_in_class_tuple(const DirProblem& p, uint32_t ct, const double* dem,
                                            uint32_t W, unsigned long long* s_min) {
  uint32_t cnt[T], inv[T], mem_base[T];
  uint32_t J = 1;
  uint32_t r = ct;
#pragma unroll
  for (int i = 0; i < T; ++i) {
    const uint32_t nc = (uint32_t)p.n_class[i];
    const uint32_t cls = r % nc;
    r /= nc;
    const int idx = (int)LOKI_IDX(p.class_off[i] + (int)cls, p.n_classes, kSiteClass, p.debug_flags);
    cnt[i] = (uint32_t)p.class_count[idx];
    inv[i] = 0xFFFFFFFFu / cnt[i] + 1u;           // x / cnt == umulhi(x, inv) while x * cnt < 2^32
    mem_base[i] = (uint32_t)p.member_off[i] + (uint32_t)p.class_first[idx];
    J *= cnt[i];
  }
  unsigned long long mine = ~0ull;
  for (uint32_t j = threadIdx.x; j < J; j += blockDim.x) {
    uint32_t rr = j;
    double acc = kMagic;
    int32_t lat[T];
    int64_t c = 0;
#pragma unroll
    for (int i = 0; i < T; ++i) {
      const uint32_t q = __umulhi(rr, inv[i]);
      const uint32_t d = rr - q * cnt[i];
      rr = q;
      const DirRec& rec = p.members[LOKI_IDX(mem_base[i] + d, p.n_members, kSiteMember, p.debug_flags)];
      lat[i] = rec.lat;
      acc = __dadd_rn(acc, (double)rec.n_real);
      acc = __fma_rd(dem[i], rec.r[0], acc);
      acc = __fma_rd(dem[i], rec.r[1], acc);      // an unused part has r == 0
      c += (int64_t)rec.opt * p.stride[i];
    }
    bool ok = (uint32_t)__double2loint(acc) == W;
    for (int k = 0; k < p.n_leaves; ++k) {
      int32_t pl = 0;
#pragma unroll
      for (int i = 0; i < T; ++i)
        if ((p.path_mask[k] >> i) & 1u) pl += lat[i];
      ok &= pl <= p.lat_limit[k];
    }
    if (ok && (unsigned long long)c < mine) mine = (unsigned long long)c;
  }
  if (mine != ~0ull) atomicMin(s_min, mine);
}

// a9 + a10 for the direct kernel's keys, one block per level: maximum over the partial keys
// (accuracy, then fewest workers), then the lowest candidate index that attains it -- every
// class tuple with the winning accuracy is re-scored for this level -- then the plan.
template <int T>
__global__ void __launch_bounds__(kDirectFinishThreads)
direct_finish_kernel(const __grid_constant__ DirProblem p, const __grid_constant__ DevProblem dp,
                     const Key* __restrict__ partial, int n_parts, int level_begin,
                     int n_levels_here, const double* __restrict__ dem_tile,
                     const int64_t* __restrict__ demand, const Key* __restrict__ zero_key,
                     Key* __restrict__ final_key, loki_config_t* __restrict__ out) {
  const int local = blockIdx.x;
  if (local >= n_levels_here) return;
  __shared__ unsigned long long s_min;
  __shared__ double s_dem[kMaxTasks];
  if (threadIdx.x == 0) s_min = ~0ull;
  if (threadIdx.x < T) s_dem[threadIdx.x] = dem_tile[direct_dem_offset(T, local, threadIdx.x)];
  (void)LOKI_IDX((size_t)local * n_parts + n_parts - 1, p.partial_keys, kSitePartial, p.debug_flags);
  Key k = block_max_key<kDirectFinishThreads>(partial + (size_t)local * n_parts, n_parts, 1, 0);   // synchronises the block
  const int l = level_begin + local;
  const bool zero = zero_key != nullptr && demand[l] == 0;
  if (!zero && k.acc_bits != 0) {
    // the key names one class tuple with the winning accuracy; the others, if any, are its
    // neighbours in the table sorted by accuracy bits
    const uint32_t W = (uint32_t)p.S - (uint32_t)(k.tail >> 40);
    const int64_t at = p.ct_rank[LOKI_IDX(k.tail & kIndexMask, p.n_ct, kSiteClassTuple, p.debug_flags)];
    int64_t lo = at, hi = at + 1;
    while (lo > 0 && p.ct_sorted_acc[lo - 1] == k.acc_bits) --lo;
    while (hi < p.n_ct && p.ct_sorted_acc[hi] == k.acc_bits) ++hi;
    for (int64_t e = lo; e < hi; ++e)
      lowest_index_in_class_tuple<T>(p, (uint32_t)LOKI_IDX(p.ct_sorted_idx[e], p.n_ct, kSiteClassTuple, p.debug_flags), s_dem, W, &s_min);
    __syncthreads();
    // a winner always exists, since the key came from a scored candidate; if none is found the
    // index part becomes all ones, which the decode reports as an internal error
    k.tail = (k.tail & ~kIndexMask) | (s_min == ~0ull ? kIndexMask : (uint64_t)(p.N - 1 - (int64_t)s_min));
  }
  if (threadIdx.x == 0) {
    // a zero-demand level needs no workers whatever the plan: its answer is the
    // demand-free one computed once at create time
    if (zero) k = *zero_key;
    final_key[l] = k;
    if (out != nullptr) decode_level(dp, k, demand[l], l, out);
  }
}

size_t direct_smem_bytes(int T, int NP, int stage_rows, int n_groups) {
  return (size_t)stage_rows * stage_doubles(T, NP) * 32 * sizeof(double) +
         (size_t)n_groups * direct_group_levels(T) * sizeof(uint32_t);
}

struct DirectLaunch {
  const DirProblem* p;
  int n_blocks;            // 0: occupancy query
  Key* d_partial;
  uint32_t* d_counter;
  unsigned long long* d_rows;
  int stage_rows, n_groups, last_gl;
  uint32_t n_units;
  cudaStream_t st;
};

template <int T, int NP>
int act(const DirectLaunch& a) {
  auto kern = direct_score_kernel<T, NP>;
  const size_t smem = direct_smem_bytes(T, NP, a.stage_rows, a.n_groups);
  if (a.n_blocks == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, 32, smem) != cudaSuccess) return 0;
    return n;
  }
  kern<<<a.n_blocks, 32, smem, a.st>>>(*a.p, a.d_partial, a.d_counter, a.d_rows, a.stage_rows, a.n_groups, a.last_gl,
                                      a.n_units);
  return (int)cudaGetLastError();
}

template <int NP>
int by_tasks(int T, const DirectLaunch& a) {
  switch (T) {
    case 1: return act<1, NP>(a);
    case 2: return act<2, NP>(a);
    case 3: return act<3, NP>(a);
    case 4: return act<4, NP>(a);
    case 5: return act<5, NP>(a);
    case 6: return act<6, NP>(a);
    case 7: return act<7, NP>(a);
    case 8: return act<8, NP>(a);
    default: return a.n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

int dispatch(int T, int n_parts, const DirectLaunch& a) {
  return n_parts == 2 ? by_tasks<2>(T, a) : by_tasks<1>(T, a);
}

}  // namespace

bool direct_supported(int T, int split) { return T >= 1 && T <= kMaxTasks && (split == 0 || split == 1); }

// Rows of 32 candidates the stage of one warp holds: 12.5 KB, at least two rows (with five
// doubles per candidate ten rows: a pass scores nine whole rows while a tenth fills).
int direct_stage_rows(int T, int n_parts) {
  const int row_bytes = stage_doubles(T, n_parts) * 32 * (int)sizeof(double);
  const int rows = 12800 / row_bytes;
  return rows < 2 ? 2 : rows;
}

cudaError_t direct_upload_tile(const double* d_demf_tile, int n_doubles, cudaStream_t st) {
  return cudaMemcpyToSymbolAsync(loki_direct_dem, d_demf_tile, sizeof(double) * n_doubles, 0,
                                 cudaMemcpyDeviceToDevice, st);
}

cudaError_t launch_direct_score(const DirProblem& p, int tile_levels, int n_blocks, Key* d_partial,
                                uint32_t* d_unit_counter, unsigned long long* d_rows_scored,
                                uint32_t n_units, cudaStream_t st) {
  const int G = direct_group_levels(p.T);
  if (n_blocks < 1 || tile_levels < 1 || tile_levels > kDirectMaxTile ||
      tile_levels != direct_tile_levels(p.T, tile_levels))
    return cudaErrorInvalidValue;
  const int n_groups = (tile_levels - 1) / G + 1;
  const DirectLaunch a{&p, n_blocks, d_partial, d_unit_counter, d_rows_scored,
                       direct_stage_rows(p.T, p.n_parts_max), n_groups, tile_levels - (n_groups - 1) * G, n_units, st};
  return (cudaError_t)dispatch(p.T, p.n_parts_max, a);
}

// Resident blocks per SM of the instantiation that serves (T, n_parts) with a tile of n_groups groups.
int direct_max_blocks_per_sm(int T, int n_parts, int n_groups) {
  const DirectLaunch a{nullptr, 0, nullptr, nullptr, nullptr, direct_stage_rows(T, n_parts), n_groups, direct_group_levels(T), 0, nullptr};
  return dispatch(T, n_parts, a);
}

cudaError_t launch_class_tuple_accuracy(const DirProblem& p, uint64_t* d_ct_acc, cudaStream_t st) {
  class_tuple_accuracy_kernel<<<(unsigned)((p.n_ct + 127) / 128), 128, 0, st>>>(p, d_ct_acc);
  return cudaGetLastError();
}

cudaError_t launch_direct_finish(const DirProblem& p, const DevProblem& dp, const Key* d_partial, int n_parts,
                                 int level_begin, int n_levels_here,
                                 const double* d_dem_tile, const int64_t* d_demand, const Key* d_zero_key,
                                 Key* d_final, loki_config_t* d_out, cudaStream_t st) {
  switch (p.T) {
#define LOKI_FINISH_CASE(N)                                                                              \
    case N:                                                                                              \
      direct_finish_kernel<N><<<n_levels_here, kDirectFinishThreads, 0, st>>>(                                 \
          p, dp, d_partial, n_parts, level_begin, n_levels_here, d_dem_tile, d_demand,                   \
          d_zero_key, d_final, d_out);                                                                   \
      break;
    LOKI_FINISH_CASE(1) LOKI_FINISH_CASE(2) LOKI_FINISH_CASE(3) LOKI_FINISH_CASE(4)
    LOKI_FINISH_CASE(5) LOKI_FINISH_CASE(6) LOKI_FINISH_CASE(7) LOKI_FINISH_CASE(8)
#undef LOKI_FINISH_CASE
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace loki
