// The level-lane scoring kernel for per-variant multiplicative factors r(i,k)
// (Eq. 1 of the paper: the requests a task forwards depend on the variant that
// served them; Algorithm 1 multiplies multFactor by branchRatio the same way).
// The stage demand of a task then depends on the options chosen for its
// ancestors, so nothing can be computed per level ahead of the candidate.
// Problems without such factors are the special case of one ratio per edge; the
// library serves its level-lane path with this kernel for them as well.
//
// Mapping.  One warp per block, a lane owns LPL demand levels, the candidate is
// the same for the whole warp (as in the level-lane kernel).  The walk nests the
// tasks root first -- task 0 outermost, task T-1 innermost; parents precede
// children because parent[i] < i -- so that when the loop of task i runs, the
// demand of task i at this lane's levels is already fixed by the options of its
// ancestors:
//     dem_i = ceil(dem_parent * fanout_milli[i] * vf16(parent's option) / 16e6)
//           = 1 + floor(dem_parent * r),   r the largest double below that ratio,
// one fma rounded toward minus infinity onto 1.5 * 2^52 and two exact adds, once per
// move of an ancestor's digit; the planner admits the kernel only when the
// rounding of r cannot reach the next integer (the argument of the worker fma, with
// the parent's demand cap as the bound).  Inside the loop of task i each member
// costs one fma per part (the exact worker count 1 + floor(dem * r), as in the
// direct kernel), and the innermost loop scores a pair with that fma, one add and
// one minimum.  A demand above the task's cap (every option
// then needs more than S workers) is clamped: the candidate is infeasible
// whatever its descendants need, and the packed key stays inside 32 bits.
//
// A class is staged in ascending task latency (a member's record carries its own
// digit, folded with the worker count of a real part into one constant, so the order
// is free): a digit loop stops at the first member that does not fit the latency
// slack (Eq. 7), and the innermost loop runs over the fitting prefix with no test.
#include "loki_internal.h"

namespace loki {

namespace {

// Warp-uniform description of a work unit plus, per lane, the demands fixed so far.
template <int T, int NP, int LPL>
struct Walk {
  const UniRec<NP>* rec;     // staged member records, all tasks
  const double* dr;          // staged demand ratios [member][T], same order
  uint32_t cnt[T], roff[T];
  int32_t parent[T];
  double cap[T];             // demand cap of task i
  uint32_t jmul;
  int32_t n_leaves;
  uint32_t path_mask[kMaxTasks];
  // state along the current path of the walk
  double dem[T][LPL];        // this lane's stage demands of the tasks whose ancestors are fixed
  uint32_t row_of[T];        // row (first word) of the demand ratios of the member chosen for task i
};

// Loop of task I (root first).  slack[k]: what tasks 0..I-1 leave of leaf k's latency bound;
// ps: packed-key sum of tasks 0..I-1 at this lane's levels.
// NS: slack slots carried (1 for a chain, 2 for two leaves, else kMaxTasks).
template <int I, int T, int NP, int LPL, int NS>
__device__ __forceinline__ void walk_task(Walk<T, NP, LPL>& wk, uint32_t begin, uint32_t end,
                                          const int32_t (&slack)[NS], const uint32_t (&ps)[LPL],
                                          uint32_t (&best)[LPL]) {
  // a4: this task's demand at the lane's levels, from its parent's demand and chosen option
  double dd[LPL];
  if constexpr (I == 0) {
#pragma unroll
    for (int g = 0; g < LPL; ++g) dd[g] = wk.dem[0][g];
  } else {
    // the parent's row and demand, picked with masks: on a chain the parent is task I - 1; on a tree
    // a compare per ancestor (indexing the per-task arrays with parent[I] would move them out of
    // registers)
    uint32_t row = 0;
#pragma unroll
    for (int j = 0; j < I; ++j) {
      const bool hit = NS == 1 ? j == I - 1 : j == wk.parent[I];
      row |= wk.row_of[j] & (0u - (uint32_t)hit);
    }
    const double r = wk.dr[row + I];
#pragma unroll
    for (int g = 0; g < LPL; ++g) {
      unsigned long long up = 0;
#pragma unroll
      for (int j = 0; j < I; ++j) {
        const bool hit = NS == 1 ? j == I - 1 : j == wk.parent[I];
        up |= (unsigned long long)__double_as_longlong(wk.dem[j][g]) & (0ull - (unsigned long long)hit);
      }
      const double acc = __fma_rd(__longlong_as_double((long long)up), r, kMagic);
      double d = __dadd_rn(__dsub_rn(acc, kMagic), 1.0);      // both exact: integers below 2^51
      d = d > wk.cap[I] ? wk.cap[I] : d;
      wk.dem[I][g] = d;
      dd[g] = d;
    }
  }
  if constexpr (I == T - 1) {
    // innermost task: the members that fit what the outer tasks leave of every path through it
    int32_t via = slack[0];
    if (NS > 1) {
      via = 0x7FFFFFFF;
#pragma unroll
      for (int k = 0; k < NS; ++k)
        if (k < wk.n_leaves && ((wk.path_mask[k] >> I) & 1u)) via = min(via, slack[k]);
    }
    const UniRec<NP>* rp = wk.rec + wk.roff[I];
    uint32_t n = end;
    while (n > begin && rp[n - 1].lat > via) --n;
    rp += begin;
#pragma unroll 4
    for (uint32_t left = n - begin; left > 0; --left, ++rp) {
      const UniRec<NP> rc = *rp;
      // a5 + a6: workers of this member at the lane's levels complete the packed key
#pragma unroll
      for (int g = 0; g < LPL; ++g) {
        double acc = __fma_rd(dd[g], rc.r[0], kMagic);
        if (NP == 2) acc = __fma_rd(dd[g], rc.r[NP - 1], acc);
        best[g] = min(best[g], (uint32_t)__double2loint(acc) * wk.jmul + (ps[g] + rc.nsh));
      }
    }
  } else {
    for (uint32_t m = begin; m < end; ++m) {
      const UniRec<NP> rc = wk.rec[wk.roff[I] + m];
      // a3: latency bound on every path through this task; members come in ascending latency,
      // so once one does not fit none of the later ones does
      int32_t s2[NS];
      int32_t tight = 0x7FFFFFFF;
      if (NS == 1) {                           // a chain: every task is on the one path
        s2[0] = slack[0] - rc.lat;
        tight = s2[0];
      } else {
#pragma unroll
        for (int k = 0; k < NS; ++k) {
          s2[k] = slack[k];
          if (k < wk.n_leaves) {
            if ((wk.path_mask[k] >> I) & 1u) s2[k] -= rc.lat;
            tight = min(tight, s2[k]);
          }
        }
      }
      if (tight < 0) break;
      // a5: workers of this member at the lane's levels, added to the packed key
      uint32_t ps2[LPL];
#pragma unroll
      for (int g = 0; g < LPL; ++g) {
        double acc = __fma_rd(dd[g], rc.r[0], kMagic);
        if (NP == 2) acc = __fma_rd(dd[g], rc.r[NP - 1], acc);
        ps2[g] = ps[g] + (uint32_t)__double2loint(acc) * wk.jmul + rc.nsh;
      }
      wk.row_of[I] = (wk.roff[I] + m) * (uint32_t)T;
      walk_task<I + 1, T, NP, LPL, NS>(wk, 0u, wk.cnt[I + 1], s2, ps2, best);
    }
  }
}

// Dynamic shared memory: 32 header words | member records of the class tuple | their demand ratios.
template <int T, int NP, int LPL, int NS>
__global__ void __launch_bounds__(32)
variant_score_kernel(const __grid_constant__ DirProblem p, const LevelSpan span,
                     Key* __restrict__ partial, int max_members) {
  using Rec = UniRec<NP>;
  constexpr int LT = 32 * LPL;
  constexpr int kHdrWords = 32;
  const int lane = threadIdx.x;
  const int tile_level0 = span.level_begin + (int)blockIdx.y * LT;      // grid.y: consecutive level tiles
  const size_t partial_off = (size_t)blockIdx.y * gridDim.x * LT;
  extern __shared__ __align__(16) unsigned char s_raw[];
  uint32_t* const s_hdr = reinterpret_cast<uint32_t*>(s_raw);
  Rec* const s_rec = reinterpret_cast<Rec*>(s_raw + kHdrWords * 4);
  double* const s_dr = reinterpret_cast<double*>(s_rec + max_members);
  __shared__ double s_pp[kMaxTasks];
#ifdef LOKI_DEBUG
  if (lane == 0 && (size_t)(reinterpret_cast<unsigned char*>(s_dr + (size_t)max_members * T) - s_raw) > loki_dynamic_smem_bytes())
    (void)LOKI_IDX(-1, 0, kSiteSharedLayout, p.debug_flags);
#endif

  Walk<T, NP, LPL> wk;
  wk.rec = s_rec;
  wk.dr = s_dr;
  wk.jmul = 1u << p.jbits;
  wk.n_leaves = p.n_leaves;
#pragma unroll
  for (int k = 0; k < kMaxTasks; ++k) wk.path_mask[k] = p.path_mask[k];
#pragma unroll
  for (int i = 0; i < T; ++i) {
    wk.parent[i] = p.parent[i];
    wk.cap[i] = (double)p.dem_cap[i];
    wk.row_of[i] = 0;
  }
  // a4 for the root: its demand at this lane's levels (levels g * 32 + lane of the tile), clamped to its cap;
  // a level past the end of the sweep or with a demand out of range is scored with zero demand
#pragma unroll
  for (int g = 0; g < LPL; ++g) {
    const int l = tile_level0 + g * 32 + lane;
    int64_t D = l < span.n_levels ? span.demand[l] : 0;
    if (D < 0 || D > p.max_demand_mqps) D = 0;
    const int64_t cap = p.dem_cap[0];
    wk.dem[0][g] = (double)(D > cap ? cap : D);
  }

  uint64_t rb_acc[LPL];
  uint32_t rb_ct[LPL], rb_w[LPL], rb_j[LPL];
#pragma unroll
  for (int g = 0; g < LPL; ++g) { rb_acc[g] = 0; rb_ct[g] = 0; rb_w[g] = 0; rb_j[g] = 0; }

  const uint32_t jbits = (uint32_t)p.jbits;
  const uint32_t jmask = wk.jmul - 1u;
  const Rec* const recs = reinterpret_cast<const Rec*>(p.uni_members);
  const uint32_t SL = (uint32_t)p.uni_slices;
  const uint32_t n_units = (uint32_t)p.n_ct * SL;

  for (uint32_t u = blockIdx.x; u < n_units; u += gridDim.x) {
    const uint32_t ct = u / SL;
    const uint32_t sl = u - ct * SL;
    __syncwarp();
    // ---- stage the class tuple: member records, factors, counts, path accuracy ----
    {
      uint32_t q = ct, off = 0, stride = 1;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        const uint32_t nc = (uint32_t)p.n_class[i];
        const uint32_t cls = q % nc;
        q /= nc;
        const int idx = (int)LOKI_IDX(p.class_off[i] + (int)cls, p.n_classes, kSiteClass, p.debug_flags);
        const uint32_t c = (uint32_t)p.class_count[idx];
        const size_t first = (size_t)p.member_off[i] + (size_t)p.class_first[idx];
        for (uint32_t k = lane; k < c; k += 32) {
          const uint32_t m = (uint32_t)p.lat_order[LOKI_IDX(first + k, p.n_members, kSiteMember, p.debug_flags)];   // the member's own digit
          Rec rc = recs[LOKI_IDX(first + m, p.n_members, kSiteMember, p.debug_flags)];
          rc.nsh += m * stride;                                       // constant part of its key share
          s_rec[LOKI_IDX(off + k, max_members, kSiteVariantStage, p.debug_flags)] = rc;
#pragma unroll
          for (int c2 = 0; c2 < T; ++c2) s_dr[(off + k) * T + c2] = p.uni_dem_r[(first + m) * T + c2];
        }
        if (lane == 0) {
          s_hdr[i] = c;
          s_hdr[8 + i] = off;
          // a2: path accuracy products in task order (no fused multiply-add)
          const double a = p.class_acc[idx];
          s_pp[i] = i == 0 ? a : __dmul_rn(s_pp[p.parent[i]], a);
        }
        off += c;
        stride *= c;
      }
    }
    __syncwarp();
    double sum = s_pp[p.leaf_task[0]];
    for (int k = 1; k < p.n_leaves; ++k) sum = __dadd_rn(sum, s_pp[p.leaf_task[k]]);
    const uint64_t acc_bits = (uint64_t)__double_as_longlong(__ddiv_rn(sum, (double)p.n_leaves));

#pragma unroll
    for (int i = 0; i < T; ++i) {
      wk.cnt[i] = s_hdr[i];
      wk.roff[i] = s_hdr[8 + i];
    }
    // this unit's slice of the outermost digit (task 0)
    const uint32_t d_begin = wk.cnt[0] * sl / SL, d_end = wk.cnt[0] * (sl + 1) / SL;
    if (d_begin >= d_end) continue;

    uint32_t best[LPL], ps[LPL];
#pragma unroll
    for (int g = 0; g < LPL; ++g) { best[g] = kEmpty; ps[g] = 0; }
    int32_t slack[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) slack[k] = k < p.n_leaves ? p.lat_limit[k] : 0x7FFFFFFF;
    walk_task<0, T, NP, LPL, NS>(wk, d_begin, d_end, slack, ps, best);

    // ---- merge this lane's levels into its running best ----
#pragma unroll
    for (int g = 0; g < LPL; ++g) {
      const uint32_t key = best[g];
      if (key == kEmpty) continue;
      const uint32_t W = key >> jbits;
      const uint32_t jj = key & jmask;
      if (W > (uint32_t)p.S) continue;
      bool better = acc_bits > rb_acc[g] || (acc_bits == rb_acc[g] && W < rb_w[g]);
      if (!better && acc_bits == rb_acc[g] && W == rb_w[g])
        better = cand_index<T>(p, ct, jj) < cand_index<T>(p, rb_ct[g], rb_j[g]);
      if (better) { rb_acc[g] = acc_bits; rb_w[g] = W; rb_ct[g] = ct; rb_j[g] = jj; }
    }
  }

  // ---- a8: one partial key per (warp, level) ----
#pragma unroll
  for (int g = 0; g < LPL; ++g) {
    Key k{0ull, 0ull};
    if (rb_acc[g] != 0) {
      const int64_t c = cand_index<T>(p, rb_ct[g], rb_j[g]);
      k.acc_bits = rb_acc[g];
      k.tail = ((uint64_t)((uint32_t)p.S - rb_w[g]) << 40) | (uint64_t)(p.N - 1 - c);
    }
    // [tile][level][block]
    partial[LOKI_IDX(partial_off + (size_t)(g * 32 + lane) * gridDim.x + blockIdx.x, p.partial_keys, kSitePartial,
                     p.debug_flags)] = k;
  }
}

// Either launches (n_blocks > 0) or reports resident blocks per SM (n_blocks == 0).
template <int T, int NP, int LPL, int NS>
int act2(const DirProblem* p, LevelSpan dem_tile, int n_blocks, Key* d_partial, cudaStream_t st, int n_tiles) {
  const size_t smem = (size_t)p->uni_stage_bytes + (size_t)p->uni_max_members * 8 * (size_t)T;
  if (n_blocks == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, variant_score_kernel<T, NP, LPL, NS>, 32, smem) != cudaSuccess)
      return 0;
    return n;
  }
  variant_score_kernel<T, NP, LPL, NS><<<dim3(n_blocks, n_tiles), 32, smem, st>>>(*p, dem_tile, d_partial,
                                                                             p->uni_max_members);
  return (int)cudaGetLastError();
}

template <int T, int NP, int LPL>
int act(const DirProblem* p, LevelSpan dem_tile, int n_blocks, Key* d_partial, cudaStream_t st, int n_tiles) {
  if (p->n_leaves == 1) return act2<T, NP, LPL, 1>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
  if (p->n_leaves == 2) return act2<T, NP, LPL, 2>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
  return act2<T, NP, LPL, kMaxTasks>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
}

template <int NP, int LPL>
int by_tasks(int T, const DirProblem* p, LevelSpan dem_tile, int n_blocks, Key* d_partial, cudaStream_t st,
             int n_tiles) {
  switch (T) {
    case 1: return act<1, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 2: return act<2, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 3: return act<3, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 4: return act<4, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 5: return act<5, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 6: return act<6, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 7: return act<7, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 8: return act<8, NP, LPL>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

int dispatch(const DirProblem* p, int tile_levels, LevelSpan dem_tile, int n_blocks, Key* d_partial,
             cudaStream_t st, int n_tiles) {
  const bool two = p->n_parts_max == 2;
  switch (tile_levels) {
    case 32: return two ? by_tasks<2, 1>(p->T, p, dem_tile, n_blocks, d_partial, st, n_tiles)
                        : by_tasks<1, 1>(p->T, p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 64: return two ? by_tasks<2, 2>(p->T, p, dem_tile, n_blocks, d_partial, st, n_tiles)
                        : by_tasks<1, 2>(p->T, p, dem_tile, n_blocks, d_partial, st, n_tiles);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

}  // namespace

// Tiles of 32 or 64 levels (one or two levels per lane: the lane's demands of all tasks are registers).
cudaError_t launch_variant_score(const DirProblem& p, LevelSpan d_dem_tile, int tile_levels, int n_blocks,
                                 Key* d_partial, cudaStream_t st, int n_tiles) {
  if (n_blocks < 1 || n_tiles < 1 || n_tiles > 65535) return cudaErrorInvalidValue;
  return (cudaError_t)dispatch(&p, tile_levels, d_dem_tile, n_blocks, d_partial, st, n_tiles);
}

int variant_max_blocks_per_sm(const DirProblem& p, int tile_levels) {
  return dispatch(&p, tile_levels, LevelSpan{nullptr, 0, 0}, 0, nullptr, nullptr, 1);
}

}  // namespace loki
