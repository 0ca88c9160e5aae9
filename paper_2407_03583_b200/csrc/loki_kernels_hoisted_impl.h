// Templates of the hoisted (tabulated) scoring kernel; included by the translation units
// loki_kernels_hoisted_l1/_l2/_l4.cu, one per number of levels a lane owns, so that the
// instantiations compile in parallel.  See loki_kernels_hoisted.cu for the description.
#ifndef LOKI_KERNELS_HOISTED_IMPL_H_
#define LOKI_KERNELS_HOISTED_IMPL_H_

#include "loki_internal.h"

namespace loki {

namespace {

template <int LPL> struct Entries;                       // a lane's entries of one member
template <> struct Entries<1> { uint32_t v[1]; };
template <> struct __align__(8) Entries<2> { uint32_t v[2]; };
template <> struct __align__(16) Entries<4> { uint32_t v[4]; };

// Warp-uniform state of a work unit.
template <int T, int LPL>
struct Unit {
  const int32_t* lat;            // staged member latencies, all tasks
  const Entries<LPL>* tab;       // this lane's table column: tab[member * 32]
  uint32_t cnt[T];
  uint32_t roff[T];              // offset of task i's members in `lat`; in `tab` it is roff[i] - tskip
  uint32_t tskip;                // joined: members of tasks 0 and 1, which have no table rows
  int32_t need[T];               // sum_{k<i} smallest latency of task k's class
  int32_t n_leaves;
  uint32_t path_mask[kMaxTasks];
  // the innermost loop's rows, ascending latency: task 0's members, or (JOIN) the pairs of
  // task 0's and task 1's members
  const int32_t* in_lat;
  const Entries<LPL>* in_tab;    // this lane's column, rows 32 entries apart
  uint32_t in_cnt;
  const int32_t* in_lat0;        // JOIN on a tree: task 0's own latency of every joint row
  int32_t max_lat0;              // ... and the largest latency in task 0's class
  // prefix minima of the inner rows (row n: the minimum over rows 0 .. n), or nullptr: with them the
  // inner loop over a fitting prefix is one read
  const Entries<LPL>* in_pmin;
  // tables shared by all class tuples (one per task and class): an outer row carries no rank, the
  // walk adds the member's digit times the weight of its task in this class tuple; nullptr: the
  // entries of a table built for one class tuple already hold it
  const uint32_t* row_digit;
  uint32_t weight[T];
};

// The inner rows [begin, end) -- all of them fit -- against fixed outer tasks:
// one read, LPL adds, LPL minima per candidate.
template <int T, int LPL>
__device__ __forceinline__ void walk_inner(const Unit<T, LPL>& un, uint32_t begin, uint32_t end,
                                           const uint32_t (&ps)[LPL], uint32_t (&best)[LPL]) {
  const Entries<LPL>* t0 = un.in_tab + begin * 32u;
  // reads in flight per trip: eight rows of up to two levels, four rows of four (registers)
  constexpr int kRowsPerTrip = LPL <= 2 ? 8 : 4;
#pragma unroll kRowsPerTrip
  for (uint32_t n = end - begin; n > 0; --n, t0 += 32) {
    const Entries<LPL> v = *t0;
#pragma unroll
    for (int g = 0; g < LPL; ++g) best[g] = min(best[g], ps[g] + v.v[g]);
  }
}

// The same for a tree whose tasks 0 and 1 are joined: rows [begin, end) fit the paths through
// task 1; the paths that bypass task 1 see task 0's latency alone and are checked row by row.
// The same minimum over the fitting prefix [0, n_fit), n_fit > 0, from the table of prefix minima.
template <int T, int LPL>
__device__ __forceinline__ void take_prefix(const Unit<T, LPL>& un, uint32_t n_fit,
                                            const uint32_t (&ps)[LPL], uint32_t (&best)[LPL]) {
  const Entries<LPL> v = un.in_pmin[(n_fit - 1u) * 32u];
#pragma unroll
  for (int g = 0; g < LPL; ++g) best[g] = min(best[g], ps[g] + v.v[g]);
}
template <int T, int LPL>
__device__ __forceinline__ void walk_inner_checked(const Unit<T, LPL>& un, uint32_t begin, uint32_t end,
                                                   int32_t slack0, const uint32_t (&ps)[LPL],
                                                   uint32_t (&best)[LPL]) {
  const Entries<LPL>* t0 = un.in_tab + begin * 32u;
  const int32_t* l0 = un.in_lat0 + begin;
#pragma unroll 4
  for (uint32_t n = end - begin; n > 0; --n, t0 += 32, ++l0) {
    const bool fits = *l0 <= slack0;
    const Entries<LPL> v = *t0;
#pragma unroll
    for (int g = 0; g < LPL; ++g) {
      const uint32_t key = ps[g] + v.v[g];
      if (fits) best[g] = min(best[g], key);
    }
  }
}

// Number of leading inner rows (ascending latency) whose latency is at most `slack`,
// given that it is at most `n`.
template <int T, int LPL>
__device__ __forceinline__ uint32_t fit_prefix(const Unit<T, LPL>& un, uint32_t n, int32_t slack) {
  const int32_t* l0 = un.in_lat;
  while (n > 0 && l0[n - 1] > slack) --n;
  return n;
}

// Member d of task I joins the partial candidate: its latency comes off the slack of the leaf
// paths through task I, its table entry goes onto the partial key sums.  False: it does not fit
// (members come in ascending latency: then none of the later ones of the class does).
template <int I, int T, int LPL, int NS>
__device__ __forceinline__ bool take_member(const Unit<T, LPL>& un, uint32_t d, const int32_t (&slack)[NS],
                                            const uint32_t (&ps)[LPL], int32_t (&s2)[NS], uint32_t (&ps2)[LPL],
                                            int32_t& tight) {
  // the three reads are issued together: the entry and the digit do not wait for the latency test
  const int32_t lat = un.lat[un.roff[I] + d];
  const Entries<LPL> v = un.tab[(un.roff[I] + d - un.tskip) * 32u];
  const uint32_t rank = un.row_digit != nullptr ? un.row_digit[un.roff[I] + d] * un.weight[I] : 0u;
  if (NS == 1) {
    s2[0] = slack[0] - lat;
    tight = s2[0];
    if (tight < un.need[I]) return false;    // no member of the classes below can fit
  } else {
    tight = 0x7FFFFFFF;
#pragma unroll
    for (int k = 0; k < NS; ++k) {
      s2[k] = slack[k];
      if (k < un.n_leaves) {
        if ((un.path_mask[k] >> I) & 1u) s2[k] -= lat;
        tight = min(tight, s2[k]);
      }
    }
    if (tight < 0) return false;
  }
#pragma unroll
  for (int g = 0; g < LPL; ++g) ps2[g] = ps[g] + v.v[g] + rank;
  return true;
}

// Digit I of the odometer, down to digit IMIN (1, or 2 when tasks 0 and 1 are joined): members
// begin, begin + step, ... below end.
template <int I, int IMIN, int T, int LPL, int NS>
__device__ __forceinline__ void walk_outer(const Unit<T, LPL>& un, uint32_t begin, uint32_t end,
                                           const int32_t (&slack)[NS],
                                           const uint32_t (&ps)[LPL], uint32_t (&best)[LPL], uint32_t step = 1u) {
  uint32_t n_fit = un.in_cnt;                // I == IMIN: the inner rows' fitting prefix, shrinking with d
  for (uint32_t d = begin; d < end; d += step) {
    int32_t s2[NS];
    int32_t tight;
    uint32_t ps2[LPL];
    if (!take_member<I, T, LPL, NS>(un, d, slack, ps, s2, ps2, tight)) break;
    if constexpr (I == IMIN && IMIN == 2 && NS > 1) {
      // joined tasks 0 and 1 on a tree: `via1` is what the paths through task 1 leave, `past1`
      // what the paths that bypass it leave (both only shrink while d advances)
      int32_t via1 = 0x7FFFFFFF, past1 = 0x7FFFFFFF;
#pragma unroll
      for (int k = 0; k < NS; ++k)
        if (k < un.n_leaves) {
          if ((un.path_mask[k] >> 1) & 1u) via1 = min(via1, s2[k]); else past1 = min(past1, s2[k]);
        }
      n_fit = fit_prefix<T, LPL>(un, n_fit, via1);
      if (n_fit == 0) break;
      if (past1 >= un.max_lat0) walk_inner<T, LPL>(un, 0u, n_fit, ps2, best);
      else walk_inner_checked<T, LPL>(un, 0u, n_fit, past1, ps2, best);
    } else if constexpr (I == IMIN) {
      n_fit = fit_prefix<T, LPL>(un, n_fit, tight);
      if (n_fit == 0) break;
      if (un.in_pmin != nullptr) take_prefix<T, LPL>(un, n_fit, ps2, best);
      else walk_inner<T, LPL>(un, 0u, n_fit, ps2, best);
    } else {
      walk_outer<I - 1, IMIN, T, LPL, NS>(un, 0u, un.cnt[I - 1], s2, ps2, best);
    }
  }
}

// One warp's share of a class tuple.  The block's warps split the candidates along the outer
// digits (tasks T-1 down to IMIN): with three or more of them the two most significant are
// flattened and dealt round-robin, with two the most significant one, with one its members; a
// single task's rows are cut into runs.
template <int IMIN, int T, int LPL, int NS>
__device__ __forceinline__ void walk_share(const Unit<T, LPL>& un, uint32_t warp, uint32_t n_warps,
                                           const int32_t (&slack)[NS], const uint32_t (&ps)[LPL],
                                           uint32_t (&best)[LPL]) {
  constexpr int kOuter = T - IMIN;           // digits T-1 .. IMIN
  if constexpr (T == 1) {
    int32_t tight = 0x7FFFFFFF;
#pragma unroll
    for (int k = 0; k < NS; ++k) tight = min(tight, slack[k]);
    const uint32_t n_fit = fit_prefix<T, LPL>(un, un.cnt[0], tight);
    const uint32_t b = n_fit * warp / n_warps, e = n_fit * (warp + 1u) / n_warps;
    if (e > b) walk_inner<T, LPL>(un, b, e, ps, best);
  } else if constexpr (kOuter <= 1) {
    walk_outer<T - 1, IMIN, T, LPL, NS>(un, warp, un.cnt[T - 1], slack, ps, best, n_warps);
  } else if constexpr (kOuter == 2) {
    for (uint32_t d = warp; d < un.cnt[T - 1]; d += n_warps) {
      int32_t s2[NS];
      int32_t tight;
      uint32_t ps2[LPL];
      if (!take_member<T - 1, T, LPL, NS>(un, d, slack, ps, s2, ps2, tight)) break;
      walk_outer<T - 2, IMIN, T, LPL, NS>(un, 0u, un.cnt[T - 2], s2, ps2, best);
    }
  } else {
    const uint32_t c2 = un.cnt[T - 2], n_flat = un.cnt[T - 1] * c2;
    for (uint32_t f = warp; f < n_flat; f += n_warps) {
      const uint32_t d1 = f / c2, d2 = f - d1 * c2;
      int32_t s2[NS], s3[NS];
      int32_t tight;
      uint32_t ps2[LPL], ps3[LPL];
      if (!take_member<T - 1, T, LPL, NS>(un, d1, slack, ps, s2, ps2, tight)) break;   // d1 only grows with f
      if (!take_member<T - 2, T, LPL, NS>(un, d2, s2, ps2, s3, ps3, tight)) continue;
      walk_outer<T - 3, IMIN, T, LPL, NS>(un, 0u, un.cnt[T - 3], s3, ps3, best);
    }
  }
}

// One block of lay.warps warps per class tuple at a time; the warps build the tuple's table together
// and share it.  Dynamic shared memory: 32 header words | member latencies (int32, padded to 16 bytes)
// | table [member][lane] of Entries<LPL> | (JOIN) four int32 arrays of join_rows | (JOIN) member
// records of tasks 0 and 1 | joint table [row][lane].  Joined tasks have no rows in the first
// table: their entries exist only summed, in the joint table.  JOIN (at least three tasks, the classes of tasks 0 and 1 small): the pairs of their
// members become one inner loop, in ascending latency of the pair, so that the bookkeeping of a
// digit move is paid once per pair of classes instead of once per member of task 1.  Task 1 is a
// child of the root; on a tree the leaf paths that bypass it are checked against task 0's latency.
template <int T, int NP, int LPL, int NS, bool JOIN>
__global__ void __launch_bounds__(kHoistMaxWarps * 32)
hoisted_score_kernel(const __grid_constant__ DirProblem p, const LevelSpan span,
                     Key* __restrict__ partial, int max_members, int join_rows, int zero_demand,
                     int tab_members, int join_members, const int32_t* __restrict__ slo_limits,
                     int pmin_mode) {
  using Rec = UniRec<NP>;
  constexpr int LT = 32 * LPL;
  constexpr int kHdrWords = 32;
  const int lane = threadIdx.x & 31;
  const uint32_t warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const int tile_level0 = span.level_begin + (int)blockIdx.y * LT;      // grid.y: consecutive level tiles
  // grid.z: latency SLOs (the per-leaf limits of SLO z are slo_limits[z][.]; nullptr: the problem's own).
  // The SLO enters only as the slack the walk starts from, so the tables are the same for all of them.
  // Partial keys: [SLO][tile][level][block x warp].
  const size_t n_parts = (size_t)gridDim.x * n_warps;
  const size_t partial_off = ((size_t)blockIdx.z * gridDim.y + blockIdx.y) * n_parts * LT;
  const int32_t* const my_limits = slo_limits != nullptr ? slo_limits + (size_t)blockIdx.z * kMaxTasks : nullptr;
  extern __shared__ __align__(16) unsigned char s_raw[];
  uint32_t* const s_hdr = reinterpret_cast<uint32_t*>(s_raw);
  int32_t* const s_lat = reinterpret_cast<int32_t*>(s_raw + kHdrWords * 4);
  Entries<LPL>* const s_tab =
      reinterpret_cast<Entries<LPL>*>(s_raw + kHdrWords * 4 + ((size_t)max_members * 4 + 15) / 16 * 16);
  int32_t* const j_raw = reinterpret_cast<int32_t*>(s_tab + (size_t)tab_members * 32);   // pair latencies, pair order
  int32_t* const j_ord = j_raw + join_rows;
  int32_t* const j_lat = j_ord + join_rows;                                               // sorted
  int32_t* const j_lat0 = j_lat + join_rows;                                              // task 0's share, sorted
  // the four int32 arrays are padded to 16 bytes so that the joint table keeps the alignment of its entries
  Rec* const j_rec = reinterpret_cast<Rec*>(
      reinterpret_cast<unsigned char*>(j_raw) + ((size_t)join_rows * 4 * 4 + 15) / 16 * 16);
  Entries<LPL>* const j_tab = reinterpret_cast<Entries<LPL>*>(j_rec + join_members);
  __shared__ double s_pp[kMaxTasks];
#ifdef LOKI_DEBUG
  // the carve-up above must end inside the dynamic shared memory the launch was given
  if (threadIdx.x == 0 &&
      (size_t)(reinterpret_cast<unsigned char*>(j_tab + (size_t)join_rows * 32) - s_raw) > loki_dynamic_smem_bytes())
    (void)LOKI_IDX(-1, 0, kSiteSharedLayout, p.debug_flags);
#endif

  // a4: the stage demands of this lane's levels, lane * LPL + g of the tile (the same in every warp)
  double dem[LPL][T];
#pragma unroll
  for (int g = 0; g < LPL; ++g)
    level_stage_demands<T>(p, span.demand, span.n_levels, tile_level0 + lane * LPL + g, dem[g]);

  uint64_t rb_acc[LPL];
  uint32_t rb_ct[LPL], rb_w[LPL], rb_j[LPL];
#pragma unroll
  for (int g = 0; g < LPL; ++g) { rb_acc[g] = 0; rb_ct[g] = 0; rb_w[g] = 0; rb_j[g] = 0; }

  const uint32_t jbits = (uint32_t)p.jbits;
  const uint32_t jmul = 1u << jbits;
  const uint32_t jmask = jmul - 1u;
  // zero_demand: no option needs a worker whatever its latency and batch size, so an entry is
  // the rank alone (the "1 + floor" form of the fma needs a demand of at least 1)
  const uint32_t w_mul = zero_demand ? 0u : jmul;
  const uint32_t w_mask = zero_demand ? 0u : 0xFFFFFFFFu;
  const Rec* const recs = reinterpret_cast<const Rec*>(p.uni_members);

  // a block takes class tuples round-robin: its warps build the tuple's table together and then
  // split its candidates (walk_share)
  for (uint32_t ct = blockIdx.x; ct < (uint32_t)p.n_ct; ct += gridDim.x) {
    uint64_t acc_bits;
    __syncthreads();                       // the walks of the previous class tuple are over
    {
      // ---- stage the class tuple: latencies, counts, path accuracy, and per lane the
      //      table column of its levels: the worker arithmetic of Eq. 2, once per (level, task, member) ----
      uint32_t q = ct, off = 0, stride = 1, joined = 0;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        const uint32_t nc = (uint32_t)p.n_class[i];
        const uint32_t cls = q % nc;
        q /= nc;
        const int idx = (int)LOKI_IDX(p.class_off[i] + (int)cls, p.n_classes, kSiteClass, p.debug_flags);
        const uint32_t c = (uint32_t)p.class_count[idx];
        (void)LOKI_IDX(p.member_off[i] + p.class_first[idx] + (long long)c - 1, p.n_members, kSiteMember, p.debug_flags);
        const Rec* src = recs + p.member_off[i] + p.class_first[idx];
        const int32_t* order = p.lat_order + p.member_off[i] + p.class_first[idx];
        for (uint32_t k = threadIdx.x; k < c; k += blockDim.x)
          s_lat[LOKI_IDX(off + k, max_members, kSiteHoistLat, p.debug_flags)] = src[LOKI_IDX(order[k], c, kSiteMember, p.debug_flags)].lat;
        if (JOIN && i < 2) {
          // a joined task: its records, with the entry's constant part folded into `nsh`
          for (uint32_t k = threadIdx.x; k < c; k += blockDim.x) {
            const uint32_t m = (uint32_t)order[k];
            Rec rc = src[m];
            rc.nsh = (rc.nsh & w_mask) + m * stride;
            j_rec[LOKI_IDX(off + k, join_members, kSiteHoistJoin, p.debug_flags)] = rc;
          }
          joined += c;
        } else {
          for (uint32_t k = warp; k < c; k += n_warps) {       // a member per warp, a level column per lane
            const uint32_t m = (uint32_t)order[k];     // the member's own digit
            const Rec rc = src[m];
            Entries<LPL> e;
#pragma unroll
            for (int g = 0; g < LPL; ++g) {
              double acc = __fma_rd(dem[g][i], rc.r[0], kMagic);
              if (NP == 2) acc = __fma_rd(dem[g][i], rc.r[NP - 1], acc);
              e.v[g] = (uint32_t)__double2loint(acc) * w_mul + (rc.nsh & w_mask) + m * stride;
            }
            s_tab[(size_t)LOKI_IDX(off - joined + k, tab_members, kSiteHoistTab, p.debug_flags) * 32 + lane] = e;
          }
        }
        if (threadIdx.x == 0) {
          s_hdr[i] = c;
          s_hdr[8 + i] = off;
          s_hdr[16 + i] = (uint32_t)p.class_min_lat[idx];
          // a2: path accuracy products in task order (no fused multiply-add)
          const double a = p.class_acc[idx];
          s_pp[i] = i == 0 ? a : __dmul_rn(s_pp[p.parent[i]], a);
        }
        off += c;
        stride *= c;
      }
      __syncthreads();
      if (JOIN) {
        // pairs (k0, k1) of the two innermost classes: latency, rank by (latency, pair index), joint entries
        const uint32_t c0 = s_hdr[0], c1 = s_hdr[1], o0 = s_hdr[8], o1 = s_hdr[9];
        const uint32_t n = c0 * c1;
        if (p.join_order != nullptr) {
          // the order depends on the two classes alone and was tabulated when the handle was built
          const uint32_t cls0 = ct % (uint32_t)p.n_class[0], cls1 = ct / (uint32_t)p.n_class[0] % (uint32_t)p.n_class[1];
          const int32_t* ord = p.join_order + ((size_t)cls1 * (size_t)p.n_class[0] + cls0) * (size_t)p.join_stride;
          for (uint32_t r = threadIdx.x; r < n; r += blockDim.x) {
            const uint32_t q = (uint32_t)LOKI_IDX(ord[LOKI_IDX(r, p.join_stride, kSiteHoistJoin, p.debug_flags)], n, kSiteHoistJoin, p.debug_flags);
            j_ord[r] = (int32_t)q;
            j_lat[r] = s_lat[o0 + q % c0] + s_lat[o1 + q / c0];
            j_lat0[r] = s_lat[o0 + q % c0];
          }
        } else {
        for (uint32_t q = threadIdx.x; q < n; q += blockDim.x) j_raw[q] = s_lat[o0 + q % c0] + s_lat[o1 + q / c0];
        __syncthreads();
        for (uint32_t q = threadIdx.x; q < n; q += blockDim.x) {
          const int32_t mine = j_raw[q];
          uint32_t rank = 0;
          for (uint32_t r = 0; r < n; ++r) {
            const int32_t other = j_raw[r];
            rank += (other < mine || (other == mine && r < q)) ? 1u : 0u;
          }
          rank = (uint32_t)LOKI_IDX(rank, join_rows, kSiteHoistJoin, p.debug_flags);
          j_ord[rank] = (int32_t)q;
          j_lat[rank] = mine;
          j_lat0[rank] = s_lat[o0 + q % c0];
        }
        }
        __syncthreads();
        for (uint32_t r = warp; r < n; r += n_warps) {           // a row per warp, a level column per lane
          const uint32_t q = (uint32_t)j_ord[r];
          const Rec a = j_rec[o0 + q % c0];
          const Rec b = j_rec[o1 + q / c0];
          Entries<LPL> e;
#pragma unroll
          for (int g = 0; g < LPL; ++g) {
            double acc0 = __fma_rd(dem[g][0], a.r[0], kMagic);
            double acc1 = __fma_rd(dem[g][1], b.r[0], kMagic);
            if (NP == 2) {
              acc0 = __fma_rd(dem[g][0], a.r[NP - 1], acc0);
              acc1 = __fma_rd(dem[g][1], b.r[NP - 1], acc1);
            }
            e.v[g] = ((uint32_t)__double2loint(acc0) + (uint32_t)__double2loint(acc1)) * w_mul + a.nsh + b.nsh;
          }
          j_tab[(size_t)LOKI_IDX(r, join_rows, kSiteHoistJoin, p.debug_flags) * 32 + lane] = e;
        }
        __syncthreads();
      }
    }
    {
      double sum = s_pp[p.leaf_task[0]];
      for (int k = 1; k < p.n_leaves; ++k) sum = __dadd_rn(sum, s_pp[p.leaf_task[k]]);
      acc_bits = (uint64_t)__double_as_longlong(__ddiv_rn(sum, (double)p.n_leaves));
    }

    // pmin_mode: the inner rows are replaced, in place, by their prefix minima (row n: the minimum
    // over rows 0 .. n); the walk then reads one row per fitting prefix.  Not with joined tasks on a
    // tree, whose rows are also walked one by one where a path bypasses task 1 (the host gives such
    // problems the layout without the join).  Warp 0, a level column per lane, the rows in order.
    const bool pmin = pmin_mode != 0 && T > 1 && !(JOIN && NS > 1);
    if (pmin) {
      Entries<LPL>* const rows = JOIN ? j_tab : s_tab + (size_t)s_hdr[8] * 32;
      const uint32_t n_rows = JOIN ? s_hdr[0] * s_hdr[1] : s_hdr[0];
      if (warp == 0) {
        Entries<LPL> run = rows[lane];
        for (uint32_t r = 1; r < n_rows; ++r) {
          Entries<LPL>* const at = rows + (size_t)LOKI_IDX(r, JOIN ? join_rows : max_members, kSiteHoistTab, p.debug_flags) * 32 + lane;
          const Entries<LPL> v = *at;
#pragma unroll
          for (int g = 0; g < LPL; ++g) run.v[g] = min(run.v[g], v.v[g]);
          *at = run;
        }
      }
      __syncthreads();
    }

    Unit<T, LPL> un;
    un.in_pmin = pmin ? (JOIN ? j_tab : s_tab + (size_t)s_hdr[8] * 32) + lane : nullptr;
    un.row_digit = nullptr;
    un.lat = s_lat;
    un.tab = s_tab + lane;
    un.in_lat = JOIN ? j_lat : s_lat + s_hdr[8];
    un.in_tab = JOIN ? j_tab + lane : s_tab + (size_t)s_hdr[8] * 32 + lane;
    un.in_cnt = JOIN ? s_hdr[0] * s_hdr[1] : s_hdr[0];
    un.in_lat0 = j_lat0;
    un.tskip = JOIN ? s_hdr[0] + s_hdr[1] : 0u;
    un.max_lat0 = s_lat[s_hdr[8] + s_hdr[0] - 1];      // classes are staged in ascending latency
    un.n_leaves = p.n_leaves;
#pragma unroll
    for (int k = 0; k < kMaxTasks; ++k) un.path_mask[k] = p.path_mask[k];
    {
      int32_t nd = 0;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        un.cnt[i] = s_hdr[i];
        un.roff[i] = s_hdr[8 + i];
        un.need[i] = nd;
        nd += (int32_t)s_hdr[16 + i];
      }
    }

    uint32_t best[LPL], ps[LPL];
#pragma unroll
    for (int g = 0; g < LPL; ++g) { best[g] = kEmpty; ps[g] = 0; }
    int32_t slack[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k)
      slack[k] = k < p.n_leaves ? (my_limits != nullptr ? my_limits[k] : p.lat_limit[k]) : 0x7FFFFFFF;
    walk_share<(JOIN ? 2 : 1), T, LPL, NS>(un, warp, n_warps, slack, ps, best);

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
    // [SLO][tile][level][block x warp]
    partial[LOKI_IDX(partial_off + (size_t)(lane * LPL + g) * n_parts + (size_t)blockIdx.x * n_warps + warp,
                     p.partial_keys, kSitePartial, p.debug_flags)] = k;
  }
}

// Either launches (n_blocks > 0) or reports resident blocks per SM (n_blocks == 0).
template <int T, int NP, int LPL, int NS, bool JOIN>
int act2(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks, Key* d_partial,
         cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits) {
  auto kern = hoisted_score_kernel<T, NP, LPL, NS, JOIN>;
  if (n_blocks == 0) {
    int n = 0;
    if (lay->smem_bytes > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, lay->smem_bytes) != cudaSuccess)
      return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, lay->warps * 32, (size_t)lay->smem_bytes) != cudaSuccess)
      return 0;
    return n;
  }
  kern<<<dim3(n_blocks, n_tiles, n_slos), lay->warps * 32, (size_t)lay->smem_bytes, st>>>(*p, dem_tile, d_partial, lay->max_members,
                                                                          lay->join_rows, zero, lay->tab_members,
                                                                          lay->join_members, slo_limits,
                                                                          zero ? 0 : lay->pmin_mode);
  return (int)cudaGetLastError();
}

template <int T, int NP, int LPL, int NS>
int act(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks, Key* d_partial,
        cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits) {
  if constexpr (T >= 3) {
    if (lay->join_rows > 0) return act2<T, NP, LPL, NS, true>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
  }
  return act2<T, NP, LPL, NS, false>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
}

template <int NP, int LPL, int NS>
int by_tasks(int T, const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks,
             Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits) {
  switch (T) {
    case 1: return act<1, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 2: return act<2, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 3: return act<3, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 4: return act<4, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 5: return act<5, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 6: return act<6, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 7: return act<7, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 8: return act<8, NP, LPL, NS>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

template <int NP, int LPL>
int by_shape(int n_leaves, int T, const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile,
             int n_blocks, Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits) {
  // latency slack slots carried down the walk: one per leaf path (a tree with one leaf is a chain)
  if (n_leaves == 1) return by_tasks<NP, LPL, 1>(T, p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
  if (n_leaves == 2) return by_tasks<NP, LPL, 2>(T, p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
  return by_tasks<NP, LPL, kMaxTasks>(T, p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
}

// Launch (n_blocks > 0) or occupancy query (n_blocks == 0) for LPL levels per lane.
template <int LPL>
int hoisted_for_lpl(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks,
                    Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits) {
  return p->n_parts_max == 2 ? by_shape<2, LPL>(p->n_leaves, p->T, p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits)
                             : by_shape<1, LPL>(p->n_leaves, p->T, p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
}


// ---- tables shared by all class tuples (PrefixTables) ----

// One entry of a row for a lane's level: the worker arithmetic of Eq. 2 for the row's member (or
// pair of members) at that level's stage demands, shifted above the rank bits, plus the row's constant.
template <int T, int NP>
__device__ __forceinline__ uint32_t prefix_entry(const UniRec<NP>* recs, const int4 d, const double (&dem)[T], uint32_t jmul) {
  const UniRec<NP> a = recs[d.x];
  const int ta = d.w & 255, tb = (d.w >> 8) & 255;
  double da = 0.0, db = 0.0;
#pragma unroll
  for (int i = 0; i < T; ++i) {
    if (i == ta) da = dem[i];
    if (i == tb) db = dem[i];
  }
  double acc = __fma_rd(da, a.r[0], kMagic);
  if (NP == 2) acc = __fma_rd(da, a.r[NP - 1], acc);
  uint32_t w = (uint32_t)__double2loint(acc), nsh = a.nsh;
  if (d.y >= 0) {
    const UniRec<NP> b = recs[d.y];
    double acc1 = __fma_rd(db, b.r[0], kMagic);
    if (NP == 2) acc1 = __fma_rd(db, b.r[NP - 1], acc1);
    w += (uint32_t)__double2loint(acc1);
    nsh += b.nsh;
  }
  return w * jmul + nsh + (uint32_t)d.z;
}

// One warp per outer row, or per inner group (its rows in order, each replaced by the minimum so
// far); a level column per lane; grid.y: level tiles.
template <int T, int NP, int LPL>
__global__ void __launch_bounds__(kPrefixWarps * 32)
prefix_build_kernel(const __grid_constant__ DirProblem p, const __grid_constant__ PrefixTables t, const LevelSpan span) {
  const int lane = threadIdx.x & 31;
  const int job = (int)blockIdx.x * kPrefixWarps + (int)(threadIdx.x >> 5);
  if (job >= t.n_outer + t.n_groups) return;
  const int tile_level0 = span.level_begin + (int)blockIdx.y * 32 * LPL;
  double dem[LPL][T];
#pragma unroll
  for (int g = 0; g < LPL; ++g)
    level_stage_demands<T>(p, span.demand, span.n_levels, tile_level0 + lane * LPL + g, dem[g]);
  const UniRec<NP>* const recs = reinterpret_cast<const UniRec<NP>*>(p.uni_members);
  const uint32_t jmul = 1u << (uint32_t)p.jbits;
  Entries<LPL>* const tab = reinterpret_cast<Entries<LPL>*>(t.tab) + (size_t)blockIdx.y * (size_t)t.n_rows * 32 + lane;
  if (job < t.n_outer) {
    const int4 d = t.row_desc[job];
    Entries<LPL> e;
#pragma unroll
    for (int g = 0; g < LPL; ++g) e.v[g] = prefix_entry<T, NP>(recs, d, dem[g], jmul);
    tab[(size_t)job * 32] = e;
    return;
  }
  const int2 grp = t.groups[job - t.n_outer];
  Entries<LPL> run;
#pragma unroll
  for (int g = 0; g < LPL; ++g) run.v[g] = kEmpty;
  for (int r = 0; r < grp.y; ++r) {
    const int row = (int)LOKI_IDX(grp.x + r, t.n_rows, kSiteHoistTab, p.debug_flags);
    const int4 d = t.row_desc[row];
#pragma unroll
    for (int g = 0; g < LPL; ++g) run.v[g] = min(run.v[g], prefix_entry<T, NP>(recs, d, dem[g], jmul));
    tab[(size_t)row * 32] = run;
  }
}


// The walk over the shared tables: a warp takes one class tuple at a time (no block-wide step), a
// lane owns LPL adjacent levels of the tile; outer tasks as in the hoisted kernel, the innermost
// task (JOIN: pair of tasks) is one read of the prefix minimum of its fitting rows.  grid.y: level
// tiles (table tile tile0 + blockIdx.y), grid.z: latency SLOs.
template <int T, int LPL, int NS, bool JOIN>
__global__ void __launch_bounds__(kPrefixWarps * 32)
prefix_walk_kernel(const __grid_constant__ DirProblem p, const __grid_constant__ PrefixTables t,
                   Key* __restrict__ partial, int tile0, const int32_t* __restrict__ slo_limits) {
  constexpr int LT = 32 * LPL;
  const int lane = threadIdx.x & 31;
  const uint32_t gw = blockIdx.x * kPrefixWarps + (threadIdx.x >> 5);
  const size_t n_parts = (size_t)gridDim.x * kPrefixWarps;
  const size_t partial_off = ((size_t)blockIdx.z * gridDim.y + blockIdx.y) * n_parts * LT;
  const int32_t* const my_limits = slo_limits != nullptr ? slo_limits + (size_t)blockIdx.z * kMaxTasks : nullptr;
  const Entries<LPL>* const tab =
      reinterpret_cast<const Entries<LPL>*>(t.tab) + (size_t)(tile0 + (int)blockIdx.y) * (size_t)t.n_rows * 32 + lane;

  uint64_t rb_acc[LPL];
  uint32_t rb_ct[LPL], rb_w[LPL], rb_j[LPL];
#pragma unroll
  for (int g = 0; g < LPL; ++g) { rb_acc[g] = 0; rb_ct[g] = 0; rb_w[g] = 0; rb_j[g] = 0; }
  const uint32_t jbits = (uint32_t)p.jbits;
  const uint32_t jmask = (1u << jbits) - 1u;

  Unit<T, LPL> un;
  un.lat = t.row_lat;
  un.tab = tab;
  un.tskip = 0;
  un.n_leaves = p.n_leaves;
#pragma unroll
  for (int k = 0; k < kMaxTasks; ++k) un.path_mask[k] = p.path_mask[k];
  un.in_tab = tab;
  un.in_lat0 = nullptr;
  un.max_lat0 = 0;
  un.row_digit = t.row_digit;

  for (uint32_t ct = gw; ct < (uint32_t)p.n_ct; ct += (uint32_t)n_parts) {
    uint32_t q = ct, weight = 1, cls01[2] = {0, 0};
    int32_t nd = 0;
#pragma unroll
    for (int i = 0; i < T; ++i) {
      const uint32_t nc = (uint32_t)p.n_class[i];
      const uint32_t cls = q % nc;
      q /= nc;
      if (i < 2) cls01[i] = cls;
      const int idx = (int)LOKI_IDX(p.class_off[i] + (int)cls, p.n_classes, kSiteClass, p.debug_flags);
      un.cnt[i] = (uint32_t)p.class_count[idx];
      un.roff[i] = (uint32_t)t.class_rows[idx];
      un.need[i] = nd;
      nd += p.class_min_lat[idx];
      un.weight[i] = weight;
      weight *= un.cnt[i];
    }
    const uint32_t in_row = JOIN ? (uint32_t)t.pair_rows[cls01[1] * (uint32_t)p.n_class[0] + cls01[0]] : un.roff[0];
    (void)LOKI_IDX(in_row, t.n_rows, kSiteHoistTab, p.debug_flags);
    un.in_cnt = JOIN ? un.cnt[0] * un.cnt[1] : un.cnt[0];
    un.in_lat = t.row_lat + in_row;
    un.in_pmin = tab + (size_t)in_row * 32;
    const uint64_t acc_bits = p.ct_acc[ct];

    uint32_t best[LPL], ps[LPL];
#pragma unroll
    for (int g = 0; g < LPL; ++g) { best[g] = kEmpty; ps[g] = 0; }
    int32_t slack[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k)
      slack[k] = k < p.n_leaves ? (my_limits != nullptr ? my_limits[k] : p.lat_limit[k]) : 0x7FFFFFFF;
    walk_share<(JOIN ? 2 : 1), T, LPL, NS>(un, 0u, 1u, slack, ps, best);

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

#pragma unroll
  for (int g = 0; g < LPL; ++g) {
    Key k{0ull, 0ull};
    if (rb_acc[g] != 0) {
      const int64_t c = cand_index<T>(p, rb_ct[g], rb_j[g]);
      k.acc_bits = rb_acc[g];
      k.tail = ((uint64_t)((uint32_t)p.S - rb_w[g]) << 40) | (uint64_t)(p.N - 1 - c);
    }
    partial[LOKI_IDX(partial_off + (size_t)(lane * LPL + g) * n_parts + gw, p.partial_keys, kSitePartial, p.debug_flags)] = k;
  }
}


template <int T, int NP, int LPL>
int prefix_build_act(const PrefixCall& c) {
  const int jobs = c.t->n_outer + c.t->n_groups;
  prefix_build_kernel<T, NP, LPL><<<dim3((unsigned)((jobs + kPrefixWarps - 1) / kPrefixWarps), (unsigned)c.n_tiles),
                                    kPrefixWarps * 32, 0, c.st>>>(*c.p, *c.t, c.span);
  return (int)cudaGetLastError();
}

template <int T, int LPL, int NS, bool JOIN>
int prefix_walk_act(const PrefixCall& c) {
  auto kern = prefix_walk_kernel<T, LPL, NS, JOIN>;
  if (c.n_blocks == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kPrefixWarps * 32, 0) != cudaSuccess) return 0;
    return n;
  }
  kern<<<dim3((unsigned)c.n_blocks, (unsigned)c.n_tiles, (unsigned)c.n_slos), kPrefixWarps * 32, 0, c.st>>>(
      *c.p, *c.t, c.d_partial, c.tile0, c.slo_limits);
  return (int)cudaGetLastError();
}

template <int T, int LPL>
int prefix_by_shape(const PrefixCall& c) {
  if (c.build) return c.p->n_parts_max == 2 ? prefix_build_act<T, 2, LPL>(c) : prefix_build_act<T, 1, LPL>(c);
  if (c.p->n_leaves == 1) {
    if constexpr (T >= 3) {
      if (c.t->joined) return prefix_walk_act<T, LPL, 1, true>(c);
    }
    return prefix_walk_act<T, LPL, 1, false>(c);
  }
  if (c.p->n_leaves == 2) return prefix_walk_act<T, LPL, 2, false>(c);
  return prefix_walk_act<T, LPL, kMaxTasks, false>(c);
}

template <int LPL>
int prefix_for_lpl(const PrefixCall& c) {
  const int fail = c.build || c.n_blocks > 0 ? (int)cudaErrorInvalidValue : 0;
  switch (c.p->T) {
    case 2: return prefix_by_shape<2, LPL>(c);
    case 3: return prefix_by_shape<3, LPL>(c);
    case 4: return prefix_by_shape<4, LPL>(c);
    case 5: return prefix_by_shape<5, LPL>(c);
    case 6: return prefix_by_shape<6, LPL>(c);
    case 7: return prefix_by_shape<7, LPL>(c);
    case 8: return prefix_by_shape<8, LPL>(c);
    default: return fail;
  }
}

}  // namespace

}  // namespace loki

#endif  // LOKI_KERNELS_HOISTED_IMPL_H_
