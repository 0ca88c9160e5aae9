// The level-lane scoring kernel of libloki_alloc: lanes hold demand levels, the
// candidate is the same for the whole warp.  Every (candidate, demand level) pair
// of a latency-feasible candidate is scored with the full per-task worker
// arithmetic, one FP64 fused multiply-add per option part, as in the
// candidate-lane kernel; the two differ in which operand of that fma is
// warp-uniform.
//
// Why this mapping.  A double-precision fma whose three sources are ordinary
// registers issues at two thirds of the FP64 pipe's rate on this machine (three
// 64-bit register reads per lane); with one source in a uniform register it
// issues at the full rate (csrc/fp64_issue_probe.cu measures both).  Here the
// stage demands of a lane's levels sit in ordinary registers for the whole
// launch, the accumulator is an ordinary register, and the reciprocal constant of
// the candidate's option is identical for all lanes, i.e. a candidate for the
// uniform operand; the block is one warp so that every loop bound and table
// address derives from blockIdx alone.  In practice the compiler keeps the
// constants it loads from shared memory in ordinary registers, so the kernel does
// not reach that rate; what the mapping does deliver is that a latency-infeasible
// candidate costs one compare instead of a full set of fmas, and that no
// cross-lane reduction is needed (a lane owns its levels).
//
// Walk.  The candidates of a class tuple (per task, options with bit-identical
// task accuracy form a class) are ranked mixed-radix over the class members,
// task 0 least significant.  A work unit is one slice of a class tuple along its
// most significant digit; units are dealt round-robin to the warps, so that every
// warp sees the same mix of cheap (latency-infeasible, skipped after one compare)
// and expensive candidates.  Inside a unit the warp runs an odometer: the records
// of tasks 1..T-1 stay put until their digit changes, task 0's members are the
// inner loop.  Task 0 is the root and lies on every root-to-leaf path, so the
// latency bound of a candidate (Eq. 7) is one compare of the member's latency
// against the slack the outer tasks leave.
//
// Workers (Eq. 2 with Eq. 5): 1 + floor(dem * r) per part, r the largest double
// strictly below share * lat / (16 * batch * 1e9), from one fma rounded toward
// minus infinity onto an integer-valued accumulator in [2^52, 2^53); the host
// has checked that this is exact for every demand the kernel can see.  The
// running best of a level is (workers << jbits | rank) under an unsigned
// minimum: fewest workers, then lowest candidate index within the class tuple;
// across class tuples the accuracy decides first.
#include "loki_internal.h"

namespace loki {

namespace {

constexpr double kMagic = 6755399441055744.0;   // 1.5 * 2^52: ulp 1, low mantissa word 0
constexpr uint32_t kEmpty = 0xFFFFFFFFu;

template <int NP> struct UniRec;
template <> struct __align__(16) UniRec<1> { double r[1]; int32_t lat; uint32_t nsh; };
template <> struct __align__(16) UniRec<2> { double r[2]; int32_t lat; uint32_t nsh; int32_t pad[2]; };
static_assert(sizeof(UniRec<1>) == kUniRecBytes1 && sizeof(UniRec<2>) == kUniRecBytes2, "UniRec layout");

template <int T>
__device__ __forceinline__ int64_t cand_index(const DirProblem& p, uint64_t ct, uint32_t j) {
  int64_t c = 0;
#pragma unroll
  for (int i = 0; i < T; ++i) {
    const uint32_t nc = (uint32_t)p.n_class[i];
    const uint32_t cls = (uint32_t)(ct % nc);
    ct /= nc;
    const int32_t first = p.class_first[p.class_off[i] + cls];
    const uint32_t cnt = (uint32_t)p.class_count[p.class_off[i] + cls];
    const uint32_t d = j % cnt;
    j /= cnt;
    c += (int64_t)p.members[p.member_off[i] + first + d].opt * p.stride[i];
  }
  return c;
}

// State of a work unit that the nested walk reads (all of it warp-uniform).
template <int T, int NP>
struct Unit {
  const UniRec<NP>* rec;     // staged member records
  uint32_t cnt[T];           // members of the class of task i
  uint32_t roff[T];          // offset of task i's records in `rec`
  uint32_t stride[T];        // prod_{k<i} cnt[k]: rank weight of digit i
  int32_t need[T];           // sum_{k<i} smallest latency of task k's class (chains: pruning bound)
  uint32_t jmul;
  int32_t n_leaves;
  uint32_t path_mask[kMaxTasks];
};

// Task 0's members against fixed outer tasks: the inner loop (a3, a5-a7).
// `slack` is what the outer tasks leave of the tightest path bound, `kb` the packed
// key's constant part of the outer tasks (their parts << jbits, plus their rank).
template <int T, int NP, int LPL>
__device__ __forceinline__ void walk_inner(const Unit<T, NP>& un, uint32_t begin, uint32_t end,
                                           int32_t slack, uint32_t kb,
                                           const double (&rh)[T][NP], const double (&dem)[LPL][T],
                                           uint32_t (&best)[LPL]) {
  const UniRec<NP>* m0 = un.rec + un.roff[0];
  for (uint32_t e = begin; e < end; ++e) {
    const UniRec<NP> rc = m0[e];
    if (rc.lat > slack) continue;
    const uint32_t kconst = kb + e + rc.nsh;
#pragma unroll
    for (int g = 0; g < LPL; ++g) {
      double acc = __fma_rd(dem[g][0], rc.r[0], kMagic);
      if (NP == 2) acc = __fma_rd(dem[g][0], rc.r[NP - 1], acc);
#pragma unroll
      for (int i = 1; i < T; ++i)
#pragma unroll
        for (int s = 0; s < NP; ++s) acc = __fma_rd(dem[g][i], rh[i][s], acc);
      best[g] = min(best[g], (uint32_t)__double2loint(acc) * un.jmul + kconst);
    }
  }
}

// Digit I of the odometer (I >= 1): one nested loop per task, the task's record
// loaded when its digit moves.  slack[k] is what the tasks above leave of leaf k's
// latency bound (chains: one entry).
template <int I, int T, int NP, int LPL, bool CHAIN>
__device__ __forceinline__ void walk_outer(const Unit<T, NP>& un, uint32_t begin, uint32_t end,
                                           const int32_t (&slack)[CHAIN ? 1 : kMaxTasks], uint32_t kb,
                                           double (&rh)[T][NP], const double (&dem)[LPL][T],
                                           uint32_t (&best)[LPL]) {
  constexpr int NS = CHAIN ? 1 : kMaxTasks;
  for (uint32_t d = begin; d < end; ++d) {
    const UniRec<NP> rc = un.rec[un.roff[I] + d];
    int32_t s2[NS];
    int32_t tight;
    if (CHAIN) {
      s2[0] = slack[0] - rc.lat;
      tight = s2[0];
      if (tight < un.need[I]) continue;      // no member of the classes below can fit
    } else {
      tight = 0x7FFFFFFF;
#pragma unroll
      for (int k = 0; k < NS; ++k) {
        s2[k] = slack[k];
        if (k < un.n_leaves) {
          if ((un.path_mask[k] >> I) & 1u) s2[k] -= rc.lat;
          tight = min(tight, s2[k]);
        }
      }
      if (tight < 0) continue;
    }
#pragma unroll
    for (int s = 0; s < NP; ++s) rh[I][s] = rc.r[s];
    const uint32_t kb2 = kb + rc.nsh + d * un.stride[I];
    if constexpr (I == 1) walk_inner<T, NP, LPL>(un, 0u, un.cnt[0], tight, kb2, rh, dem, best);
    else walk_outer<I - 1, T, NP, LPL, CHAIN>(un, 0u, un.cnt[I - 1], s2, kb2, rh, dem, best);
  }
}

// T tasks, NP parts per option (2 when split options exist), LPL levels per lane,
// CHAIN: the tree is a chain (one leaf, every task on its path).
//
// Dynamic shared memory: a header of 32 words (members per class of the current
// class tuple, offset of each task's records, smallest latency of each class)
// followed by the member records of the class tuple's T classes.  The warp copies
// them from the global tables once per work unit and then reads them back at
// warp-uniform addresses.
template <int T, int NP, int LPL, bool CHAIN>
__global__ void __launch_bounds__(32)
uniform_score_kernel(const __grid_constant__ DirProblem p, const double* __restrict__ dem_tile,
                     Key* __restrict__ partial) {
  using Rec = UniRec<NP>;
  constexpr int LT = 32 * LPL;
  constexpr int kHdrWords = 32;
  const int lane = threadIdx.x;
  dem_tile += (size_t)blockIdx.y * LT * T;                 // grid.y: consecutive level tiles
  partial += (size_t)blockIdx.y * gridDim.x * LT;
  extern __shared__ __align__(16) unsigned char s_raw[];
  uint32_t* const s_hdr = reinterpret_cast<uint32_t*>(s_raw);
  Rec* const s_rec = reinterpret_cast<Rec*>(s_raw + kHdrWords * 4);
  __shared__ double s_pp[kMaxTasks];

  // a4 is done by the level kernel; this lane's levels are g * 32 + lane
  double dem[LPL][T];
#pragma unroll
  for (int g = 0; g < LPL; ++g) {
    const int ll = g * 32 + lane;
#pragma unroll
    for (int i = 0; i < T; ++i) dem[g][i] = dem_tile[((ll >> 1) * T + i) * 2 + (ll & 1)];
  }

  uint64_t rb_acc[LPL];
  uint32_t rb_ct[LPL], rb_w[LPL], rb_j[LPL];
#pragma unroll
  for (int g = 0; g < LPL; ++g) { rb_acc[g] = 0; rb_ct[g] = 0; rb_w[g] = 0; rb_j[g] = 0; }

  const uint32_t jbits = (uint32_t)p.jbits;
  const uint32_t jmul = 1u << jbits;
  const uint32_t jmask = jmul - 1u;
  const Rec* const recs = reinterpret_cast<const Rec*>(p.uni_members);
  const uint32_t SL = (uint32_t)p.uni_slices;
  const uint32_t n_units = (uint32_t)p.n_ct * SL;

  for (uint32_t u = blockIdx.x; u < n_units; u += gridDim.x) {
    const uint32_t ct = u / SL;
    const uint32_t sl = u - ct * SL;
    __syncwarp();
    // ---- stage the class tuple: member records, counts, path accuracy ----
    {
      uint32_t q = ct, off = 0;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        const uint32_t nc = (uint32_t)p.n_class[i];
        const uint32_t cls = q % nc;
        q /= nc;
        const int idx = p.class_off[i] + (int)cls;
        const uint32_t c = (uint32_t)p.class_count[idx];
        const Rec* src = recs + p.member_off[i] + p.class_first[idx];
        for (uint32_t m = lane; m < c; m += 32) s_rec[off + m] = src[m];
        if (lane == 0) {
          s_hdr[i] = c;
          s_hdr[8 + i] = off;
          s_hdr[16 + i] = (uint32_t)p.class_min_lat[idx];
          // a2: path accuracy products in task order (no fused multiply-add)
          const double a = p.class_acc[idx];
          s_pp[i] = i == 0 ? a : __dmul_rn(s_pp[p.parent[i]], a);
        }
        off += c;
      }
    }
    __syncwarp();
    double sum = s_pp[p.leaf_task[0]];
    for (int k = 1; k < p.n_leaves; ++k) sum = __dadd_rn(sum, s_pp[p.leaf_task[k]]);
    const uint64_t acc_bits = (uint64_t)__double_as_longlong(__ddiv_rn(sum, (double)p.n_leaves));

    Unit<T, NP> un;
    un.rec = s_rec;
    un.jmul = jmul;
    un.n_leaves = p.n_leaves;
#pragma unroll
    for (int k = 0; k < kMaxTasks; ++k) un.path_mask[k] = p.path_mask[k];
    {
      uint32_t st = 1;
      int32_t nd = 0;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        un.cnt[i] = s_hdr[i];
        un.roff[i] = s_hdr[8 + i];
        un.stride[i] = st;
        un.need[i] = nd;
        st *= un.cnt[i];
        nd += (int32_t)s_hdr[16 + i];
      }
    }
    // this unit's slice of the most significant digit
    const uint32_t top_begin = un.cnt[T - 1] * sl / SL, top_end = un.cnt[T - 1] * (sl + 1) / SL;
    if (top_begin >= top_end) continue;

    uint32_t best[LPL];
#pragma unroll
    for (int g = 0; g < LPL; ++g) best[g] = kEmpty;

    double rh[T][NP];
    constexpr int NS = CHAIN ? 1 : kMaxTasks;
    int32_t slack[NS];
    int32_t tight = 0x7FFFFFFF;
#pragma unroll
    for (int k = 0; k < NS; ++k) {
      slack[k] = k < p.n_leaves ? p.lat_limit[k] : 0x7FFFFFFF;
      tight = min(tight, slack[k]);
    }
    if constexpr (T == 1) walk_inner<T, NP, LPL>(un, top_begin, top_end, tight, 0u, rh, dem, best);
    else walk_outer<T - 1, T, NP, LPL, CHAIN>(un, top_begin, top_end, slack, 0u, rh, dem, best);

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
    partial[(size_t)blockIdx.x * LT + g * 32 + lane] = k;
  }
}

// Either launches (n_blocks > 0) or reports resident blocks per SM (n_blocks == 0).
template <int T, int NP, int LPL, bool CHAIN>
int act(const DirProblem* p, const double* dem_tile, int n_blocks, Key* d_partial, cudaStream_t st, int n_tiles) {
  if (n_blocks == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, uniform_score_kernel<T, NP, LPL, CHAIN>,
                                                      32, (size_t)p->uni_stage_bytes) != cudaSuccess)
      return 0;
    return n;
  }
  uniform_score_kernel<T, NP, LPL, CHAIN><<<dim3(n_blocks, n_tiles), 32, (size_t)p->uni_stage_bytes, st>>>(*p, dem_tile, d_partial);
  return (int)cudaGetLastError();
}

template <int NP, int LPL, bool CHAIN>
int by_tasks(int T, const DirProblem* p, const double* dem_tile, int n_blocks, Key* d_partial,
             cudaStream_t st, int n_tiles) {
  switch (T) {
    case 1: return act<1, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 2: return act<2, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 3: return act<3, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 4: return act<4, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 5: return act<5, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 6: return act<6, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 7: return act<7, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 8: return act<8, NP, LPL, CHAIN>(p, dem_tile, n_blocks, d_partial, st, n_tiles);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

template <int NP, int LPL>
int by_shape(bool chain, int T, const DirProblem* p, const double* dem_tile, int n_blocks,
             Key* d_partial, cudaStream_t st, int n_tiles) {
  return chain ? by_tasks<NP, LPL, true>(T, p, dem_tile, n_blocks, d_partial, st, n_tiles)
               : by_tasks<NP, LPL, false>(T, p, dem_tile, n_blocks, d_partial, st, n_tiles);
}

int dispatch(int T, int n_parts, int tile_levels, bool chain, const DirProblem* p,
             const double* dem_tile, int n_blocks, Key* d_partial, cudaStream_t st, int n_tiles) {
  const bool two = n_parts == 2;
  switch (tile_levels) {
    case 32: return two ? by_shape<2, 1>(chain, T, p, dem_tile, n_blocks, d_partial, st, n_tiles)
                        : by_shape<1, 1>(chain, T, p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 64: return two ? by_shape<2, 2>(chain, T, p, dem_tile, n_blocks, d_partial, st, n_tiles)
                        : by_shape<1, 2>(chain, T, p, dem_tile, n_blocks, d_partial, st, n_tiles);
    case 128: return two ? by_shape<2, 4>(chain, T, p, dem_tile, n_blocks, d_partial, st, n_tiles)
                         : by_shape<1, 4>(chain, T, p, dem_tile, n_blocks, d_partial, st, n_tiles);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

bool is_chain(const DirProblem& p) {
  return p.n_leaves == 1 && p.path_mask[0] == (p.T >= 32 ? 0xFFFFFFFFu : ((1u << p.T) - 1u));
}

}  // namespace

cudaError_t launch_uniform_score(const DirProblem& p, const double* d_dem_tile, int tile_levels,
                                 int n_blocks, Key* d_partial, cudaStream_t st, int n_tiles) {
  if (n_blocks < 1 || n_tiles < 1 || n_tiles > 65535) return cudaErrorInvalidValue;
  return (cudaError_t)dispatch(p.T, p.n_parts_max, tile_levels, is_chain(p), &p, d_dem_tile, n_blocks,
                               d_partial, st, n_tiles);
}

// Resident blocks (warps) per SM of the instantiation that serves this problem and tile.
int uniform_max_blocks_per_sm(const DirProblem& p, int tile_levels) {
  return dispatch(p.T, p.n_parts_max, tile_levels, is_chain(p), &p, nullptr, 0, nullptr, nullptr, 1);
}

}  // namespace loki
