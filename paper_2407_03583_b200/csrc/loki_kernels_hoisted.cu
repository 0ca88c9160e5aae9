// The hoisted scoring kernel of libloki_alloc.  With one fan-out factor per edge
// the workers a task needs depend on (level, task, option) only, not on the rest
// of the candidate (Eq. 2 of the paper couples tasks only through the sum of
// Eq. 3).  A block therefore tabulates, per class tuple, the worker count of every
// member option of every task for the levels of the tile in shared memory --
// with the same exact fma as the direct kernel -- and then scores every
// (candidate, level) pair with one table read, one add and one minimum, keeping
// the partial sums of the slower digits in registers.  Every pair is still
// evaluated; only the per-task arithmetic is shared between candidates.
//
// Mapping: thread = (level of the tile, slice); a slice walks the outer digits
// (tasks 1..T-1 of the candidate's rank in the class tuple) round robin and runs
// the task-0 digit in the inner loop.  Lanes of a warp hold consecutive levels,
// so table rows are read without bank conflicts and the candidate is
// warp-uniform: the latency test (Eqs. 6-7) is a uniform branch.
#include "loki_internal.h"

namespace loki {

namespace {

constexpr int kHoistThreads = 128;
constexpr double kMagic = 6755399441055744.0;   // 1.5 * 2^52
constexpr uint32_t kEmpty = 0xFFFFFFFFu;

template <int T>
__device__ __forceinline__ int64_t cand_index_h(const DirProblem& p, uint64_t ct, uint32_t j) {
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

constexpr int kInnerCache = 16;   // task-0 members held in registers by the inner loop

// Depth-first walk over the member digits of a class tuple for one thread
// (= one level of the tile).  NL is the number of leaf paths the latency test
// tracks (kMaxTasks = any number, checked against n_leaves at run time).
template <int T, int LT, int NL>
struct Walk {
  const uint32_t* rows;
  const int32_t* lat;
  const HoistLayout* lay;
  uint32_t cnt[T];
  uint32_t stride[T];               // rank stride of each digit
  uint32_t tmask[T];                // bit k set: task lies on leaf path k
  uint32_t r0[kInnerCache];
  int32_t l0[kInnerCache];
  int cache;                        // 0: inner loop reads shared memory; else 8 or 16 cached members
  int l;
  uint32_t jmul, best;

  template <int W>
  __device__ __forceinline__ void inner_cached(uint32_t rest, int32_t s, uint32_t jbase) {
#pragma unroll
    for (int d = 0; d < W; ++d)
      if (l0[d] <= s)                  // warp-uniform; padded entries never pass
        best = min(best, (rest + r0[d]) * jmul + (jbase + (uint32_t)d));
  }

  // I: task whose digit this level iterates; rest: workers of the tasks above;
  // slack[k]: latency still available on leaf path k; jbase: rank so far.
  template <int I>
  __device__ __forceinline__ void run(uint32_t rest, const int32_t (&slack)[NL], uint32_t jbase,
                                      int first, int step) {
    if constexpr (I == 0) {
      int32_t s = slack[0];               // task 0 is the root: it lies on every path
#pragma unroll
      for (int k = 1; k < NL; ++k) s = min(s, slack[k]);
      if (cache == 8 && step == 1) {
        inner_cached<8>(rest, s, jbase);
      } else if (cache == 16 && step == 1) {
        inner_cached<16>(rest, s, jbase);
      } else {
        const uint32_t* row0 = rows + lay->row_base[0] + l;
        const int32_t* lat0 = lat + lay->lat_off[0];
        for (uint32_t d = (uint32_t)first; d < cnt[0]; d += (uint32_t)step)
          if (lat0[d] <= s) best = min(best, (rest + row0[d * LT]) * jmul + (jbase + d));
      }
    } else {
      const uint32_t* rowi = rows + lay->row_base[I] + l;
      const int32_t* lati = lat + lay->lat_off[I];
      for (uint32_t d = (uint32_t)first; d < cnt[I]; d += (uint32_t)step) {
        const int32_t li = lati[d];
        int32_t sl[NL];
        bool any = true;
#pragma unroll
        for (int k = 0; k < NL; ++k) {
          sl[k] = slack[k] - (((tmask[I] >> k) & 1u) ? li : 0);
          any &= sl[k] >= 0;
        }
        if (!any) continue;                // no completion of this prefix can meet the SLO
        run<I - 1>(rest + rowi[d * LT], sl, jbase + d * stride[I], 0, 1);
      }
    }
  }
};

template <int T, int NP, int LT, int NL>
__global__ void __launch_bounds__(kHoistThreads)
hoisted_score_kernel(const __grid_constant__ DirProblem p, const __grid_constant__ HoistLayout lay,
                     const double* __restrict__ dem_tile, Key* __restrict__ partial) {
  constexpr int NS = kHoistThreads / LT;      // slices
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* s_rows = reinterpret_cast<uint32_t*>(smem_raw);                 // [task][member][LT]
  int32_t* s_lat = reinterpret_cast<int32_t*>(smem_raw) + lay.lat_base;    // [task][member]
  uint32_t* s_red = reinterpret_cast<uint32_t*>(smem_raw) + lay.red_base;  // [NS][LT]
  __shared__ double s_pp[kMaxTasks];
  __shared__ unsigned long long s_acc_bits;

  const int l = threadIdx.x % LT;
  const int slice = threadIdx.x / LT;
  const uint32_t jmul = 1u << p.jbits;
  const uint32_t jmask = jmul - 1u;

  // running best of level l, held by the threads of slice 0
  uint64_t rb_acc = 0, rb_ct = 0;
  uint32_t rb_w = 0, rb_j = 0;

  for (uint64_t ct = blockIdx.x; ct < (uint64_t)p.n_ct; ct += gridDim.x) {
    // ---- class tuple set-up (block-uniform) ----
    uint32_t cnt[T], inv[T];
    int64_t mem_base[T];
    {
      uint64_t r = ct;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        const uint32_t nc = (uint32_t)p.n_class[i];
        const uint32_t cls = (uint32_t)(r % nc);
        r /= nc;
        const int idx = p.class_off[i] + (int)cls;
        cnt[i] = (uint32_t)p.class_count[idx];
        inv[i] = 0xFFFFFFFFu / cnt[i] + 1u;
        mem_base[i] = p.member_off[i] + p.class_first[idx];
        if (threadIdx.x == 0) {
          // a2: path accuracy products in task order (no fused multiply-add)
          const double a = p.class_acc[idx];
          s_pp[i] = i == 0 ? a : __dmul_rn(s_pp[p.parent[i]], a);
        }
      }
      if (threadIdx.x == 0) {
        double sum = s_pp[p.leaf_task[0]];
        for (int k = 1; k < p.n_leaves; ++k) sum = __dadd_rn(sum, s_pp[p.leaf_task[k]]);
        s_acc_bits = (unsigned long long)__double_as_longlong(__ddiv_rn(sum, (double)p.n_leaves));
      }
    }
    // ---- a4/a5 hoisted: workers of every member option at every level of the tile ----
#pragma unroll
    for (int i = 0; i < T; ++i) {
      for (uint32_t x = threadIdx.x; x < cnt[i] * LT; x += kHoistThreads) {
        const uint32_t m = x / LT, ll = x % LT;
        const DirRec* rec = p.members + mem_base[i] + m;
        const double d = dem_tile[((ll >> 1) * T + i) * 2 + (ll & 1)];
        double acc = __fma_rd(d, rec->r[0], kMagic);
        if (NP == 2) acc = __fma_rd(d, rec->r[1], acc);
        s_rows[lay.row_base[i] + m * LT + ll] = (uint32_t)__double2loint(acc) + (uint32_t)rec->n_real;
        if (ll == 0) s_lat[lay.lat_off[i] + m] = rec->lat;
      }
    }
    __syncthreads();
    const uint64_t acc_bits = s_acc_bits;

    // ---- a1/a3/a6/a7: every candidate of the class tuple ----
    // Nested loops over the member digits, task T-1 outermost: the worker sum and
    // the per-path latency of the outer tasks are carried down, so a candidate
    // costs one add, one pack and one minimum plus its share of the outer steps.
    Walk<T, LT, NL> w;
    w.rows = s_rows; w.lat = s_lat; w.lay = &lay;
    w.l = l; w.jmul = jmul; w.best = kEmpty;
    {
      uint32_t st = 1;
#pragma unroll
      for (int i = 0; i < T; ++i) {
        w.cnt[i] = cnt[i];
        w.stride[i] = st;
        st *= cnt[i];
        uint32_t m = 0;
#pragma unroll
        for (int k = 0; k < NL; ++k)
          if (k < p.n_leaves && ((p.path_mask[k] >> i) & 1u)) m |= 1u << k;
        w.tmask[i] = m;
      }
    }
    // task 0's column of the table and its latencies, in registers when they fit
    w.cache = cnt[0] <= 8u ? 8 : cnt[0] <= (uint32_t)kInnerCache ? 16 : 0;
#pragma unroll
    for (int d = 0; d < kInnerCache; ++d) {
      const bool in = (uint32_t)d < cnt[0];
      w.r0[d] = in ? s_rows[lay.row_base[0] + d * LT + l] : 0u;
      w.l0[d] = in ? s_lat[lay.lat_off[0] + d] : 0x7FFFFFFF;
    }
    int32_t slack[NL];
#pragma unroll
    for (int k = 0; k < NL; ++k) slack[k] = k < p.n_leaves ? p.lat_limit[k] : 0x7FFFFFFF;
    if constexpr (T >= 3) {
      // the two outermost digits are dealt out to the slices together (better balance)
      const uint32_t c1 = cnt[T - 1], c2 = cnt[T - 2];
      for (uint32_t u = (uint32_t)slice; u < c1 * c2; u += (uint32_t)NS) {
        const uint32_t dA = u / c2, dB = u - dA * c2;        // digits of tasks T-1 and T-2
        const int32_t la = s_lat[lay.lat_off[T - 1] + dA], lb = s_lat[lay.lat_off[T - 2] + dB];
        int32_t sl[NL];
        bool any = true;
#pragma unroll
        for (int k = 0; k < NL; ++k) {
          sl[k] = slack[k] - (((w.tmask[T - 1] >> k) & 1u) ? la : 0) - (((w.tmask[T - 2] >> k) & 1u) ? lb : 0);
          any &= sl[k] >= 0;
        }
        if (!any) continue;
        const uint32_t rest = s_rows[lay.row_base[T - 1] + dA * LT + l] +
                              s_rows[lay.row_base[T - 2] + dB * LT + l];
        w.template run<T - 3>(rest, sl, dA * w.stride[T - 1] + dB * w.stride[T - 2], 0, 1);
      }
    } else {
      w.template run<T - 1>(0u, slack, 0u, slice, NS);
    }
    const uint32_t best = w.best;

    // ---- a8: minimum over the slices, merge into the running best of the level ----
    s_red[slice * LT + l] = best;
    __syncthreads();
    if (slice == 0) {
      uint32_t key = best;
#pragma unroll
      for (int s = 1; s < NS; ++s) key = min(key, s_red[s * LT + l]);
      if (key != kEmpty) {
        const uint32_t W = key >> p.jbits;
        const uint32_t jj = key & jmask;
        if (W <= (uint32_t)p.S) {
          bool better = acc_bits > rb_acc || (acc_bits == rb_acc && W < rb_w);
          if (!better && acc_bits == rb_acc && W == rb_w)
            better = cand_index_h<T>(p, ct, jj) < cand_index_h<T>(p, rb_ct, rb_j);
          if (better) { rb_acc = acc_bits; rb_w = W; rb_ct = ct; rb_j = jj; }
        }
      }
    }
    __syncthreads();                      // the tables are rebuilt for the next class tuple
  }

  // one partial key per (block, level)
  if (slice == 0) {
    Key k{0ull, 0ull};
    if (rb_acc != 0) {
      const int64_t c = cand_index_h<T>(p, rb_ct, rb_j);
      k.acc_bits = rb_acc;
      k.tail = ((uint64_t)((uint32_t)p.S - rb_w) << 40) | (uint64_t)(p.N - 1 - c);
    }
    partial[(size_t)blockIdx.x * LT + l] = k;
  }
}

template <int T, int NP, int LT, int NL>
int act_nl(const DirProblem* p, const HoistLayout* lay, const double* dem_tile, int n_blocks,
           Key* d_partial, cudaStream_t st) {
  auto kern = hoisted_score_kernel<T, NP, LT, NL>;
  const size_t smem = lay ? (size_t)lay->smem_bytes : 0;
  if (n_blocks == 0) {       // occupancy query for the given dynamic shared memory
    int n = 0;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kHoistThreads, smem) != cudaSuccess)
      return 0;
    return n;
  }
  kern<<<n_blocks, kHoistThreads, smem, st>>>(*p, *lay, dem_tile, d_partial);
  return (int)cudaGetLastError();
}

// chains (one leaf) and two-leaf trees get their own instantiation; others the general one
template <int T, int NP, int LT>
int act(const DirProblem* p, const HoistLayout* lay, const double* dem_tile, int n_blocks,
        Key* d_partial, cudaStream_t st) {
  const int nl = lay->n_leaves;
  if (nl == 1) return act_nl<T, NP, LT, 1>(p, lay, dem_tile, n_blocks, d_partial, st);
  if (nl == 2) return act_nl<T, NP, LT, 2>(p, lay, dem_tile, n_blocks, d_partial, st);
  return act_nl<T, NP, LT, kMaxTasks>(p, lay, dem_tile, n_blocks, d_partial, st);
}

template <int NP, int LT>
int by_tasks(int T, const DirProblem* p, const HoistLayout* lay, const double* dem_tile,
             int n_blocks, Key* d_partial, cudaStream_t st) {
  switch (T) {
    case 1: return act<1, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 2: return act<2, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 3: return act<3, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 4: return act<4, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 5: return act<5, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 6: return act<6, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 7: return act<7, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    case 8: return act<8, NP, LT>(p, lay, dem_tile, n_blocks, d_partial, st);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

int dispatch(int T, int n_parts, int tile_levels, const DirProblem* p, const HoistLayout* lay,
             const double* dem_tile, int n_blocks, Key* d_partial, cudaStream_t st) {
  const bool two = n_parts == 2;
  if (tile_levels == kDirectTile)
    return two ? by_tasks<2, kDirectTile>(T, p, lay, dem_tile, n_blocks, d_partial, st)
               : by_tasks<1, kDirectTile>(T, p, lay, dem_tile, n_blocks, d_partial, st);
  if (tile_levels == kDirectTileSmall)
    return two ? by_tasks<2, kDirectTileSmall>(T, p, lay, dem_tile, n_blocks, d_partial, st)
               : by_tasks<1, kDirectTileSmall>(T, p, lay, dem_tile, n_blocks, d_partial, st);
  return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_hoisted_score(const DirProblem& p, const HoistLayout& lay, const double* d_dem_tile,
                                 int tile_levels, int n_blocks, Key* d_partial, cudaStream_t st) {
  if (n_blocks < 1) return cudaErrorInvalidValue;
  return (cudaError_t)dispatch(p.T, p.n_parts_max, tile_levels, &p, &lay, d_dem_tile, n_blocks,
                               d_partial, st);
}

// Resident blocks per SM for this problem's shared-memory layout (0 if it does not fit).
int hoisted_max_blocks_per_sm(int T, int n_parts, int tile_levels, const HoistLayout& lay) {
  return dispatch(T, n_parts, tile_levels, nullptr, &lay, nullptr, 0, nullptr, nullptr);
}

}  // namespace loki
