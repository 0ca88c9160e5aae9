// The direct scoring kernel of libloki_alloc: every (candidate, demand level)
// pair is scored with the full per-task worker arithmetic.  Hand-written CUDA
// for sm_100a; bound by the FP64 pipe (one fused multiply-add per option part
// and pair), not by memory.
//
// Mapping.  Candidates are grouped into class tuples: per task, options with
// bit-identical task accuracy form a class, so all candidates of a class tuple
// have the same end-to-end accuracy and differ only in workers.  A warp walks a
// contiguous run of iterations of 32 * CB candidates; lanes hold candidates
// (their reciprocal constants live in registers; CB = 2 per lane in split mode so
// that every demand operand fetched feeds more fmas), the demand levels of the current
// tile are an unrolled loop whose stage demands are compile-time offsets into
// constant memory, and the running best of every level is one packed 32-bit
// register per lane: (workers << jbits) | rank-in-class-tuple, so that an
// unsigned minimum implements "fewest workers, then lowest candidate index".
// At the end of a class tuple the warp reduces each level with a single
// redux.sync and merges it into a lane-distributed running best that carries
// the accuracy.
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
#include "loki_internal.h"

#include <utility>

// Demand operands of the current tile, layout [level pair][task][2].  C linkage
// gives the symbol a name that the inline assembly below can spell.
extern "C" {
__constant__ __align__(16) double loki_direct_dem[loki::kDirectTile * loki::kMaxTasks];
}

namespace loki {

namespace {

// Levels advanced together (independent fma chains per candidate): four, or two
// where the candidates' constants already fill most of the register budget.
__host__ __device__ constexpr int level_step(int T, int NP, int CB) { return CB * T * NP >= 24 ? 2 : 4; }

constexpr double kMagic = 6755399441055744.0;   // 1.5 * 2^52: ulp 1, low mantissa word 0

constexpr uint32_t kEmpty = 0xFFFFFFFFu;

// One demand operand at a compile-time offset.  The load is issued afresh at every
// use (asm volatile keeps the compiler from hoisting the loop-invariant loads of
// a whole tile into registers, which would cost more registers than the kernel has).
template <int IDX>
__device__ __forceinline__ double dem_operand() {
  double x;
  asm volatile("ld.const.f64 %0, [loki_direct_dem+%1];" : "=d"(x) : "n"(IDX * 8));
  return x;
}

// Compile-time loop: f(integral_constant<int, 0>) ... f(integral_constant<int, N - 1>).
template <int... Is, class F>
__device__ __forceinline__ void static_for(std::integer_sequence<int, Is...>, F&& f) {
  (f(std::integral_constant<int, Is>{}), ...);
}

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

template <int T, int NP, int LT>
__global__ void __launch_bounds__(kDirectThreads, 3)   // at most 168 registers: three blocks per SM
direct_score_kernel(const __grid_constant__ DirProblem p, Key* __restrict__ partial) {
  constexpr int CB = direct_cands_per_lane(NP);
  constexpr int NB = (LT + 31) / 32;          // running-best slots per lane
  constexpr int WARPS = kDirectThreads / 32;
  constexpr int kLevelStep = level_step(T, NP, CB);
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  const uint64_t gw = (uint64_t)blockIdx.x * WARPS + wib;
  const uint64_t nw = (uint64_t)gridDim.x * WARPS;
  const uint64_t it_begin = (uint64_t)p.total_iters * gw / nw;
  const uint64_t it_end = (uint64_t)p.total_iters * (gw + 1) / nw;

  __shared__ double s_pp[WARPS][kMaxTasks];
  __shared__ Key s_keys[WARPS][LT];

  uint64_t rb_acc[NB], rb_ct[NB];
  uint32_t rb_w[NB], rb_j[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) { rb_acc[b] = 0; rb_ct[b] = 0; rb_w[b] = 0; rb_j[b] = 0; }

  uint32_t jmul = 1u << p.jbits;
  const uint32_t jmask = jmul - 1u;
  // Opaque to the compiler from here on: the key is then formed by one integer
  // multiply-add on the otherwise idle FMA pipe instead of a shift and an add, and
  // the accumulators start from a register instead of a re-materialised constant.
  asm volatile("" : "+r"(jmul));
  double magic = kMagic;
  asm volatile("" : "+d"(magic));

  if (it_begin < it_end) {
    // class tuple holding iteration it_begin: largest ct with prefix[ct] <= it_begin
    uint64_t lo = 0, hi = (uint64_t)p.n_ct;     // invariant: prefix[lo] <= it_begin < prefix[hi]
    while (hi - lo > 1) {
      const uint64_t mid = (lo + hi) >> 1;
      if (p.iter_prefix[mid] <= it_begin) lo = mid; else hi = mid;
    }
    uint64_t ct = lo;
    uint64_t it = it_begin;
    while (it < it_end) {
      // ---- class tuple set-up (warp-uniform) ----
      uint32_t cnt[T], inv[T];
      int64_t mem_base[T];
      uint32_t J = 1;
      {
        uint64_t r = ct;
#pragma unroll
        for (int i = 0; i < T; ++i) {
          const uint32_t nc = (uint32_t)p.n_class[i];
          const uint32_t cls = (uint32_t)(r % nc);
          r /= nc;
          const int idx = p.class_off[i] + (int)cls;
          cnt[i] = (uint32_t)p.class_count[idx];
          inv[i] = 0xFFFFFFFFu / cnt[i] + 1u;     // x / cnt == umulhi(x, inv) while x * cnt < 2^32
          mem_base[i] = p.member_off[i] + p.class_first[idx];
          J *= cnt[i];
          // a2: path accuracy products in task order (no fused multiply-add)
          const double a = p.class_acc[idx];
          if (lane == 0) s_pp[wib][i] = i == 0 ? a : __dmul_rn(s_pp[wib][p.parent[i]], a);
        }
      }
      __syncwarp();
      double sum = s_pp[wib][p.leaf_task[0]];
      for (int k = 1; k < p.n_leaves; ++k) sum = __dadd_rn(sum, s_pp[wib][p.leaf_task[k]]);
      const uint64_t acc_bits = (uint64_t)__double_as_longlong(__ddiv_rn(sum, (double)p.n_leaves));
      __syncwarp();

      const uint64_t ct_first = p.iter_prefix[ct];
      const uint64_t ct_iters = p.iter_prefix[ct + 1] - ct_first;
      const uint32_t li0 = (uint32_t)(it - ct_first);
      const uint64_t room = it_end - it;
      const uint32_t li1 = (uint32_t)((ct_iters - li0) < room ? ct_iters : li0 + room);

      uint32_t best[LT];
#pragma unroll
      for (int l = 0; l < LT; ++l) best[l] = kEmpty;

      for (uint32_t li = li0; li < li1; ++li) {
        // ---- a1: decode this lane's CB candidates, fetch their constants ----
        double rr[CB][T][NP];
        uint32_t kconst[CB];
        bool any_alive = false;
#pragma unroll
        for (int c = 0; c < CB; ++c) {
          const uint32_t j = (li * CB + c) * 32u + (uint32_t)lane;
          bool alive = j < J;
          int32_t lat[T];
          uint32_t base = 0;
          uint32_t r = alive ? j : 0u;
#pragma unroll
          for (int i = 0; i < T; ++i) {
            const uint32_t q = __umulhi(r, inv[i]);
            const uint32_t d = r - q * cnt[i];
            r = q;
            const DirRec* rec = p.members + mem_base[i] + d;
            const double2 a = *reinterpret_cast<const double2*>(&rec->r[0]);
            rr[c][i][0] = a.x;
            if (NP == 2) rr[c][i][NP - 1] = a.y;
            const int2 m = *reinterpret_cast<const int2*>(&rec->lat);
            lat[i] = m.x;
            base += (uint32_t)m.y;
          }
          // ---- a3: latency bound on every root-to-leaf path ----
          for (int k = 0; k < p.n_leaves; ++k) {
            int32_t pl = 0;
#pragma unroll
            for (int i = 0; i < T; ++i)
              if ((p.path_mask[k] >> i) & 1u) pl += lat[i];
            alive &= pl <= p.lat_limit[k];
          }
          kconst[c] = (base << p.jbits) | j;
          if (!alive) {
            kconst[c] = kEmpty;
#pragma unroll
            for (int i = 0; i < T; ++i)
#pragma unroll
              for (int s = 0; s < NP; ++s) rr[c][i][s] = 0.0;
          }
          any_alive |= alive;
        }
        if (!__any_sync(0xFFFFFFFFu, any_alive)) continue;
        // ---- a5-a7: workers per task, packed key, running minimum per level ----
        // kLevelStep levels are advanced together, so that kLevelStep * CB independent
        // fma chains are in flight per warp.
        static_for(std::make_integer_sequence<int, LT / kLevelStep>{}, [&](auto lp) {
          constexpr int l0 = kLevelStep * decltype(lp)::value;
          double acc[kLevelStep][CB];
#pragma unroll
          for (int g = 0; g < kLevelStep; ++g)
#pragma unroll
            for (int c = 0; c < CB; ++c) acc[g][c] = magic;
          static_for(std::make_integer_sequence<int, T>{}, [&](auto ti) {
            constexpr int i = decltype(ti)::value;
            static_for(std::make_integer_sequence<int, kLevelStep>{}, [&](auto gi) {
              constexpr int g = decltype(gi)::value;
              constexpr int l = l0 + g;
              const double d = dem_operand<((l / 2) * T + i) * 2 + (l & 1)>();
#pragma unroll
              for (int s = 0; s < NP; ++s)
#pragma unroll
                for (int c = 0; c < CB; ++c) acc[g][c] = __fma_rd(d, rr[c][i][s], acc[g][c]);
            });
          });
#pragma unroll
          for (int g = 0; g < kLevelStep; ++g) {
            uint32_t b = best[l0 + g];
#pragma unroll
            for (int c = 0; c < CB; ++c)
              b = min(b, (uint32_t)__double2loint(acc[g][c]) * jmul + kconst[c]);
            best[l0 + g] = b;
          }
        });
      }

      // ---- flush: warp minimum per level, merge into the running best ----
      uint32_t got[NB];
#pragma unroll
      for (int b = 0; b < NB; ++b) got[b] = kEmpty;
#pragma unroll
      for (int l = 0; l < LT; ++l) {
        const uint32_t r = __reduce_min_sync(0xFFFFFFFFu, best[l]);
        if ((l & 31) == lane) got[l >> 5] = r;
      }
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        const uint32_t key = got[b];
        if (key == kEmpty) continue;
        const uint32_t W = key >> p.jbits;
        const uint32_t jj = key & jmask;
        if (W > (uint32_t)p.S) continue;
        bool better = acc_bits > rb_acc[b] || (acc_bits == rb_acc[b] && W < rb_w[b]);
        if (!better && acc_bits == rb_acc[b] && W == rb_w[b])
          better = cand_index<T>(p, ct, jj) < cand_index<T>(p, rb_ct[b], rb_j[b]);
        if (better) { rb_acc[b] = acc_bits; rb_w[b] = W; rb_ct[b] = ct; rb_j[b] = jj; }
      }
      it += (uint64_t)(li1 - li0);
      ++ct;
    }
  }

  // ---- a8: block argmax per level, one partial key per (block, level) ----
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const int l = b * 32 + lane;
    if (l < LT) {
      Key k{0ull, 0ull};
      if (rb_acc[b] != 0) {
        const int64_t c = cand_index<T>(p, rb_ct[b], rb_j[b]);
        k.acc_bits = rb_acc[b];
        k.tail = ((uint64_t)((uint32_t)p.S - rb_w[b]) << 40) | (uint64_t)(p.N - 1 - c);
      }
      s_keys[wib][l] = k;
    }
  }
  __syncthreads();
  if (threadIdx.x < LT) {
    Key k = s_keys[0][threadIdx.x];
#pragma unroll
    for (int w = 1; w < WARPS; ++w)
      if (key_less(k, s_keys[w][threadIdx.x])) k = s_keys[w][threadIdx.x];
    partial[(size_t)blockIdx.x * LT + threadIdx.x] = k;
  }
}

template <int T, int NP, int LT>
cudaError_t launch_one(const DirProblem& p, int n_blocks, Key* d_partial, cudaStream_t st) {
  direct_score_kernel<T, NP, LT><<<n_blocks, kDirectThreads, 0, st>>>(p, d_partial);
  return cudaGetLastError();
}

template <int T, int NP, int LT>
int occ_one() {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, direct_score_kernel<T, NP, LT>,
                                                    kDirectThreads, 0) != cudaSuccess)
    return 0;
  return n;
}

// Either launches (n_blocks > 0) or reports resident blocks per SM (n_blocks == 0).
template <int T, int NP, int LT>
int act(const DirProblem* p, int n_blocks, Key* d_partial, cudaStream_t st) {
  if (n_blocks == 0) return occ_one<T, NP, LT>();
  return (int)launch_one<T, NP, LT>(*p, n_blocks, d_partial, st);
}

template <int NP, int LT>
int by_tasks(int T, const DirProblem* p, int n_blocks, Key* d_partial, cudaStream_t st) {
  switch (T) {
    case 1: return act<1, NP, LT>(p, n_blocks, d_partial, st);
    case 2: return act<2, NP, LT>(p, n_blocks, d_partial, st);
    case 3: return act<3, NP, LT>(p, n_blocks, d_partial, st);
    case 4: return act<4, NP, LT>(p, n_blocks, d_partial, st);
    case 5: return act<5, NP, LT>(p, n_blocks, d_partial, st);
    case 6: return act<6, NP, LT>(p, n_blocks, d_partial, st);
    case 7: return act<7, NP, LT>(p, n_blocks, d_partial, st);
    case 8: return act<8, NP, LT>(p, n_blocks, d_partial, st);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

int dispatch(int T, int n_parts, int tile_levels, const DirProblem* p, int n_blocks,
             Key* d_partial, cudaStream_t st) {
  const bool two = n_parts == 2;
  if (tile_levels == kDirectTile)
    return two ? by_tasks<2, kDirectTile>(T, p, n_blocks, d_partial, st)
               : by_tasks<1, kDirectTile>(T, p, n_blocks, d_partial, st);
  if (tile_levels == kDirectTileSmall)
    return two ? by_tasks<2, kDirectTileSmall>(T, p, n_blocks, d_partial, st)
               : by_tasks<1, kDirectTileSmall>(T, p, n_blocks, d_partial, st);
  return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
}

}  // namespace

bool direct_supported(int T, int split) { return T >= 1 && T <= kMaxTasks && (split == 0 || split == 1); }

cudaError_t direct_upload_tile(const double* d_demf_tile, int n_doubles, cudaStream_t st) {
  return cudaMemcpyToSymbolAsync(loki_direct_dem, d_demf_tile, sizeof(double) * n_doubles, 0,
                                 cudaMemcpyDeviceToDevice, st);
}

cudaError_t launch_direct_score(const DirProblem& p, int tile_levels, int n_blocks, Key* d_partial,
                                cudaStream_t st) {
  if (n_blocks < 1) return cudaErrorInvalidValue;
  return (cudaError_t)dispatch(p.T, p.n_parts_max, tile_levels, &p, n_blocks, d_partial, st);
}

// Resident blocks per SM of the instantiation that serves (T, n_parts, tile).
int direct_max_blocks_per_sm(int T, int n_parts, int tile_levels) {
  return dispatch(T, n_parts, tile_levels, nullptr, 0, nullptr, nullptr);
}

}  // namespace loki
