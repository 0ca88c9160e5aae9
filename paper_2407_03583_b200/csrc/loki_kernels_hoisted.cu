// The hoisted (tabulated) scoring kernel of libloki_alloc.  With one fan-out factor
// per edge, the workers of a task (Eq. 2 with Eq. 5) depend on (demand level, task,
// option) only, not on the rest of the candidate.  The kernel therefore evaluates
// the worker arithmetic once per (level, task, class member) -- the same exact fma
// as the direct kernel, so the exactness argument is unchanged -- into a table in
// shared memory, and scores a (candidate, level) pair with one table read, one
// add and one minimum.  Every pair of a latency-feasible candidate is still
// visited (unless prefix minima are asked for, see below); what is hoisted is the
// arithmetic the pairs have in common.
//
// Mapping (as in the level-lane kernel): one warp per block; a lane owns LPL
// adjacent demand levels (LPL = 1, 2 or 4, tiles of 32, 64, 128), so that its
// table entries for one member are one 32-, 64- or 128-bit shared-memory read and a
// lane only ever reads entries it wrote itself.  A work unit is one slice of a
// class tuple along its most significant digit, units are dealt round-robin.
//
// Table entry of member m of task i for level l:
//     (workers(l, i, m) << jbits) + m * stride_i
// with stride_i the rank weight of digit i, so that the sum of a candidate's T
// entries is its packed key (workers << jbits | rank in the class tuple) and the
// nested walk -- one loop per task, task 0 innermost, partial sums carried down --
// needs no other per-candidate arithmetic.  A class is laid out in ascending task
// latency (the entry carries the member's own digit, so the order is free): the
// members that fit the latency slack the outer tasks leave (Eq. 7) are then a
// prefix, a digit loop can stop at the first member that does not fit, and since
// the slack only shrinks while digit 1 advances, the length of task 0's prefix is
// maintained with a pointer that only moves down.
//
// Prefix minima (HoistLayout::pmin_mode, LOKI_PATH_PREFIX).  The outer tasks add the same
// partial sum to every inner row, so the best inner row for a given slack is the minimum
// of the rows of the fitting prefix whatever the outer tasks chose.  After a class
// tuple's table is built, the inner rows (task 0's members, or the member pairs of the
// joined tasks 0 and 1) are replaced by their running minima, and the walk reads one row
// per fitting prefix instead of all of them.  Keys carry the rank, so ties still go to the
// lowest candidate index and the plans are those of the plain walk; the candidates of the
// innermost task are then no longer visited one by one.
#include "loki_internal.h"

namespace loki {

// defined in loki_kernels_hoisted_l1/_l2/_l4.cu: launch (n_blocks > 0) or occupancy query (n_blocks == 0)
int hoisted_dispatch_l1(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks,
                        Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits);
int hoisted_dispatch_l2(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks,
                        Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits);
int hoisted_dispatch_l4(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks,
                        Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos, const int32_t* slo_limits);

int prefix_dispatch_l1(const void* call);
int prefix_dispatch_l2(const void* call);
int prefix_dispatch_l4(const void* call);

namespace {

int prefix_dispatch(int tile_levels, const PrefixCall& c) {
  switch (tile_levels) {
    case 32: return prefix_dispatch_l1(&c);
    case 64: return prefix_dispatch_l2(&c);
    case 128: return prefix_dispatch_l4(&c);
    default: return c.build || c.n_blocks > 0 ? (int)cudaErrorInvalidValue : 0;
  }
}

int dispatch(const DirProblem* p, const HoistLayout* lay, int tile_levels, LevelSpan dem_tile,
             int n_blocks, Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos,
             const int32_t* slo_limits) {
  switch (tile_levels) {
    case 32: return hoisted_dispatch_l1(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 64: return hoisted_dispatch_l2(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    case 128: return hoisted_dispatch_l4(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
    default: return n_blocks == 0 ? 0 : (int)cudaErrorInvalidValue;
  }
}

}  // namespace
cudaError_t launch_hoisted_score(const DirProblem& p, const HoistLayout& lay, LevelSpan d_dem_tile,
                                 int tile_levels, int n_blocks, Key* d_partial, cudaStream_t st,
                                 bool zero_demand, int n_tiles, int n_slos, const int32_t* d_slo_limits) {
  if (n_blocks < 1 || n_tiles < 1 || n_tiles > 65535 || n_slos < 1 || n_slos > 65535) return cudaErrorInvalidValue;
  return (cudaError_t)dispatch(&p, &lay, tile_levels, d_dem_tile, n_blocks, d_partial, st, zero_demand ? 1 : 0,
                               n_tiles, n_slos, d_slo_limits);
}

cudaError_t launch_prefix_build(const DirProblem& p, const PrefixTables& t, LevelSpan span, int tile_levels,
                                int n_tiles, cudaStream_t st) {
  if (n_tiles < 1 || n_tiles > 65535 || t.n_rows < 1) return cudaErrorInvalidValue;
  const PrefixCall c{&p, &t, span, 1, 0, n_tiles, 0, 1, nullptr, nullptr, st};
  return (cudaError_t)prefix_dispatch(tile_levels, c);
}

cudaError_t launch_prefix_walk(const DirProblem& p, const PrefixTables& t, LevelSpan span, int tile_levels,
                               int tile0, int n_tiles, int n_blocks, Key* d_partial, cudaStream_t st,
                               int n_slos, const int32_t* d_slo_limits) {
  if (n_blocks < 1 || n_tiles < 1 || n_tiles > 65535 || n_slos < 1 || n_slos > 65535 || tile0 < 0)
    return cudaErrorInvalidValue;
  const PrefixCall c{&p, &t, span, 0, tile0, n_tiles, n_blocks, n_slos, d_partial, d_slo_limits, st};
  return (cudaError_t)prefix_dispatch(tile_levels, c);
}

int prefix_walk_max_blocks_per_sm(const DirProblem& p, const PrefixTables& t, int tile_levels) {
  const PrefixCall c{&p, &t, LevelSpan{nullptr, 0, 0}, 0, 0, 1, 0, 1, nullptr, nullptr, nullptr};
  return prefix_dispatch(tile_levels, c);
}

// Resident blocks (warps) per SM of the instantiation that serves this problem and tile.
int hoisted_max_blocks_per_sm(const DirProblem& p, const HoistLayout& lay, int tile_levels) {
  return dispatch(&p, &lay, tile_levels, LevelSpan{nullptr, 0, 0}, 0, nullptr, nullptr, 0, 1, 1, nullptr);
}

}  // namespace loki
