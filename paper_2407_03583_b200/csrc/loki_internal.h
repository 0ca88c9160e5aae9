// Internal declarations shared by the host planner and the CUDA kernels of
// libloki_alloc.  Not part of the public interface.
#ifndef LOKI_INTERNAL_H_
#define LOKI_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>

#include "loki_alloc.h"

namespace loki {

constexpr int kMaxTasks = LOKI_MAX_TASKS;
constexpr int kDirectMaxTile = 256;    // demand levels per launch of the direct kernel, at most
// The direct kernel scores a tile in groups of G levels whose G x T stage demands are resident
// operands of the loop over the staged candidates (at most 30 doubles).
__host__ __device__ constexpr int direct_group_levels(int T) { return 30 / T > 16 ? 16 : 30 / T; }
// Doubles a group occupies in the demand tile: its G x T operands [level in group][task], padded to an
// even count so that every group starts on a 16-byte boundary.
__host__ __device__ constexpr int direct_group_stride(int T) { return (direct_group_levels(T) * T + 1) / 2 * 2; }
// Offset of (level, task) within a tile of the direct kernel's demand layout.
__host__ __device__ constexpr int direct_dem_offset(int T, int level, int task) {
  return level / direct_group_levels(T) * direct_group_stride(T) + level % direct_group_levels(T) * T + task;
}
// The last group of a tile may be shorter than G: about two thirds or one third of it, so that a
// tile is padded by less than a third of a group.
__host__ __device__ constexpr int direct_short_group(int T, int which) {
  return which == 0 ? direct_group_levels(T)
       : which == 1 ? (2 * direct_group_levels(T) + 2) / 3 : (direct_group_levels(T) + 2) / 3;
}
// Levels of the last group of a tile that holds `levels` levels: the smallest admitted size that takes
// what the whole groups before it leave.
__host__ __device__ constexpr int direct_last_group_levels(int T, int levels) {
  const int G = direct_group_levels(T);
  const int rest = levels - (levels - 1) / G * G;      // 1 .. G
  return rest <= direct_short_group(T, 2) ? direct_short_group(T, 2)
       : rest <= direct_short_group(T, 1) ? direct_short_group(T, 1) : G;
}
// Levels a tile of `levels` levels scores: whole groups and the last group.
__host__ __device__ constexpr int direct_tile_levels(int T, int levels) {
  return (levels - 1) / direct_group_levels(T) * direct_group_levels(T) + direct_last_group_levels(T, levels);
}
// Every tile takes its levels, is padded by less than a third of a group (rounded up), and ends
// in a group of an admitted size.
constexpr bool direct_tiles_consistent() {
  for (int T = 1; T <= kMaxTasks; ++T) {
    const int G = direct_group_levels(T);
    for (int levels = 1; levels <= kDirectMaxTile / G * G; ++levels) {
      const int tile = direct_tile_levels(T, levels);
      const int last = tile - (tile - 1) / G * G;
      if (tile < levels || tile - levels > (G + 2) / 3 || tile > kDirectMaxTile / G * G) return false;
      if (last != G && last != direct_short_group(T, 1) && last != direct_short_group(T, 2)) return false;
      if (direct_tile_levels(T, tile) != tile) return false;
    }
  }
  return true;
}
static_assert(direct_tiles_consistent(), "tiles of the direct kernel");
static_assert(direct_tile_levels(5, 64) == 64 && direct_tile_levels(2, 205) == 205 && direct_tile_levels(4, 241) == 241,
              "sweeps of 64, 1024 and 4096 levels split into tiles without padding");
constexpr int kDirectBatch = 32;       // candidates decoded per step of the direct kernel: one per lane
// Level-lane kernel: one warp per block, 32 * LPL demand levels per launch (LPL = 1, 2 or 4
// levels per lane); a class tuple's member records are staged in shared memory.
constexpr int kUniformMaxTile = 128;
constexpr int kUniformUnitsPerWarp = 8;      // work units aimed at per warp
constexpr int kUniformMaxSlices = 16;        // at most this many slices per class tuple
constexpr int kUniformHeaderBytes = 128;
constexpr int kUniformMaxStageBytes = 6144;  // header + records; keeps 32 warps resident per SM
constexpr int kUniRecBytes1 = 16;      // member record when every option has one part
constexpr int kUniRecBytes2 = 32;      // member record when split options exist
constexpr int kGenericThreads = 256;
constexpr int kGenericLevelGroup = 4;  // levels scored per decode in the generic kernel

// One option of a task, fully resolved (device table, 64 bytes).
// A single option has parts == 1 and mult[1] == 0, den[1] == 1.
struct OptRec {
  double acc;        // task accuracy a_i of this option
  int64_t lat;       // task latency L_i: the larger of the parts
  int64_t mult[2];   // share * lat_us per part (share = 1 for a single option)
  int64_t den[2];    // batch * 1e9 (single) or 16 * batch * 1e9 (split part)
  int32_t variant[2];
  uint8_t batch_idx[2];
  uint8_t k;         // 16 for a single option, else sixteenths sent to part 0
  uint8_t parts;
  uint32_t vf16;     // multiplicative factor in thousandths x 16 (share-weighted sum for a split option)
};
static_assert(sizeof(OptRec) == 64, "OptRec layout");

// Result key of the argmax, ordered lexicographically as unsigned integers:
// accuracy bits (positive doubles order like their bit patterns), then
// (S - W) << 40 | (N - 1 - c).  {0, 0} means "no feasible candidate".
struct Key {
  uint64_t acc_bits;
  uint64_t tail;
};

__host__ __device__ inline bool key_less(const Key& a, const Key& b) {
  return a.acc_bits < b.acc_bits || (a.acc_bits == b.acc_bits && a.tail < b.tail);
}

// Problem description passed to kernels by value.
struct DevProblem {
  int32_t T;
  int32_t n_leaves;
  int32_t split;
  int32_t S;
  int64_t N;
  int32_t parent[kMaxTasks];
  int32_t fanout_milli[kMaxTasks];
  int32_t leaf_task[kMaxTasks];      // [n_leaves] leaves in ascending task index
  uint32_t path_mask[kMaxTasks];     // [n_leaves] bit i set if task i is on root..leaf
  int64_t lat_limit[kMaxTasks];      // [n_leaves] floor((slo - hops*comm) / 2), -1 if negative
  int64_t O[kMaxTasks];              // options per task
  int64_t stride[kMaxTasks];         // prod_{j<i} O_j
  int64_t opt_off[kMaxTasks];        // offset of the task's first record in `opts`
  const OptRec* opts;                // device
  int64_t max_demand_mqps;
  int32_t variant_fanout;            // 1: stage demands depend on the parents' chosen variants
  int32_t pad1;
  // bounds of the tables and of the partial-key scratch, and the status words that the checked
  // (LOKI_DEBUG) build records violations in; the release build carries but does not read them
  int64_t n_opts;                    // records in `opts`
  int64_t partial_keys;              // keys the partial-key scratch of the launch holds
  uint32_t* debug_flags;             // device, kDebugWords words, or null
};

// ---- direct path -----------------------------------------------------------

// Per option, the reciprocal constants of its parts (device table).
// workers(part) = 1 + floor(dem * r) for 1 <= dem <= cap, where r is the largest
// double strictly below share*lat / (16*batch*1e9); the floor comes out of one
// fused multiply-add rounded toward minus infinity.  An unused part has r == 0
// and is not counted in n_real.
struct DirRec {
  double r[2];
  int32_t lat;        // task latency
  int32_t n_real;     // number of real parts (1 or 2)
  int32_t opt;        // option index within the task
  int32_t pad;
};
static_assert(sizeof(DirRec) == 32, "DirRec layout");

struct DirProblem {
  int32_t T;
  int32_t n_leaves;
  int32_t S;
  int32_t jbits;                     // bits of the in-class-tuple candidate rank in the packed key
  int32_t n_parts_max;               // 1, or 2 when split options exist
  int32_t pad0;
  int32_t n_class[kMaxTasks];        // accuracy classes per task
  int32_t class_off[kMaxTasks];      // offset of the task's first class in class tables
  int32_t parent[kMaxTasks];
  int32_t leaf_task[kMaxTasks];
  uint32_t path_mask[kMaxTasks];
  int32_t lat_limit[kMaxTasks];      // clamped to int32
  int64_t stride[kMaxTasks];
  int64_t N;
  int64_t n_ct;                      // class tuples
  int64_t total_iters;               // sum over class tuples of ceil(J / 32): batches of one candidate per lane
  const int32_t* class_first;        // [sum n_class] first member (index into members of the task)
  const int32_t* class_count;        // [sum n_class] members in the class
  const double* class_acc;           // [sum n_class] task accuracy of the class
  const DirRec* members;             // per task, members of all classes, class-major, ascending option
  int64_t member_off[kMaxTasks];     // offset of the task's first member record
  const uint64_t* iter_prefix;       // [n_ct + 1] exclusive prefix of iterations
  const uint64_t* ct_acc;            // [n_ct] end-to-end accuracy bits of every class tuple
  const uint64_t* ct_sorted_acc;     // [n_ct] the same in ascending order ...
  const uint32_t* ct_sorted_idx;     // ... and the class tuple each entry belongs to
  const uint32_t* ct_rank;           // [n_ct] position of every class tuple in that order
  const uint32_t* unit_start;        // [n_units + 1] first batch of every work unit of the direct kernel
  // level-lane kernel
  const void* uni_members;           // member records in the order of `members`: r[parts], lat, n_real << jbits
  const int32_t* class_min_lat;      // [sum n_class] smallest task latency among the members
  const int32_t* lat_order;          // in the order of `members`: per class, in-class indices by ascending latency
  // hoisted kernel, joined tasks 0 and 1: per pair of their classes (class of task 1 major) the member
  // pairs q = k0 + count0 * k1 (k: position in ascending latency) in ascending order of (joint
  // latency, q), join_stride entries per pair of classes; nullptr: ranked by the kernel
  const int32_t* join_order;
  int32_t join_stride;
  int32_t uni_slices;                // work units per class tuple (slices of its top digit)
  int32_t uni_stage_bytes;           // dynamic shared memory: header + the largest class tuple's records
  // per-variant multiplicative factors (level-lane kernel, root-first walk)
  const double* uni_dem_r;           // [member][T]: largest double below edge factor x option factor into child task i
  const int64_t* dem_cap;            // [T] demand from which every option of the task needs more than S workers
  int32_t fanout_milli[kMaxTasks];
  int32_t uni_max_members;           // sum over tasks of the largest class
  int32_t pad2;
  int64_t max_demand_mqps;           // demands above it (or below 0) are scored as zero and reported as bad
  // bounds for the checked (LOKI_DEBUG) build, as in DevProblem
  int32_t n_classes;                 // entries of the class tables
  int32_t n_members;                 // member records (all tasks)
  int64_t partial_keys;
  uint32_t* debug_flags;
};


// ---- the checked build ------------------------------------------------------
// Compiled with -DLOKI_DEBUG, every index into the class, member, option and class-tuple tables,
// into the shared-memory stages and tables of the scoring kernels and into the partial-key
// scratch goes through LOKI_IDX: an index out of range sets bit `site` of status word 0, counts
// in word 1, and is replaced by 0, so the access itself stays in bounds and the kernel runs on
// (no trap, no fault).  In the release build LOKI_IDX is the index itself.
constexpr int kDebugWords = 4;
enum DebugSite {
  kSiteClass = 0, kSiteMember = 1, kSiteOption = 2, kSitePartial = 3, kSiteDirectStage = 4,
  kSiteDirectWmin = 5, kSiteHoistLat = 6, kSiteHoistTab = 7, kSiteHoistJoin = 8, kSiteVariantStage = 9,
  kSiteClassTuple = 10, kSiteDemandTile = 11, kSiteSharedLayout = 12
};

#ifdef __CUDACC__
#ifdef LOKI_DEBUG
__device__ __forceinline__ long long loki_checked_index(long long idx, long long limit, int site, uint32_t* flags) {
  if (idx >= 0 && idx < limit) return idx;
  if (flags != nullptr) { atomicOr(flags, 1u << site); atomicAdd(flags + 1, 1u); }
  return 0;
}
#define LOKI_IDX(idx, limit, site, flags) \
  loki::loki_checked_index((long long)(idx), (long long)(limit), (int)(site), (flags))
// Bytes of dynamic shared memory the launch was given.
__device__ __forceinline__ uint32_t loki_dynamic_smem_bytes() {
  uint32_t n;
  asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(n));
  return n;
}
#else
#define LOKI_IDX(idx, limit, site, flags) (idx)
#endif

// ---- device helpers shared by the scoring kernels ---------------------------

constexpr double kMagic = 6755399441055744.0;   // 1.5 * 2^52: ulp 1, low mantissa word 0
constexpr uint32_t kEmpty = 0xFFFFFFFFu;        // "no candidate" in a packed 32-bit key

// Member record of the level-lane kernels (device table `uni_members`).
template <int NP> struct UniRec;
template <> struct __align__(16) UniRec<1> { double r[1]; int32_t lat; uint32_t nsh; };
template <> struct __align__(16) UniRec<2> { double r[2]; int32_t lat; uint32_t nsh; int32_t pad[2]; };
static_assert(sizeof(UniRec<1>) == kUniRecBytes1 && sizeof(UniRec<2>) == kUniRecBytes2, "UniRec layout");

// a4 for the level-lane kernels: the stage demands of one level (Eq. 1, ceiling on every edge) from
// its root demand, clamped per task to the cap above which every option needs more than S workers,
// as doubles (exact: the caps are below 2^53).  A level past the end of the sweep or with a demand
// out of range is scored with zero demand; the finishing kernel reports it.
template <int T>
__device__ __forceinline__ void level_stage_demands(const DirProblem& p, const int64_t* __restrict__ demand,
                                                    int n_levels, int l, double (&out)[T]) {
  int64_t dem[T];
  int64_t D = l < n_levels ? demand[l] : 0;
  if (D < 0 || D > p.max_demand_mqps) D = 0;
  dem[0] = D;
#pragma unroll
  for (int i = 1; i < T; ++i) {
    int64_t up = 0;
#pragma unroll
    for (int j = 0; j < T - 1; ++j)
      if (j == p.parent[i]) up = dem[j];
    const uint64_t num = (uint64_t)(up * (int64_t)p.fanout_milli[i]);
    const uint64_t q = num / 1000u;
    dem[i] = (int64_t)(q + (num - q * 1000u != 0 ? 1 : 0));
  }
#pragma unroll
  for (int i = 0; i < T; ++i) {
    const int64_t cap = p.dem_cap[i];
    out[i] = (double)(dem[i] > cap ? cap : dem[i]);
  }
}

// Candidate index of rank j within class tuple ct: both are mixed-radix numbers, task 0 least
// significant (ct over the class counts, j over the member counts of ct's classes).
template <int T>
__device__ __forceinline__ int64_t cand_index(const DirProblem& p, uint64_t ct, uint32_t j) {
  int64_t c = 0;
#pragma unroll
  for (int i = 0; i < T; ++i) {
    const uint32_t nc = (uint32_t)p.n_class[i];
    const uint32_t cls = (uint32_t)(ct % nc);
    ct /= nc;
    const int idx = (int)LOKI_IDX(p.class_off[i] + cls, p.n_classes, kSiteClass, p.debug_flags);
    const int32_t first = p.class_first[idx];
    const uint32_t cnt = (uint32_t)p.class_count[idx];
    const uint32_t d = j % cnt;
    j /= cnt;
    c += (int64_t)p.members[LOKI_IDX(p.member_off[i] + first + d, p.n_members, kSiteMember, p.debug_flags)].opt * p.stride[i];
  }
  return c;
}
#endif  // __CUDACC__

// The demand levels a level-lane launch covers: root demands of the sweep (device), the sweep's
// length, and the level the launch's first tile starts at.
struct LevelSpan {
  const int64_t* demand;
  int32_t n_levels;
  int32_t level_begin;
};

// Host-side launch wrappers (defined in the .cu files).
cudaError_t launch_option_accuracy(OptRec* d_opts, int64_t n, const double* d_variant_acc,
                                   cudaStream_t st);
// n_zero_words: 32-bit words at d_zero_words cleared by the same launch (work counters of the solve).
// The clamped demands go to d_demf tile by tile: [tile][level pair][task][2], or, with tile < 0,
// the direct kernel's layout (direct_dem_offset) in tiles of -tile levels (each stored as whole groups).
cudaError_t launch_prepare_levels(const DevProblem& p, const int64_t* d_demand, int n_levels,
                                  int64_t* d_dem64, int32_t* d_status, const int64_t* d_dem_cap,
                                  double* d_demf, int tile, cudaStream_t st,
                                  uint32_t* d_zero_words = nullptr, int n_zero_words = 0);
// Partial keys of every scoring kernel: [level][block], so that a level's keys lie in a row.
cudaError_t launch_generic_score(const DevProblem& p, const int64_t* d_dem64, const int32_t* d_status,
                                 int n_levels, int n_blocks_x, Key* d_partial, cudaStream_t st);
// K2 + K3 in one launch, one block per level: the maximum over the partial keys ([level][n_parts];
// tile_levels > 0: several tiles of [tile_levels][n_parts] back to back), then the winner's plan.
// d_out == nullptr: only the reduced key is written (to d_final).  n_slos > 1 (grid.y): the sweep under
// several latency SLOs; SLO s reads its keys at d_partial + s * slo_keys, takes d_zero_key[s], and writes
// d_final and d_out at + s * slo_levels.
cudaError_t launch_finish(const DevProblem& p, const Key* d_partial, int n_parts, int tile_levels,
                          int level_begin, int n_levels_here, const int64_t* d_demand, const Key* d_zero_key,
                          Key* d_final, loki_config_t* d_out, cudaStream_t st, int n_slos = 1,
                          long long slo_keys = 0, int slo_levels = 0);
cudaError_t direct_upload_tile(const double* d_demf_tile, int n_doubles, cudaStream_t st);
int direct_max_blocks_per_sm(int T, int n_parts, int n_groups);
int direct_stage_rows(int T, int n_parts);
// One tile of the direct kernel, tile_levels = direct_tile_levels(T, .) levels in groups of
// direct_group_levels(T), the last one possibly shorter (partial keys: [level][n_blocks]): the n_units
// work units of p.unit_start are dealt through *d_unit_counter (zero before the launch);
// *d_rows_scored accumulates the rows of 32 candidates scored.
cudaError_t launch_direct_score(const DirProblem& p, int tile_levels, int n_blocks, Key* d_partial,
                                uint32_t* d_unit_counter, unsigned long long* d_rows_scored,
                                uint32_t n_units, cudaStream_t st);
cudaError_t launch_class_tuple_accuracy(const DirProblem& p, uint64_t* d_ct_acc, cudaStream_t st);
// K2 + K3 for the direct kernel's keys (accuracy and workers only; d_partial is [level][n_parts]):
// reduction, the lowest candidate index that attains the winning pair, then the plan.
cudaError_t launch_direct_finish(const DirProblem& p, const DevProblem& dp, const Key* d_partial, int n_parts,
                                 int level_begin, int n_levels_here,
                                 const double* d_dem_tile, const int64_t* d_demand, const Key* d_zero_key,
                                 Key* d_final, loki_config_t* d_out, cudaStream_t st);
bool direct_supported(int T, int split);
// n_tiles consecutive level tiles in one launch (grid.y): tile t writes d_partial + t * n_blocks * tile_levels,
// each tile [tile_levels][n_blocks].
// The level-lane kernel (root-first walk; tiles of 32 or 64 levels), with or without per-variant factors.
cudaError_t launch_variant_score(const DirProblem& p, LevelSpan span, int tile_levels, int n_blocks,
                                 Key* d_partial, cudaStream_t st, int n_tiles = 1);
int variant_max_blocks_per_sm(const DirProblem& p, int tile_levels);

// Shared memory of the hoisted kernel for one level tile: 32 header words, the member
// latencies of the largest class tuple, and its table of 32 lanes x (tile / 32) entries per member.
struct HoistLayout {
  int32_t smem_bytes;
  int32_t max_members;           // sum over tasks of the largest class
  int32_t join_rows;             // > 0: tasks 0 and 1 are walked as one loop over this many member pairs at most
  int32_t tab_members;           // members with a table row: all, or (joined) those of tasks 2 and up
  int32_t join_members;          // joined: largest class of task 0 + largest class of task 1 (their records are staged instead)
  int32_t warps;                 // warps per block: they share the staged table and split the class tuple's candidates
  // 0: every inner row is read; 1: the inner loop over a fitting prefix is one read of the rows'
  // prefix minima, which replace the rows in place (not with joined tasks on a tree)
  int32_t pmin_mode;
};
constexpr int kHoistMaxWarps = 8;
constexpr int kHoistMaxJoinRows = 64;
constexpr int kHoistSmemPerWarp = 9 * 1024;     // table bytes per warp of the block that keep about 24 warps per SM
constexpr int kHoistMaxSmemBytes = kHoistMaxWarps * kHoistSmemPerWarp;   // 72 KB: the largest table taken
constexpr int kHoistLastResortSmemBytes = 160 * 1024;   // accepted only when no tile fits the bound above
// zero_demand: score the demand-free case (no option needs a worker) instead of the tile's demands.
// n_slos > 1 (grid.z): the same sweep under several latency SLOs in one launch; d_slo_limits is
// [n_slos][kMaxTasks], the per-leaf latency limits of each (nullptr: the problem's own limits);
// partial keys: [slo][tile][level][block].
// The level-lane kernels derive the stage demands themselves (level_stage_demands) from the sweep's
// root demands: tile t of the launch covers levels level_begin + t * tile_levels ...
cudaError_t launch_hoisted_score(const DirProblem& p, const HoistLayout& lay, LevelSpan span,
                                 int tile_levels, int n_blocks, Key* d_partial, cudaStream_t st,
                                 bool zero_demand = false, int n_tiles = 1, int n_slos = 1,
                                 const int32_t* d_slo_limits = nullptr);
// Worker tables shared by all class tuples (LOKI_PATH_PREFIX): one row per member of every class
// of the outer tasks, and per inner group -- a class of task 0, or (joined: a chain of three or more
// tasks whose two innermost classes are small) a pair of classes of tasks 0 and 1 -- its rows in
// ascending latency, replaced by their prefix minima.  Rows [0, n_outer) are the outer ones, the
// groups follow.  A row is [32 lanes][levels per lane] entries; a level tile's rows are consecutive.
struct PrefixTables {
  const int4* row_desc;        // [n_rows] member a, member b or -1 (indices into uni_members), constant of the entry, task a | task b << 8
  const int32_t* row_lat;      // [n_rows] latency of the member, or of the pair
  const uint32_t* row_digit;   // [n_rows] outer rows: the member's own digit within its class
  const int32_t* class_rows;   // [sum n_class] first row of the class (its members in ascending latency), or -1
  const int32_t* pair_rows;    // joined: [class of task 1][class of task 0] first row of the pair's group
  const int2* groups;          // [n_groups] first row and number of rows
  uint32_t* tab;               // entries, written by the build kernel of every solve
  int32_t n_rows, n_outer, n_groups, joined;
};
// Arguments of the shared-table launches, so that the dispatch by template arguments has one shape.
struct PrefixCall {
  const DirProblem* p;
  const PrefixTables* t;
  LevelSpan span;
  int build;            // 1: build the tables; 0: walk them (n_blocks == 0: resident blocks per SM of the walk)
  int tile0, n_tiles, n_blocks, n_slos;
  Key* d_partial;
  const int32_t* slo_limits;
  cudaStream_t st;
};

// Builds the tables for n_tiles tiles of tile_levels levels from span.level_begin on.
cudaError_t launch_prefix_build(const DirProblem& p, const PrefixTables& t, LevelSpan span, int tile_levels,
                                int n_tiles, cudaStream_t st);
// Walks every class tuple against the tables of n_tiles tiles starting at table tile `tile0` (levels
// span.level_begin ...), one warp per class tuple at a time, n_blocks blocks of kPrefixWarps warps per
// tile and SLO; partial keys [slo][tile][level][n_blocks x kPrefixWarps].  d_slo_limits as for the hoisted kernel.
constexpr int kPrefixWarps = 4;
cudaError_t launch_prefix_walk(const DirProblem& p, const PrefixTables& t, LevelSpan span, int tile_levels,
                               int tile0, int n_tiles, int n_blocks, Key* d_partial, cudaStream_t st,
                               int n_slos = 1, const int32_t* d_slo_limits = nullptr);
int prefix_walk_max_blocks_per_sm(const DirProblem& p, const PrefixTables& t, int tile_levels);
constexpr long long kMaxPartialKeys = 4LL << 20;   // keys of scratch a multi-tile launch may use (64 MB)
int hoisted_max_blocks_per_sm(const DirProblem& p, const HoistLayout& lay, int tile_levels);

// Read-only view of a handle for entry points that live in other source files.
struct HandleView {
  DevProblem dev;     // problem description with its device table pointers
  int device;         // CUDA device the handle was created on
  int n_sms;
  int n_tasks;
  int n_batches;      // |B|: single option o of a task is variant o / n_batches, batch index o % n_batches
};
bool handle_view(const loki_alloc_t* h, HandleView* out);

// Resolves, once per device, the address of the fixed working array of loki_alloc_solve_static
// (the device must be current).  Called by loki_alloc_create.
int static_scratch_prepare(int device);

}  // namespace loki

#endif  // LOKI_INTERNAL_H_
