// Hoisted scoring kernel, instantiations with 4 demand levels per lane (128-level tiles).
#include "loki_kernels_hoisted_impl.h"

namespace loki {

int hoisted_dispatch_l4(const DirProblem* p, const HoistLayout* lay, LevelSpan dem_tile, int n_blocks,
                         Key* d_partial, cudaStream_t st, int zero, int n_tiles, int n_slos,
                         const int32_t* slo_limits) {
  return hoisted_for_lpl<4>(p, lay, dem_tile, n_blocks, d_partial, st, zero, n_tiles, n_slos, slo_limits);
}

int prefix_dispatch_l4(const void* call) { return prefix_for_lpl<4>(*static_cast<const PrefixCall*>(call)); }

}  // namespace loki
