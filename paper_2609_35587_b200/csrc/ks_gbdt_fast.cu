// Quantised fast path for ensembles of complete trees (placeholder: not built yet).
#include "ks_internal.h"

namespace ks {

cudaError_t build_fast_gbdt(GbdtModel& m, int, const int64_t*, const ks_node_host*) {
  m.fast = false;
  return cudaSuccess;
}

}  // namespace ks
