// The level launchers for __half operands (see adasum_levels.cuh).
#include "adasum_levels.cuh"

namespace adasum {
ADASUM_INSTANTIATE_LEVELS(__half)
}  // namespace adasum
