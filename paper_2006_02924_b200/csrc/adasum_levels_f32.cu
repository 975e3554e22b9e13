// The level launchers for float operands (see adasum_levels.cuh).
#include "adasum_levels.cuh"

namespace adasum {
ADASUM_INSTANTIATE_LEVELS(float)
}  // namespace adasum
