// The level launchers for __nv_bfloat16 operands (see adasum_levels.cuh).
#include "adasum_levels.cuh"

namespace adasum {
ADASUM_INSTANTIATE_LEVELS(__nv_bfloat16)
}  // namespace adasum
