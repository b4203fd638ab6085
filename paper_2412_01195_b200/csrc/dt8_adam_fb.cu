// Fused 8-bit Adam step: kernels for gradients binary32, parameters bfloat16.
#include "dt8_adam_impl.cuh"

namespace dt8 {
DT8_INSTANTIATE_ADAM(false, true)
}  // namespace dt8
