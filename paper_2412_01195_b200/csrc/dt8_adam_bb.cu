// Fused 8-bit Adam step: kernels for gradients bfloat16, parameters bfloat16.
#include "dt8_adam_impl.cuh"

namespace dt8 {
DT8_INSTANTIATE_ADAM(true, true)
}  // namespace dt8
