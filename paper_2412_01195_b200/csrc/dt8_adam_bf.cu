// Fused 8-bit Adam step: kernels for gradients bfloat16, parameters binary32.
#include "dt8_adam_impl.cuh"

namespace dt8 {
DT8_INSTANTIATE_ADAM(true, false)
}  // namespace dt8
