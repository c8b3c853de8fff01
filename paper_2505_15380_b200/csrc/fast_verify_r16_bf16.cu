// Persistent verify kernel, variants for 9..16 rows with plain bf16 activations.
#include "fast_kernel.cuh"

namespace ssd {

const void* fast_kernel_r16_bf16(bool trace) { return fast_kernel_variant<true, false>(trace); }

}  // namespace ssd
