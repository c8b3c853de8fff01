// Persistent verify kernel, variants for at most 8 rows with plain bf16 activations.
#include "fast_kernel.cuh"

namespace ssd {

const void* fast_kernel_r8_bf16(bool trace) { return fast_kernel_variant<false, false>(trace); }

}  // namespace ssd
