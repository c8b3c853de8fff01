// Persistent verify kernel, variants for 9..16 rows with split (bf16 hi + lo) activations.
#include "fast_kernel.cuh"

namespace ssd {

const void* fast_kernel_r16_split(bool trace) { return fast_kernel_variant<true, true>(trace); }

}  // namespace ssd
