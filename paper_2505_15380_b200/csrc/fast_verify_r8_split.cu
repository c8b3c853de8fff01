// Persistent verify kernel, variants for at most 8 rows with split (bf16 hi + lo) activations.
#include "fast_kernel.cuh"

namespace ssd {

const void* fast_kernel_r8_split(bool trace) { return fast_kernel_variant<false, true>(trace); }

size_t fast_misc_bytes() { return sizeof(FastMisc); }

}  // namespace ssd
