// Persistent verify kernel, key-split variants (long prefixes; split activations), <= 8 and <= 16 rows.
#include "fast_kernel.cuh"

namespace ssd {

const void* fast_kernel_keysplit(bool t16) {
  return t16 ? fast_kernel_keysplit_variant<true>() : fast_kernel_keysplit_variant<false>();
}

}  // namespace ssd
