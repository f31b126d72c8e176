// Tensor-core prefill kernels (bf16, d=128, S=64).  Filled in below.
#include "internal.h"

namespace hils {
bool prefill_fast_supports(const Shape&, int) { return false; }
size_t prefill_fast_scratch_bytes(const Shape&) { return 0; }
int launch_prefill_fast(const Shape&, const Tensors&, cudaStream_t) { return HILS_ERR_UNSUPPORTED; }
}  // namespace hils
