// Bandwidth-tuned decode kernels (bf16, d=128, S=64).  Filled in below.
#include "internal.h"

namespace hils {
bool decode_fast_supports(const Shape&, int) { return false; }
size_t decode_fast_scratch_bytes(const Shape&) { return 0; }
int launch_decode_fast(const Shape&, const Tensors&, cudaStream_t) { return HILS_ERR_UNSUPPORTED; }
}  // namespace hils
