// Bulk-copy pipelined decode kernel for bf16, head_dim 128.  Not built yet: the portable kernel handles every shape.
#include "fdkv_internal.h"

namespace fdkv {
cudaError_t launch_decode_fast(const DecodeArgs&, cudaStream_t, bool* handled) {
    *handled = false;
    return cudaSuccess;
}
}  // namespace fdkv
