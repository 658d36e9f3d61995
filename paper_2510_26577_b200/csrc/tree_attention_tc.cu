// Tensor-core (tcgen05 / TMEM / TMA) path of cast_tree_attention for bf16.
#include "cast_internal.h"

namespace cast {

bool tree_attention_tc_launch(cast_ctx*, const void*, const void*, const void*, int, int, int, int, int,
                              const int32_t*, int, int, const int32_t*, const uint32_t*, const int32_t*, float, void*,
                              cudaStream_t, cast_status*) {
  return false;  // not taken: the caller uses the CUDA-core path
}

}  // namespace cast
