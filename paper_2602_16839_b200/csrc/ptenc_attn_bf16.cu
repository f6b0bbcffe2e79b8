// placeholder: fast path not built yet
#include "ptenc_internal.h"
bool ptenc_attn_bf16_prepare(ptenc_cache* c, cudaError_t* err) { *err = cudaSuccess; return false; }
cudaError_t ptenc_launch_attn_bf16(ptenc_cache*, int, int, const void*, const uint8_t*, void*, float*, cudaStream_t) {
  return cudaErrorNotSupported;
}
