// Temporary routing while the dedicated kernels are being written.
#include "pq_internal.h"
namespace pq {
int launch_smallm_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M,
                       int64_t N, int64_t K, void* y, int32_t* acc, cudaStream_t stream) {
  return launch_gemm_w8a8(q, s_tok, wq, s_ch, M, N, K, y, acc, stream);
}
int launch_smallm_w4a8(const int8_t*, const float*, const void*, const void*, int64_t, int64_t, int64_t, void*,
                       int32_t*, cudaStream_t) { return PQ_ERR_CUDA; }
}
