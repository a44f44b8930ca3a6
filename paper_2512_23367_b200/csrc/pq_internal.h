// Internal declarations shared by the translation units of libpq (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/pq.h"

namespace pq {

// Device status word (one per device that loaded the library): PQ_OK or PQ_ERR_TIMEOUT.
int* device_status_ptr();  // device address of the status word of the current device, or nullptr

// Number of SMs of the current device (cached per device).
int sm_count();

// Split-K scratch of one GEMM call (the caller's `workspace` argument, or the built-in array of
// pq_gemm_w8a8_noalloc): arrival counters first, then room for the partial accumulators.  All
// null/zero when the call has none.
struct Scratch {
  unsigned int* counters = nullptr;   // kScratchCounters words, zero between calls
  int32_t* partials = nullptr;
  size_t partial_bytes = 0;
};
constexpr int kScratchCounters = 16384;                       // 64 KB
constexpr size_t kScratchHeaderBytes = kScratchCounters * 4;
// The view of a caller's workspace: empty when the pointer is null or the room is below the header.
inline Scratch scratch_from(void* workspace, size_t bytes) {
  Scratch sc;
  if (workspace != nullptr && bytes > kScratchHeaderBytes) {
    sc.counters = static_cast<unsigned int*>(workspace);
    sc.partials = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + kScratchHeaderBytes);
    sc.partial_bytes = bytes - kScratchHeaderBytes;
  }
  return sc;
}

// Poll bound handed to every kernel (pq_set_wait_limit; default kWaitPollLimit of pq_ptx.cuh).
uint32_t wait_limit();

// Clears the counter header of the built-in scratch array of pq_gemm_w8a8_noalloc on the current
// device, if that array has been used on it (after a wait ran out its counters may be non-zero).
int reset_static_scratch();

// Raises a kernel's dynamic shared-memory limit once per device (the attribute is per device and
// per kernel; `once` is a function-local static of the launcher of that kernel).  Safe to race:
// setting the attribute twice is harmless.
struct PerDeviceOnce {
  std::atomic<uint64_t> done{0};   // bit d: set on device d
};
template <typename Kernel>
int set_dynamic_smem_once(PerDeviceOnce& once, Kernel kern, int bytes) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PQ_ERR_CUDA;
  const uint64_t bit = uint64_t(1) << dev;
  if (once.done.load(std::memory_order_acquire) & bit) return PQ_OK;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  once.done.fetch_or(bit, std::memory_order_release);
  return PQ_OK;
}

// Whether kernels are launched with the programmatic-stream-serialization attribute (default
// yes; PQ_PDL=0 in the environment turns it off, for ablations).
bool pdl_enabled();

// cuTensorMapEncodeTiled obtained through the runtime (no link-time dependency on libcuda).
// Encodes a 2-D row-major tensor [rows, cols] of `elem_bytes`-sized elements with a
// box of [box_rows, box_cols]; swizzle_bytes (0, 32, 64 or 128) selects the shared-memory swizzle.
int make_tmap_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                 uint32_t box_cols, uint32_t elem_bytes, int swizzle_bytes);

// ---- launchers (each returns a pq_status; all are asynchronous on `stream`) ----
// col (nullable, [K] FP32): per-column factor applied before the maximum is taken (Eq. 3).
int launch_quantize_act(const void* x, int64_t M, int64_t K, int8_t* q, float* s, bool divide_by_scale,
                        const float* col, cudaStream_t stream);
int launch_pack_fence(cudaStream_t stream);
int launch_pack_w4(const void* w, int64_t N, int64_t K, void* wp, void* s_grp, const float* col,
                   cudaStream_t stream);
// Eq. 4: the same quantizers on rows rotated by the block Hadamard matrix (K <= 16384).
int hadamard_block_order(int64_t K);
int launch_quantize_act_hadamard(const void* x, int64_t M, int64_t K, int8_t* q, float* s, bool divide_by_scale,
                                 cudaStream_t stream);
int launch_pack_w4_hadamard(const void* w, int64_t N, int64_t K, void* wp, void* s_grp, cudaStream_t stream);
int launch_quantize_act_static(const void* x, const float* s_ptr, int64_t M, int64_t K, int8_t* q, float* s_tok,
                               cudaStream_t stream);
// SwiGLU of the gate/up outputs fused with the down projection's per-token quantizer (I <= 16384).
int launch_swiglu_quantize(const void* gate, const void* up, int64_t M, int64_t I, int8_t* q, float* s_tok,
                           cudaStream_t stream);
int launch_quantize_act_static_channel(const void* x, const float* inv_s, int64_t M, int64_t K, int8_t* q, float* s_tok,
                                       cudaStream_t stream);
int launch_col_absmax(const void* a, int64_t R, int64_t K, float* out, cudaStream_t stream);
int launch_smooth_scales(const float* xa, const float* wa, int64_t K, int alpha_quarters, float* s, float* s_inv,
                         cudaStream_t stream);
int launch_unpack_w4(const void* wp, int64_t N, int64_t K, int8_t* codes, cudaStream_t stream);

// Prefill-shaped W8A8 GEMM (tcgen05 kind::i8) on CTA pairs (cta_group::2, 256-row tiles), for M > 128.
// Exactly one of y / acc is non-null.  `sc`: split-K scratch of this call (may be empty).
int launch_gemm_w8a8_pair(const Scratch& sc, const int8_t* q, const float* s_tok, const void* wq,
                          const float* s_ch, int64_t M, int64_t N, int64_t K, void* y, int32_t* acc,
                          cudaStream_t stream);
// Linears that share the token codes and run as one launch of the pair GEMM: at most this many.
constexpr int kMaxGroup = 4;
// Host-only: the pair GEMM's choice of tile width and number of K parts (see the definition).
int64_t plan_w8a8_pair(int64_t M, int64_t N, int64_t K, int sms, size_t scratch_bytes, int force_bn,
                       int force_splits, int* bn_out, int* splits_out);
// Bytes of split-K partial sums the plan (bn, splits) needs for these members; 0 when K is not split.
size_t w8a8_pair_partial_bytes(int64_t M, const int64_t* N, int count, int bn, int splits);
// `count` (1..kMaxGroup) linears over the same codes in one launch; arrays are host arrays of
// device pointers / column counts.  acc (accumulator export) only with count == 1.
int64_t plan_w8a8_pair_group(int64_t M, const int64_t* N, int count, int64_t K, int sms, size_t scratch_bytes,
                             int force_bn, int force_splits, int* bn_out, int* splits_out);
int launch_gemm_w8a8_pair_group(const Scratch& sc, const int8_t* q, const float* s_tok, int count,
                                const void* const* wq, const float* const* s_ch, const int64_t* N, void* const* y,
                                int64_t M, int64_t K, int32_t* acc, cudaStream_t stream);
// Prefill-shaped W4A8 GEMM.  Exactly one of y / acc_g is non-null.
int launch_gemm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M,
                     int64_t N, int64_t K, void* y, int32_t* acc_g, cudaStream_t stream);
// `count` (1..kMaxGroup) W4A8 linears over the same codes in one launch (host arrays, as above).
int launch_gemm_w4a8_group(const int8_t* q, const float* s_tok, int count, const void* const* wp,
                           const void* const* s_grp, const int64_t* N, void* const* y, int64_t M, int64_t K,
                           int32_t* acc_g, cudaStream_t stream);
// Small-M (decode-shaped) weight-streaming variants; same results as the calls above.
int launch_smallm_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M,
                       int64_t N, int64_t K, void* y, int32_t* acc, cudaStream_t stream);
int launch_smallm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M,
                       int64_t N, int64_t K, void* y, int32_t* acc_g, cudaStream_t stream);

// One to four tokens on the CUDA cores (whole weight rows per CTA, ring filled ahead of the wait on the
// preceding kernel); same results as the calls above.  gemv_rows_serves: whether it is the schedule of choice.
bool gemv_rows_serves(int w_bits, int64_t M, int64_t N, int64_t K, int sms);
// The same from FP16 activations [M, K]: the kernel quantizes its tokens itself (Eq. 1-2).
int launch_gemv_rows_w8a8_x(const void* x, const void* wq, const float* s_ch, int64_t M, int64_t N, int64_t K, void* y,
                            cudaStream_t stream);
int launch_gemv_rows_w4a8_x(const void* x, const void* wp, const void* s_grp, int64_t M, int64_t N, int64_t K, void* y,
                            cudaStream_t stream);
int launch_gemv_rows_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M, int64_t N,
                          int64_t K, void* y, int32_t* acc, cudaStream_t stream);
int launch_gemv_rows_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M, int64_t N,
                          int64_t K, void* y, int32_t* acc_g, cudaStream_t stream);

// `count` (1..kMaxGroup) small-M linears over the same tokens in one launch (host arrays, as above).
int launch_smallm_w8a8_group(const int8_t* q, const float* s_tok, int count, const void* const* wq,
                             const float* const* s_ch, const int64_t* N, void* const* y, int64_t M, int64_t K,
                             int32_t* acc, cudaStream_t stream);
int launch_smallm_w4a8_group(const int8_t* q, const float* s_tok, int count, const void* const* wp,
                             const void* const* s_grp, const int64_t* N, void* const* y, int64_t M, int64_t K,
                             int32_t* acc_g, cudaStream_t stream);

// Remembers the name of a failed CUDA call for pq_last_cuda_error (per host thread).
void note_cuda_error(cudaError_t e);
inline int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return PQ_OK;
  note_cuda_error(e);
  return PQ_ERR_CUDA;
}

}  // namespace pq
