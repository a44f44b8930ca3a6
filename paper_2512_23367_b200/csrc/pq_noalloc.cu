// pq_gemm_w8a8_noalloc: the W8A8 linear for callers that cannot allocate device memory.
//
// The W8A8 GEMM gets its split-K fast path (few output tiles, long K) only when it has scratch
// memory for the parts' INT32 partial sums.  pq_gemm_w8a8 takes that scratch from the workspace
// argument of the call, a buffer which the caller had to allocate.  Some callers have
// no allocator to ask: code that runs inside a stream capture or a latency-critical serving loop
// where cudaMalloc (a synchronizing call) is forbidden, plug-ins whose host hands them only input
// and output buffers, and programs that pre-size every byte of device memory at start-up.  For
// them the scratch lives here, in a fixed array that is part of the library image: every GPU that
// loads the library holds these 32 MiB + 64 KiB from load until exit, and no allocation routine is
// ever called.
//
// Consequences of the array being one shared, persistent object:
//   - its size bounds the shapes served: the output padded to whole tiles (M and N rounded up to
//     256) may have at most kMaxPaddedOutputs = 2 Mi elements; larger calls get PQ_ERR_LIMIT;
//   - every call on a device uses the same array, so two calls that overlap on the GPU (different
//     streams, or graph branches) race on it -- serialize them;
//   - it keeps the last call's contents.  The partial sums need no clearing (each is overwritten
//     before it is read); the arrival counters must be zero when a call starts, which holds at load
//     (static storage is zero-initialized) and is re-established by the kernel itself at the end of
//     every call that completes.  A call whose bounded waits ran out (PQ_ERR_TIMEOUT) may leave them
//     non-zero: pq_device_status(), which reports that condition, clears them again with a memset on
//     the array's device address (no allocation).
#include <cuda_runtime.h>

#include <atomic>
#include <mutex>

#include "pq_internal.h"

namespace pq {
namespace {

constexpr int64_t kMaxPaddedOutputs = int64_t(1) << 21;
constexpr int kMaxKParts = 4;
constexpr size_t kStaticPartialBytes = static_cast<size_t>(kMaxPaddedOutputs) * sizeof(int32_t) * kMaxKParts;  // 32 MiB
constexpr size_t kStaticScratchBytes = kScratchHeaderBytes + kStaticPartialBytes;

// In host code this name is only a handle for the runtime's symbol table, NOT a device address:
// it must never be passed to a kernel.  The device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
struct PerDevice {
  std::atomic<bool> ready{false};   // published last; the fill happens under g_mutex
  Scratch scratch;
};
PerDevice g_per_device[kMaxDevices];
std::mutex g_mutex;

// Once per device, with that device current: resolve the array's device address.
int static_scratch(Scratch* out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  PerDevice& d = g_per_device[dev];
  if (!d.ready.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!d.ready.load(std::memory_order_relaxed)) {
      unsigned char* ptr = nullptr;
      if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess || ptr == nullptr) {
        cudaGetLastError();
        return PQ_ERR_CUDA;
      }
      d.scratch.counters = reinterpret_cast<unsigned int*>(ptr);
      d.scratch.partials = reinterpret_cast<int32_t*>(ptr + kScratchHeaderBytes);
      d.scratch.partial_bytes = kStaticPartialBytes;
      d.ready.store(true, std::memory_order_release);
    }
  }
  *out = d.scratch;
  return PQ_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// After a wait ran out: put the array's arrival counters back to zero on the current device, if the
// array was ever used there.  Called by pq_device_status (which has synchronized the device).
int reset_static_scratch() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  PerDevice& d = g_per_device[dev];
  if (!d.ready.load(std::memory_order_acquire)) return PQ_OK;
  if (cudaMemset(d.scratch.counters, 0, kScratchHeaderBytes) != cudaSuccess) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  return PQ_OK;
}

}  // namespace pq

using namespace pq;

extern "C" int pq_gemm_w8a8_noalloc(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch,
                                    int64_t M, int64_t N, int64_t K, void* y_f16, void* stream) {
  if (!q || !s_tok || !wq || !s_ch || !y_f16) return PQ_ERR_NULL;
  if (M < 1 || M > 0x7fffffff || N < 8 || N % 8 != 0 || N > 0x7fffffff) return PQ_ERR_SHAPE;
  if (K < 16 || K % 16 != 0 || K >= 131072) return PQ_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(wq) || !aligned16(y_f16)) return PQ_ERR_ALIGN;
  if (M <= 128) {
    // These token counts run on a schedule that reduces inside the SMs and uses no scratch at all:
    // no limit applies.
    return pq_gemm_w8a8(q, s_tok, wq, s_ch, M, N, K, y_f16, nullptr, 0, stream);
  }
  const int64_t padded = ((M + 255) / 256) * 256 * (((N + 255) / 256) * 256);
  if (padded > kMaxPaddedOutputs) return PQ_ERR_LIMIT;   // beyond what the fixed scratch array serves
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int major = 0, minor = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  if (major != 10 || minor != 0) return PQ_ERR_ARCH;
  Scratch sc;
  const int rc = static_scratch(&sc);
  if (rc != PQ_OK) return rc;
  return launch_gemm_w8a8_pair(sc, q, s_tok, wq, s_ch, M, N, K, y_f16, nullptr, st);
}
