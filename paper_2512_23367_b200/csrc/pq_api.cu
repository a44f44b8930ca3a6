// C-ABI entry points of libpq: argument validation, device checks, dispatch.
// See include/pq.h for the contract of every call.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "pq_internal.h"
#include "pq_ptx.cuh"

namespace pq {

__device__ int g_status_word = 0;

namespace {

constexpr int kMaxDevices = 64;
constexpr int64_t kSmallM = 128;     // W4A8: M at or below this takes the weight-streaming schedule
constexpr int64_t kSmallM_W8 = 128;  // W8A8
constexpr int64_t kStreamM = 256;    // above the limits above: the weight-streaming schedule in blocks of 128 tokens, where every
                                     // (128-channel tile, token block) pair gets an SM of its own (few, long tiles)

// Facts about a device, filled in by the first call on it.  Host threads may make that first call
// concurrently: the fill happens under a mutex and `probed` is published last.
struct DeviceInfo {
  std::atomic<bool> probed{false};
  bool ok = false;
  int sms = 0;
  int* status = nullptr;
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;
std::atomic<uint32_t> g_wait_limit{kWaitPollLimit};

DeviceInfo* current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  DeviceInfo& d = g_dev[dev];
  if (!d.probed.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!d.probed.load(std::memory_order_relaxed)) {
      int major = 0, minor = 0, sms = 0;
      if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return nullptr;
      if (cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess) return nullptr;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
      d.sms = sms;
      d.ok = (major == 10 && minor == 0);
      if (d.ok) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        d.status = static_cast<int*>(p);
      }
      d.probed.store(true, std::memory_order_release);
    }
  }
  return &d;
}

int check_arch() {
  DeviceInfo* d = current_device();
  if (d == nullptr) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  return d->ok ? PQ_OK : PQ_ERR_ARCH;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_rows(int64_t rows, int64_t K) {
  if (rows < 1 || rows > 0x7fffffff) return PQ_ERR_SHAPE;
  if (K < 16 || K % 16 != 0 || K >= 131072) return PQ_ERR_SHAPE;
  return PQ_OK;
}

int check_gemm(int64_t M, int64_t N, int64_t K) {
  int rc = check_rows(M, K);
  if (rc != PQ_OK) return rc;
  if (N < 8 || N % 8 != 0 || N > 0x7fffffff) return PQ_ERR_SHAPE;
  if (M * N > (int64_t(1) << 40)) return PQ_ERR_SHAPE;
  return PQ_OK;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);
// cuTensorMapEncodeTiled, looked up once (thread-safe: initialisation of a function-local static).
EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      p = nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

}  // namespace

int* device_status_ptr() {
  DeviceInfo* d = current_device();
  return d ? d->status : nullptr;
}

uint32_t wait_limit() { return g_wait_limit.load(std::memory_order_relaxed); }

// Name of the CUDA error behind the calling thread's most recent PQ_ERR_CUDA ("" if none was recorded).
static thread_local const char* g_last_cuda_error = "";
void note_cuda_error(cudaError_t e) {
  if (e != cudaSuccess) g_last_cuda_error = cudaGetErrorName(e);
}

int sm_count() {
  DeviceInfo* d = current_device();
  return d ? d->sms : 1;
}

// Whether one to four tokens take the CUDA-core row kernel (default yes; PQ_GEMV=0 sends them to the
// tensor-core weight-streaming kernel instead, for ablations).
static bool gemv_enabled() {
  static const bool on = [] {
    const char* e = getenv("PQ_GEMV");
    return !(e != nullptr && e[0] == '0');
  }();
  return on;
}

// PQ_LOG=1 in the environment: one line on stderr per GEMM call saying which schedule it was given.
static bool log_enabled() {
  static const bool on = [] {
    const char* e = getenv("PQ_LOG");
    return e != nullptr && e[0] == '1';
  }();
  return on;
}
static void log_dispatch(const char* call, const char* schedule, int64_t M, int64_t N, int64_t K) {
  if (log_enabled()) fprintf(stderr, "[pq] %s M=%lld N=%lld K=%lld -> %s\n", call, (long long)M, (long long)N, (long long)K, schedule);
}

bool pdl_enabled() {
  static const bool on = [] {
    const char* e = getenv("PQ_PDL");
    return !(e != nullptr && e[0] == '0');
  }();
  return on;
}

int make_tmap_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                 uint32_t box_cols, uint32_t elem_bytes, int swizzle_bytes) {
  const EncodeTiledFn g_encode = encode_fn();
  if (g_encode == nullptr) return PQ_ERR_CUDA;
  CUtensorMapDataType dt = elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                           : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16
                                             : CU_TENSOR_MAP_DATA_TYPE_UINT32;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * elem_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = swizzle_bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
                               : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                               : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                     : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = g_encode(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PQ_OK : PQ_ERR_CUDA;
}

}  // namespace pq

using namespace pq;

extern "C" {

const char* pq_last_cuda_error(void) { return g_last_cuda_error; }

const char* pq_status_str(int status) {
  switch (status) {
    case PQ_OK: return "ok";
    case PQ_ERR_NULL: return "null pointer argument";
    case PQ_ERR_SHAPE: return "invalid shape";
    case PQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case PQ_ERR_ARCH: return "device is not compute capability 10.0";
    case PQ_ERR_CUDA: return "CUDA call or launch failed";
    case PQ_ERR_TIMEOUT: return "bounded wait inside a kernel expired";
    case PQ_ERR_LIMIT: return "size exceeds the entry point's maximum";
    default: return "unknown status";
  }
}

size_t pq_packed_w8_bytes(int64_t N, int64_t K) {
  return (N > 0 && K > 0) ? static_cast<size_t>(N) * static_cast<size_t>(K) : 0;
}
size_t pq_packed_w4_bytes(int64_t N, int64_t K) {
  return (N > 0 && K > 0) ? static_cast<size_t>(N) * static_cast<size_t>(K) / 2 : 0;
}

static int quantize_act_common(const void* x_f16, const float* col, int64_t M, int64_t K, int8_t* q, float* s_tok,
                               void* stream) {
  if (!x_f16 || !q || !s_tok) return PQ_ERR_NULL;
  int rc = check_rows(M, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(x_f16) || !aligned16(q) || !aligned16(col)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_quantize_act(x_f16, M, K, q, s_tok, false, col, static_cast<cudaStream_t>(stream));
}

int pq_quantize_act(const void* x_f16, int64_t M, int64_t K, int8_t* q, float* s_tok, void* stream) {
  return quantize_act_common(x_f16, nullptr, M, K, q, s_tok, stream);
}

int pq_quantize_act_smooth(const void* x_f16, const float* s_inv, int64_t M, int64_t K, int8_t* q, float* s_tok,
                           void* stream) {
  if (!s_inv) return PQ_ERR_NULL;
  return quantize_act_common(x_f16, s_inv, M, K, q, s_tok, stream);
}

static int pack_w8_common(const void* w_f16, const float* col, int64_t N, int64_t K, void* wq, float* s_ch,
                          void* stream) {
  if (!w_f16 || !wq || !s_ch) return PQ_ERR_NULL;
  int rc = check_gemm(1, N, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(w_f16) || !aligned16(wq) || !aligned16(col)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  // The W8 layout the GEMM reads is the row-major code matrix itself (K contiguous per channel).
  rc = launch_quantize_act(w_f16, N, K, static_cast<int8_t*>(wq), s_ch, true, col, static_cast<cudaStream_t>(stream));
  return rc != PQ_OK ? rc : launch_pack_fence(static_cast<cudaStream_t>(stream));
}

int pq_pack_w8(const void* w_f16, int64_t N, int64_t K, void* wq, float* s_ch, void* stream) {
  return pack_w8_common(w_f16, nullptr, N, K, wq, s_ch, stream);
}

int pq_pack_w8_smooth(const void* w_f16, const float* s, int64_t N, int64_t K, void* wq, float* s_ch, void* stream) {
  if (!s) return PQ_ERR_NULL;
  return pack_w8_common(w_f16, s, N, K, wq, s_ch, stream);
}

static int pack_w4_common(const void* w_f16, const float* col, int64_t N, int64_t K, int32_t group, void* wp,
                          void* s_grp_f16, void* stream) {
  if (!w_f16 || !wp || !s_grp_f16) return PQ_ERR_NULL;
  int rc = check_gemm(1, N, K);
  if (rc != PQ_OK) return rc;
  if (group != 128 || K % 128 != 0) return PQ_ERR_SHAPE;
  if (!aligned16(w_f16) || !aligned16(wp) || !aligned16(s_grp_f16)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  rc = launch_pack_w4(w_f16, N, K, wp, s_grp_f16, col, static_cast<cudaStream_t>(stream));
  return rc != PQ_OK ? rc : launch_pack_fence(static_cast<cudaStream_t>(stream));
}

int pq_pack_w4(const void* w_f16, int64_t N, int64_t K, int32_t group, void* wp, void* s_grp_f16, void* stream) {
  return pack_w4_common(w_f16, nullptr, N, K, group, wp, s_grp_f16, stream);
}

int pq_pack_w4_smooth(const void* w_f16, const float* s, int64_t N, int64_t K, int32_t group, void* wp,
                      void* s_grp_f16, void* stream) {
  if (!s) return PQ_ERR_NULL;
  return pack_w4_common(w_f16, s, N, K, group, wp, s_grp_f16, stream);
}

int pq_quantize_act_static(const void* x_f16, const float* scale, int64_t M, int64_t K, int8_t* q, float* s_tok,
                           void* stream) {
  if (!x_f16 || !scale || !q || !s_tok) return PQ_ERR_NULL;
  int rc = check_rows(M, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(x_f16) || !aligned16(q)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_quantize_act_static(x_f16, scale, M, K, q, s_tok, static_cast<cudaStream_t>(stream));
}

int pq_quantize_act_static_channel(const void* x_f16, const float* inv_s, int64_t M, int64_t K, int8_t* q, float* s_tok,
                                   void* stream) {
  if (!x_f16 || !inv_s || !q || !s_tok) return PQ_ERR_NULL;
  int rc = check_rows(M, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(x_f16) || !aligned16(q) || !aligned16(inv_s)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_quantize_act_static_channel(x_f16, inv_s, M, K, q, s_tok, static_cast<cudaStream_t>(stream));
}

int pq_swiglu_quantize(const void* gate_f16, const void* up_f16, int64_t M, int64_t I, int8_t* q, float* s_tok,
                       void* stream) {
  if (!gate_f16 || !up_f16 || !q || !s_tok) return PQ_ERR_NULL;
  int rc = check_rows(M, I);
  if (rc != PQ_OK) return rc;
  if (I > 16384) return PQ_ERR_SHAPE;
  if (!aligned16(gate_f16) || !aligned16(up_f16) || !aligned16(q)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_swiglu_quantize(gate_f16, up_f16, M, I, q, s_tok, static_cast<cudaStream_t>(stream));
}

int32_t pq_hadamard_block(int64_t K) { return (K >= 16 && K % 16 == 0) ? hadamard_block_order(K) : 0; }

int pq_quantize_act_hadamard(const void* x_f16, int64_t M, int64_t K, int8_t* q, float* s_tok, void* stream) {
  if (!x_f16 || !q || !s_tok) return PQ_ERR_NULL;
  int rc = check_rows(M, K);
  if (rc != PQ_OK) return rc;
  if (K > 16384) return PQ_ERR_SHAPE;
  if (!aligned16(x_f16) || !aligned16(q)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_quantize_act_hadamard(x_f16, M, K, q, s_tok, false, static_cast<cudaStream_t>(stream));
}

int pq_pack_w8_hadamard(const void* w_f16, int64_t N, int64_t K, void* wq, float* s_ch, void* stream) {
  if (!w_f16 || !wq || !s_ch) return PQ_ERR_NULL;
  int rc = check_gemm(1, N, K);
  if (rc != PQ_OK) return rc;
  if (K > 16384) return PQ_ERR_SHAPE;
  if (!aligned16(w_f16) || !aligned16(wq)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  rc = launch_quantize_act_hadamard(w_f16, N, K, static_cast<int8_t*>(wq), s_ch, true, static_cast<cudaStream_t>(stream));
  return rc != PQ_OK ? rc : launch_pack_fence(static_cast<cudaStream_t>(stream));
}

int pq_pack_w4_hadamard(const void* w_f16, int64_t N, int64_t K, int32_t group, void* wp, void* s_grp_f16,
                        void* stream) {
  if (!w_f16 || !wp || !s_grp_f16) return PQ_ERR_NULL;
  int rc = check_gemm(1, N, K);
  if (rc != PQ_OK) return rc;
  if (group != 128 || K % 128 != 0) return PQ_ERR_SHAPE;
  if (!aligned16(w_f16) || !aligned16(wp) || !aligned16(s_grp_f16)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  rc = launch_pack_w4_hadamard(w_f16, N, K, wp, s_grp_f16, static_cast<cudaStream_t>(stream));
  return rc != PQ_OK ? rc : launch_pack_fence(static_cast<cudaStream_t>(stream));
}

int pq_col_absmax(const void* a_f16, int64_t R, int64_t K, float* out, void* stream) {
  if (!a_f16 || !out) return PQ_ERR_NULL;
  int rc = check_rows(R, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(a_f16)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_col_absmax(a_f16, R, K, out, static_cast<cudaStream_t>(stream));
}

int pq_smooth_scales_alpha(const float* x_absmax, const float* w_absmax, int64_t K, int32_t alpha_quarters, float* s,
                           float* s_inv, void* stream) {
  if (!x_absmax || !w_absmax || !s || !s_inv) return PQ_ERR_NULL;
  if (K < 1 || K >= 131072 || alpha_quarters < 0 || alpha_quarters > 4) return PQ_ERR_SHAPE;
  const int rc = check_arch();
  if (rc != PQ_OK) return rc;
  return launch_smooth_scales(x_absmax, w_absmax, K, alpha_quarters, s, s_inv, static_cast<cudaStream_t>(stream));
}

int pq_smooth_scales(const float* x_absmax, const float* w_absmax, int64_t K, float* s, float* s_inv, void* stream) {
  return pq_smooth_scales_alpha(x_absmax, w_absmax, K, 2, s, s_inv, stream);
}

int pq_unpack_w8(const void* wq, int64_t N, int64_t K, int8_t* codes, void* stream) {
  if (!wq || !codes) return PQ_ERR_NULL;
  int rc = check_gemm(1, N, K);
  if (rc != PQ_OK) return rc;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return cuda_status(cudaMemcpyAsync(codes, wq, static_cast<size_t>(N) * K, cudaMemcpyDeviceToDevice,
                                     static_cast<cudaStream_t>(stream)));
}

int pq_unpack_w4(const void* wp, int64_t N, int64_t K, int8_t* codes, void* stream) {
  if (!wp || !codes) return PQ_ERR_NULL;
  int rc = check_gemm(1, N, K);
  if (rc != PQ_OK) return rc;
  if (K % 128 != 0) return PQ_ERR_SHAPE;
  if ((rc = check_arch()) != PQ_OK) return rc;
  return launch_unpack_w4(wp, N, K, codes, static_cast<cudaStream_t>(stream));
}

static bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

// 129..256 tokens: a narrow linear gives the pair kernel few 256 x 256 tiles (256 x 4096 -> 4096: 16 on 74 SM
// pairs); the weight-streaming kernel takes it in two token blocks and splits K over clusters instead.
// `tiles` = 128-channel tiles of all members of the launch.
static bool w8a8_streams_in_blocks(int64_t M, int64_t tiles) {
  return M > kSmallM_W8 && M <= kStreamM && tiles * ((M + 127) / 128) <= sm_count();
}

static int gemm_w8a8_common(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M,
                            int64_t N, int64_t K, void* y, int32_t* acc, void* workspace, size_t workspace_bytes,
                            void* stream) {
  int rc = check_gemm(M, N, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(q) || !aligned16(wq) || !aligned16(y) || !aligned16(acc) || !aligned256(workspace)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Up to 128 tokens: the weight-streaming schedule (tokens are the narrow MMA dimension, K split over a
  // cluster); beyond that the second CTA of a pair no longer holds only padding rows.
  if (gemv_enabled() && gemv_rows_serves(8, M, N, K, sm_count())) {
    log_dispatch("w8a8", "CUDA-core row kernel", M, N, K);
    return launch_gemv_rows_w8a8(q, s_tok, wq, s_ch, M, N, K, y, acc, st);
  }
  if (M <= kSmallM_W8 || w8a8_streams_in_blocks(M, (N + 127) / 128)) {
    log_dispatch("w8a8", "tensor-core weight streaming", M, N, K);
    return launch_smallm_w8a8(q, s_tok, wq, s_ch, M, N, K, y, acc, st);
  }
  log_dispatch("w8a8", "pair GEMM", M, N, K);
  return launch_gemm_w8a8_pair(scratch_from(workspace, workspace_bytes), q, s_tok, wq, s_ch, M, N, K, y, acc, st);
}

int pq_gemm_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M, int64_t N,
                 int64_t K, void* y_f16, void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !s_tok || !wq || !s_ch || !y_f16) return PQ_ERR_NULL;
  return gemm_w8a8_common(q, s_tok, wq, s_ch, M, N, K, y_f16, nullptr, workspace, workspace_bytes, stream);
}

int pq_gemm_w8a8_group(const int8_t* q, const float* s_tok, int32_t count, const void* const* wq,
                       const float* const* s_ch, const int64_t* N, void* const* y_f16, int64_t M, int64_t K,
                       void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !s_tok || !wq || !s_ch || !N || !y_f16) return PQ_ERR_NULL;
  if (count < 1 || count > PQ_MAX_GROUP) return PQ_ERR_SHAPE;
  for (int g = 0; g < count; ++g) {
    if (!wq[g] || !s_ch[g] || !y_f16[g]) return PQ_ERR_NULL;
    const int rc = check_gemm(M, N[g], K);
    if (rc != PQ_OK) return rc;
    if (!aligned16(wq[g]) || !aligned16(y_f16[g])) return PQ_ERR_ALIGN;
  }
  if (!aligned16(q) || !aligned256(workspace)) return PQ_ERR_ALIGN;
  int rc = check_arch();
  if (rc != PQ_OK) return rc;
  int64_t tiles = 0;
  for (int g = 0; g < count; ++g) tiles += (N[g] + 127) / 128;
  if (M <= kSmallM_W8 || w8a8_streams_in_blocks(M, tiles)) {
    return launch_smallm_w8a8_group(q, s_tok, count, wq, s_ch, N, y_f16, M, K, nullptr,
                                    static_cast<cudaStream_t>(stream));
  }
  return launch_gemm_w8a8_pair_group(scratch_from(workspace, workspace_bytes), q, s_tok, count, wq, s_ch, N, y_f16,
                                     M, K, nullptr, static_cast<cudaStream_t>(stream));
}

int pq_acc_w8a8(const int8_t* q, const void* wq, int64_t M, int64_t N, int64_t K, int32_t* acc, void* stream) {
  if (!q || !wq || !acc) return PQ_ERR_NULL;
  return gemm_w8a8_common(q, nullptr, wq, nullptr, M, N, K, nullptr, acc, nullptr, 0, stream);
}

// W4A8 between kSmallM and kStreamM tokens: the pair kernel's 256 x 256 tiles leave most SM pairs idle when
// the linear is narrow (256 x 4096 -> 4096: 16 tiles, 30.9 us); the weight-streaming kernel splits K over
// clusters instead.  `tiles` = 128-channel tiles of all members of the launch.
static bool w4a8_streams_in_blocks(int64_t M, int64_t tiles) {
  return M > kSmallM && M <= kStreamM && tiles * ((M + 127) / 128) <= sm_count();
}

static int gemm_w4a8_common(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int32_t group,
                            int64_t M, int64_t N, int64_t K, void* y, int32_t* acc_g, void* stream) {
  int rc = check_gemm(M, N, K);
  if (rc != PQ_OK) return rc;
  if (group != 128 || K % 128 != 0) return PQ_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(wp) || !aligned16(s_grp) || !aligned16(y) || !aligned16(acc_g)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (gemv_enabled() && gemv_rows_serves(4, M, N, K, sm_count())) {
    log_dispatch("w4a8", "CUDA-core row kernel", M, N, K);
    return launch_gemv_rows_w4a8(q, s_tok, wp, s_grp, M, N, K, y, acc_g, st);
  }
  if (M <= kSmallM || w4a8_streams_in_blocks(M, (N + 127) / 128)) {
    log_dispatch("w4a8", "tensor-core weight streaming", M, N, K);
    return launch_smallm_w4a8(q, s_tok, wp, s_grp, M, N, K, y, acc_g, st);
  }
  log_dispatch("w4a8", "pair GEMM", M, N, K);
  return launch_gemm_w4a8(q, s_tok, wp, s_grp, M, N, K, y, acc_g, st);
}

int pq_gemm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp_f16, int32_t group,
                 int64_t M, int64_t N, int64_t K, void* y_f16, void* stream) {
  if (!q || !s_tok || !wp || !s_grp_f16 || !y_f16) return PQ_ERR_NULL;
  return gemm_w4a8_common(q, s_tok, wp, s_grp_f16, group, M, N, K, y_f16, nullptr, stream);
}

// S1-S4 in one call.  Where the CUDA-core row kernel serves the shape it quantizes its own tokens (one launch);
// otherwise the quantizer and the GEMM run one after the other through the caller's q / s_tok buffers.
int pq_linear_w8a8(const void* x_f16, const void* wq, const float* s_ch, int64_t M, int64_t N, int64_t K, void* y_f16,
                   int8_t* q_tmp, float* s_tok_tmp, void* workspace, size_t workspace_bytes, void* stream) {
  if (!x_f16 || !wq || !s_ch || !y_f16 || !q_tmp || !s_tok_tmp) return PQ_ERR_NULL;
  int rc = check_gemm(M, N, K);
  if (rc != PQ_OK) return rc;
  if (!aligned16(x_f16) || !aligned16(wq) || !aligned16(y_f16) || !aligned16(q_tmp) || !aligned256(workspace)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  if (gemv_enabled() && gemv_rows_serves(8, M, N, K, sm_count())) {
    log_dispatch("w8a8", "CUDA-core row kernel, tokens quantized in the kernel", M, N, K);
    return launch_gemv_rows_w8a8_x(x_f16, wq, s_ch, M, N, K, y_f16, static_cast<cudaStream_t>(stream));
  }
  rc = pq_quantize_act(x_f16, M, K, q_tmp, s_tok_tmp, stream);
  if (rc != PQ_OK) return rc;
  return pq_gemm_w8a8(q_tmp, s_tok_tmp, wq, s_ch, M, N, K, y_f16, workspace, workspace_bytes, stream);
}

int pq_linear_w4a8(const void* x_f16, const void* wp, const void* s_grp_f16, int32_t group, int64_t M, int64_t N,
                   int64_t K, void* y_f16, int8_t* q_tmp, float* s_tok_tmp, void* stream) {
  if (!x_f16 || !wp || !s_grp_f16 || !y_f16 || !q_tmp || !s_tok_tmp) return PQ_ERR_NULL;
  int rc = check_gemm(M, N, K);
  if (rc != PQ_OK) return rc;
  if (group != 128 || K % 128 != 0) return PQ_ERR_SHAPE;
  if (!aligned16(x_f16) || !aligned16(wp) || !aligned16(s_grp_f16) || !aligned16(y_f16) || !aligned16(q_tmp)) return PQ_ERR_ALIGN;
  if ((rc = check_arch()) != PQ_OK) return rc;
  if (gemv_enabled() && gemv_rows_serves(4, M, N, K, sm_count())) {
    log_dispatch("w4a8", "CUDA-core row kernel, tokens quantized in the kernel", M, N, K);
    return launch_gemv_rows_w4a8_x(x_f16, wp, s_grp_f16, M, N, K, y_f16, static_cast<cudaStream_t>(stream));
  }
  rc = pq_quantize_act(x_f16, M, K, q_tmp, s_tok_tmp, stream);
  if (rc != PQ_OK) return rc;
  return pq_gemm_w4a8(q_tmp, s_tok_tmp, wp, s_grp_f16, group, M, N, K, y_f16, stream);
}

int pq_gemm_w4a8_group(const int8_t* q, const float* s_tok, int32_t count, const void* const* wp,
                       const void* const* s_grp_f16, int32_t group, const int64_t* N, void* const* y_f16, int64_t M,
                       int64_t K, void* stream) {
  if (!q || !s_tok || !wp || !s_grp_f16 || !N || !y_f16) return PQ_ERR_NULL;
  if (count < 1 || count > PQ_MAX_GROUP) return PQ_ERR_SHAPE;
  if (group != 128 || K % 128 != 0) return PQ_ERR_SHAPE;
  for (int g = 0; g < count; ++g) {
    if (!wp[g] || !s_grp_f16[g] || !y_f16[g]) return PQ_ERR_NULL;
    const int rc = check_gemm(M, N[g], K);
    if (rc != PQ_OK) return rc;
    if (!aligned16(wp[g]) || !aligned16(s_grp_f16[g]) || !aligned16(y_f16[g])) return PQ_ERR_ALIGN;
  }
  if (!aligned16(q)) return PQ_ERR_ALIGN;
  int rc = check_arch();
  if (rc != PQ_OK) return rc;
  if (M <= kSmallM) {
    // One launch, unless the members together hold more 128-channel tiles than the device has SMs:
    // the K dimension would then not be split at all, and the widening makes a CTA's chain over all of K
    // slower than separate launches (2 x 4096->11008 at M=1: 23.8 us grouped, 22.4 us separately).
    int64_t tiles = 0;
    for (int g = 0; g < count; ++g) tiles += (N[g] + 127) / 128;
    if (count > 1 && tiles > sm_count()) {
      for (int g = 0; g < count; ++g) {
        rc = gemm_w4a8_common(q, s_tok, wp[g], s_grp_f16[g], group, M, N[g], K, y_f16[g], nullptr, stream);
        if (rc != PQ_OK) return rc;
      }
      return PQ_OK;
    }
    return launch_smallm_w4a8_group(q, s_tok, count, wp, s_grp_f16, N, y_f16, M, K, nullptr,
                                    static_cast<cudaStream_t>(stream));
  }
  {
    int64_t tiles = 0;
    for (int g = 0; g < count; ++g) tiles += (N[g] + 127) / 128;
    if (w4a8_streams_in_blocks(M, tiles))
      return launch_smallm_w4a8_group(q, s_tok, count, wp, s_grp_f16, N, y_f16, M, K, nullptr,
                                      static_cast<cudaStream_t>(stream));
  }
  return launch_gemm_w4a8_group(q, s_tok, count, wp, s_grp_f16, N, y_f16, M, K, nullptr,
                                static_cast<cudaStream_t>(stream));
}

int pq_acc_w4a8(const int8_t* q, const void* wp, int32_t group, int64_t M, int64_t N, int64_t K, int32_t* acc_g,
                void* stream) {
  if (!q || !wp || !acc_g) return PQ_ERR_NULL;
  return gemm_w4a8_common(q, nullptr, wp, nullptr, group, M, N, K, nullptr, acc_g, stream);
}

int pq_plan_w8a8(int64_t M, int64_t N, int64_t K, int32_t sms, size_t scratch_bytes, int32_t* tile_n,
                 int32_t* k_parts) {
  if (!tile_n || !k_parts) return PQ_ERR_NULL;
  int rc = check_gemm(M, N, K);
  if (rc != PQ_OK) return rc;
  if (sms < 2) return PQ_ERR_SHAPE;
  int bn = 256, sp = 1;
  const size_t room = scratch_bytes > kScratchHeaderBytes ? scratch_bytes - kScratchHeaderBytes : 0;
  if (plan_w8a8_pair(M, N, K, sms, room, 0, 0, &bn, &sp) < 0) return PQ_ERR_SHAPE;
  *tile_n = bn;
  *k_parts = sp;
  return PQ_OK;
}

size_t pq_workspace_bytes(int64_t M, const int64_t* N, int32_t count, int64_t K, int32_t sms) {
  if (!N || count < 1 || count > PQ_MAX_GROUP || sms < 2) return 0;
  for (int g = 0; g < count; ++g) {
    if (check_gemm(M, N[g], K) != PQ_OK) return 0;
  }
  if (M <= kSmallM_W8) return 0;   // the weight-streaming schedule reduces inside the SMs
  if (M <= kStreamM) {             // ... and so it does in two token blocks, for narrow linears
    int64_t tiles = 0;
    for (int g = 0; g < count; ++g) tiles += (N[g] + 127) / 128;
    if (tiles * ((M + 127) / 128) <= sms) return 0;
  }
  int bn = 256, sp = 1;
  // the schedule chosen when room is no constraint
  if (plan_w8a8_pair_group(M, N, count, K, sms, ~size_t(0), 0, 0, &bn, &sp) < 0 || sp <= 1) return 0;
  return kScratchHeaderBytes + w8a8_pair_partial_bytes(M, N, count, bn, sp);
}

int pq_workspace_init(void* workspace, size_t bytes, void* stream) {
  if (!workspace) return PQ_ERR_NULL;
  if (!aligned256(workspace)) return PQ_ERR_ALIGN;
  if (bytes < kScratchHeaderBytes) return PQ_ERR_SHAPE;
  // the arrival counters must read zero when a GEMM first uses them
  if (cudaMemsetAsync(workspace, 0, kScratchHeaderBytes, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  return PQ_OK;
}

int pq_set_wait_limit(uint32_t polls) {
  g_wait_limit.store(polls == 0 ? kWaitPollLimit : (polls == PQ_WAIT_NONE ? 0u : polls), std::memory_order_relaxed);
  return PQ_OK;
}

int pq_device_status(int* host_status) {
  if (!host_status) return PQ_ERR_NULL;
  int rc = check_arch();
  if (rc != PQ_OK) return rc;
  int* p = device_status_ptr();
  if (!p) return PQ_ERR_CUDA;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    note_cuda_error(e);
    return PQ_ERR_CUDA;
  }
  int v = 0;
  if ((e = cudaMemcpy(&v, p, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess) {
    note_cuda_error(e);
    return PQ_ERR_CUDA;
  }
  if (v != 0) {
    if (cudaMemset(p, 0, sizeof(int)) != cudaSuccess) return PQ_ERR_CUDA;
    // A call that gave up may have left arrival counters of the built-in scratch array non-zero.
    if ((rc = reset_static_scratch()) != PQ_OK) return rc;
  }
  *host_status = v;
  return PQ_OK;
}

}  // extern "C"
