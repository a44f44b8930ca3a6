// Row-wise symmetric quantizers (Eq. 1-2 of the paper):
//   - per-token INT8 activation quantization (hot path, HBM bound: 2 B read + 1 B written
//     per element),
//   - per-output-channel INT8 weight quantization (offline),
//   - group-wise INT4 weight quantization + nibble packing (offline), and its inverse.
#include <cuda_fp16.h>

#include <cmath>

#include "pq_internal.h"
#include "pq_ptx.cuh"
#include "pq_quant_math.cuh"

namespace pq {

// Order of the Hadamard blocks for rows of length K (Eq. 4): K itself where K is a power of two (up to
// 16384: the Sylvester matrix of the row's own order), else the largest power of two dividing K, at most 256.
int hadamard_block_order(int64_t K) {
  if (K >= 1 && K <= 16384 && (K & (K - 1)) == 0) return static_cast<int>(K);
  int B = 1;
  while (B < 256 && K % (2 * B) == 0) B *= 2;
  return B;
}

namespace {

constexpr int kThreads = 256;
constexpr int kCached = 8;  // 16-byte chunks of a row that one thread keeps in registers

// The eight values of a 16-byte chunk as the quantizer sees them: the FP16 elements, times the
// column factors of Eq. 3 (one FP32 product each, not rounded back to FP16) when kSmooth.
template <bool kSmooth>
__device__ __forceinline__ void values8(const uint4& v, const float4* __restrict__ col, int chunk, float (&t)[8]) {
  const __half* h = reinterpret_cast<const __half*>(&v);
#pragma unroll
  for (int i = 0; i < 8; ++i) t[i] = __half2float(h[i]);
  if constexpr (kSmooth) {
    const float4 c0 = __ldg(col + 2 * chunk), c1 = __ldg(col + 2 * chunk + 1);
    t[0] = __fmul_rn(t[0], c0.x); t[1] = __fmul_rn(t[1], c0.y); t[2] = __fmul_rn(t[2], c0.z); t[3] = __fmul_rn(t[3], c0.w);
    t[4] = __fmul_rn(t[4], c1.x); t[5] = __fmul_rn(t[5], c1.y); t[6] = __fmul_rn(t[6], c1.z); t[7] = __fmul_rn(t[7], c1.w);
  }
}

template <bool kSmooth>
__device__ __forceinline__ float absmax8v(const uint4& v, const float4* __restrict__ col, int chunk) {
  if constexpr (!kSmooth) {
    return absmax8(v);
  } else {
    float t[8];
    values8<true>(v, col, chunk, t);
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) a = fmaxf(a, fabsf(t[i]));
    return a;
  }
}

template <bool kDivide, bool kSmooth>
__device__ __forceinline__ uint2 quantize8(const uint4& v, float f, const float4* __restrict__ col, int chunk) {
  float t[8];
  values8<kSmooth>(v, col, chunk, t);
  return make_uint2(codes4<kDivide>(t[0], t[1], t[2], t[3], f), codes4<kDivide>(t[4], t[5], t[6], t[7], f));
}

// T threads cooperate on one row; a block of 256 threads handles 256/T rows.
//   kDivide = false: activations, code = rne(x * (127.5 / a))
//   kDivide = true : weights,     code = rne(x / (a / 127.5))
//   kSmooth: x is first multiplied by the per-column factor col[k] (Eq. 3: X S^-1 or S W)
template <int T, bool kDivide, bool kSmooth>
__global__ void __launch_bounds__(kThreads) quantize_rows_kernel(const uint4* __restrict__ x, int64_t M,
                                                                 int K8, uint2* __restrict__ q,
                                                                 float* __restrict__ scale,
                                                                 const float4* __restrict__ col) {
  constexpr int kRowsPerBlock = kThreads / T;
  constexpr int kWarpsPerRow = T / 32;
  __shared__ float red[kThreads / 32];

  const int tid = threadIdx.x;
  const int t = tid % T;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kRowsPerBlock + tid / T;
  const bool live = row < M;
  const uint4* xr = x + row * K8;

  // The input may come from the kernel that precedes this one in the stream, and the codes
  // written below may still be read by it: both wait for its completion.  The offline weight
  // quantizer never lets its successor start early (a GEMM may prefetch the weights it writes).
  if constexpr (!kDivide) grid_dep_launch();
  grid_dep_wait();

  uint4 cache[kCached];
  float a = 0.0f;
  if (live) {
#pragma unroll
    for (int i = 0; i < kCached; ++i) {
      int c = t + i * T;
      if (c < K8) {
        cache[i] = __ldg(xr + c);
        a = fmaxf(a, absmax8v<kSmooth>(cache[i], col, c));
      }
    }
    for (int c = t + kCached * T; c < K8; c += T) a = fmaxf(a, absmax8v<kSmooth>(__ldg(xr + c), col, c));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  if constexpr (kWarpsPerRow > 1) {
    if ((tid & 31) == 0) red[tid >> 5] = a;
    __syncthreads();
    const int w0 = (tid / T) * kWarpsPerRow;
#pragma unroll
    for (int w = 0; w < kWarpsPerRow; ++w) a = fmaxf(a, red[w0 + w]);
  }
  if (!live) return;

  const float s = __fdiv_rn(a, 127.5f);
  float f;
  if (kDivide) {
    f = (a == 0.0f) ? 1.0f : s;  // x / 1 = 0 for the all-zero row
  } else {
    f = (a == 0.0f) ? 0.0f : __fdiv_rn(127.5f, a);
  }
  if (t == 0) scale[row] = s;

  uint2* qr = q + row * K8;
#pragma unroll
  for (int i = 0; i < kCached; ++i) {
    int c = t + i * T;
    if (c < K8) qr[c] = quantize8<kDivide, kSmooth>(cache[i], f, col, c);
  }
  for (int c = t + kCached * T; c < K8; c += T) qr[c] = quantize8<kDivide, kSmooth>(__ldg(xr + c), f, col, c);
}

// ---------------------------------------------------------------------------- Eq. 4 (Hadamard variant)
// Rows are multiplied by H = I (x) H_B / sqrt(B) before they are quantized: H_B the Sylvester matrix
// of order B = largest power of two dividing K (at most 256), applied as the in-place butterfly with
// distances 1, 2, 4, ..., B/2 in this order.  A thread holds 16-byte chunks (8 consecutive k) and the
// 32 lanes of a warp hold 32 consecutive chunks, so distances 1, 2, 4 stay inside a thread and
// 8 .. 128 are lane exchanges at XOR distance 1 .. 16; a block never leaves its warp.

// One chunk: v[0..8) are elements 8*lane .. 8*lane+7 of the warp's 256-element span.
__device__ __forceinline__ void hadamard_chunk(float (&v)[8], int lane, int chunks_per_block, float norm) {
#pragma unroll
  for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if ((j & h) == 0) {
        const float a = v[j], b = v[j + h];
        v[j] = __fadd_rn(a, b);
        v[j + h] = __fsub_rn(a, b);
      }
    }
  }
  for (int d = 1; d < chunks_per_block; d <<= 1) {
    // a' = a + b in the lower lane, b' = a - b in the upper one: other + sign * v, one exactly rounded
    // fused multiply-add with sign = +-1 (the product is exact, so this IS the sum / difference)
    const float sign = (lane & d) != 0 ? -1.0f : 1.0f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float other = __shfl_xor_sync(0xffffffffu, v[j], d);
      v[j] = __fmaf_rn(sign, v[j], other);
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = __fmul_rn(v[j], norm);
}

// The same transform for a thread that holds C chunks of ONE block: an 8-lane group owns 8*C
// consecutive chunks (C/4 blocks of 32), lane l' of the group the chunks l' + 8 i.  Element index inside
// the block = j + 8 l' + 64 (i mod 4): distances 1-4 stay inside a chunk, 8-32 are lane exchanges at XOR
// distance 1-4, 64 and 128 pair chunks of the same thread -- three exchanges per element instead of five.
template <int C>
__device__ __forceinline__ void hadamard_rows(float (&v)[C][8], int lane, int chunks_per_block, float norm, float* xch) {
#pragma unroll
  for (int i = 0; i < C; ++i) {
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if ((j & h) == 0) {
          const float a = v[i][j], b = v[i][j + h];
          v[i][j] = __fadd_rn(a, b);
          v[i][j + h] = __fsub_rn(a, b);
        }
      }
    }
  }
#pragma unroll
  for (int d = 1; d < 8; d <<= 1) {
    if (d < chunks_per_block) {
      const float sign = (lane & d) != 0 ? -1.0f : 1.0f;   // other + sign * v: the sum below, the difference above
#pragma unroll
      for (int i = 0; i < C; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float other = __shfl_xor_sync(0xffffffffu, v[i][j], d);
          v[i][j] = __fmaf_rn(sign, v[i][j], other);
        }
      }
    }
  }
#pragma unroll
  for (int di = 1; di < C; di <<= 1) {
    if (8 * di < chunks_per_block) {
#pragma unroll
      for (int i = 0; i < C; ++i) {
        if ((i & di) == 0) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float a = v[i][j], b = v[i + di][j];
            v[i][j] = __fadd_rn(a, b);
            v[i + di][j] = __fsub_rn(a, b);
          }
        }
      }
    }
  }
  // Blocks longer than 8 C chunks (only rows rotated as a whole): the four 8-lane groups of the warp hold
  // consecutive runs of 8 C chunks -- two more lane exchanges, at chunk distances 8 C and 16 C.
#pragma unroll
  for (int dl = 8; dl < 32; dl <<= 1) {
    if (dl * C < chunks_per_block) {
      const float sign = (lane & dl) != 0 ? -1.0f : 1.0f;
#pragma unroll
      for (int i = 0; i < C; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float other = __shfl_xor_sync(0xffffffffu, v[i][j], dl);
          v[i][j] = __fmaf_rn(sign, v[i][j], other);
        }
      }
    }
  }
  // ... and the warps of the row team hold consecutive runs of 32 C chunks: one exchange through shared
  // memory per remaining level (chunk distances 32 C, 64 C, ...), `xch` = this block's exchange buffer
  // (8 C floats per thread, or null when no level needs it).  Every thread of the block takes part.
  if (xch != nullptr) {
    for (int dw = 1; dw * 32 * C < chunks_per_block; dw <<= 1) {
      __syncthreads();                      // the previous level's reads are done
#pragma unroll
      for (int i = 0; i < C; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) xch[(i * 8 + j) * kThreads + threadIdx.x] = v[i][j];
      }
      __syncthreads();
      const int partner = static_cast<int>(threadIdx.x) ^ (32 * dw);
      const float sign = (threadIdx.x & (32 * dw)) != 0 ? -1.0f : 1.0f;
#pragma unroll
      for (int i = 0; i < C; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[i][j] = __fmaf_rn(sign, v[i][j], xch[(i * 8 + j) * kThreads + partner]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < C; ++i) {
#pragma unroll
    for (int j = 0; j < 8; ++j) v[i][j] = __fmul_rn(v[i][j], norm);
  }
}

// The row quantizer on transformed rows: the whole row stays in registers as FP32 (K <= 8 * kCached * T),
// so the transform is evaluated once.  kRotate: Eq. 4 (block Hadamard rotation); otherwise Eq. 3 (times
// the column factor col[k]).
// C = chunks per thread: 4 where the row allows it (fewer registers, more resident warps), else 8.
template <int T, int C, bool kDivide, bool kRotate>
__global__ void __launch_bounds__(kThreads) quantize_rows_rot_kernel(const uint4* __restrict__ x, int64_t M,
                                                                     int K8, uint2* __restrict__ q,
                                                                     float* __restrict__ scale,
                                                                     int chunks_per_block, float norm,
                                                                     const float4* __restrict__ col) {
  constexpr int kRowsPerBlock = kThreads / T;
  constexpr int kWarpsPerRow = T / 32;
  __shared__ float red[kThreads / 32];

  const int tid = threadIdx.x;
  const int t = tid % T;
  const int lane = tid & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kRowsPerBlock + tid / T;
  const bool live = row < M;          // uniform per warp: a warp never spans two rows
  const uint4* xr = x + row * K8;

  if constexpr (!kDivide) grid_dep_launch();
  grid_dep_wait();

  // Chunk i of this thread.  Eq. 3: chunks t, t + T, ...  Eq. 4: an 8-lane group owns 8 C consecutive chunks
  // (see hadamard_rows).
  const int chunk0 = kRotate ? (t & ~31) * C + (lane >> 3) * (8 * C) + (lane & 7) : t;
  constexpr int kChunkStep = kRotate ? 8 : T;
  float v[C][8];
  float a = 0.0f;
#pragma unroll
  for (int i = 0; i < C; ++i) {
    const int c = chunk0 + i * kChunkStep;
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (live && c < K8) raw = __ldg(xr + c);
    if constexpr (kRotate) {
      const __half* h = reinterpret_cast<const __half*>(&raw);
#pragma unroll
      for (int j = 0; j < 8; ++j) v[i][j] = __half2float(h[j]);
    } else {
      if (live && c < K8) {
        values8<true>(raw, col, c, v[i]);
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[i][j] = 0.0f;
      }
    }
  }
  if constexpr (kRotate) {
    // all lanes (and, for rows rotated as a whole by more than one warp, all threads) take part in the exchanges
    extern __shared__ float xch_raw[];
    hadamard_rows<C>(v, lane, chunks_per_block, norm, chunks_per_block > 32 * C ? xch_raw : nullptr);
  }
#pragma unroll
  for (int i = 0; i < C; ++i) {
#pragma unroll
    for (int j = 0; j < 8; ++j) a = fmaxf(a, fabsf(v[i][j]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  if constexpr (kWarpsPerRow > 1) {
    if ((tid & 31) == 0) red[tid >> 5] = a;
    __syncthreads();
    const int w0 = (tid / T) * kWarpsPerRow;
#pragma unroll
    for (int w = 0; w < kWarpsPerRow; ++w) a = fmaxf(a, red[w0 + w]);
  }
  if (!live) return;

  const float s = __fdiv_rn(a, 127.5f);
  float f;
  if (kDivide) {
    f = (a == 0.0f) ? 1.0f : s;
  } else {
    f = (a == 0.0f) ? 0.0f : __fdiv_rn(127.5f, a);
  }
  if (t == 0) scale[row] = s;

  uint2* qr = q + row * K8;
#pragma unroll
  for (int i = 0; i < C; ++i) {
    const int c = chunk0 + i * kChunkStep;
    if (c < K8) {
      qr[c] = make_uint2(codes4<kDivide>(v[i][0], v[i][1], v[i][2], v[i][3], f),
                         codes4<kDivide>(v[i][4], v[i][5], v[i][6], v[i][7], f));
    }
  }
}

template <int T, int C, bool kDivide, bool kRotate>
int launch_rows_rot_team(const uint4* xp, int64_t M, int K8, uint2* qp, float* s, int chunks_per_block, float norm,
                         const float4* col, cudaStream_t stream) {
  constexpr int kRowsPerBlock = kThreads / T;
  auto kern = quantize_rows_rot_kernel<T, C, kDivide, kRotate>;
  // rows rotated as a whole by more than one warp exchange through shared memory: 8 C floats per thread
  const int xch_bytes = (kRotate && chunks_per_block > 32 * C) ? kThreads * C * 8 * static_cast<int>(sizeof(float)) : 0;
  if (xch_bytes > 48 * 1024) {
    static PerDeviceOnce once;
    if (const int rc = set_dynamic_smem_once(once, kern, xch_bytes); rc != PQ_OK) return rc;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>((M + kRowsPerBlock - 1) / kRowsPerBlock), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(xch_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (!kDivide && pdl_enabled()) ? 1 : 0;
  return cuda_status(cudaLaunchKernelEx(&cfg, kern, xp, M, K8, qp, s, chunks_per_block, norm, col));
}

// col == nullptr: Eq. 4 rotation; otherwise Eq. 3 column factors.
template <bool kDivide, bool kRotate>
int launch_rows_f32(const void* x, int64_t M, int64_t K, int8_t* q, float* s, const float* col, cudaStream_t stream) {
  const int K8 = static_cast<int>(K / 8);
  if (K8 > 256 * kCached) return PQ_ERR_SHAPE;   // the transformed row has to fit the team's registers
  const int B = hadamard_block_order(K);
  const float norm = 1.0f / sqrtf(static_cast<float>(B));   // both correctly rounded: the value the butterfly is scaled by
  const uint4* xp = static_cast<const uint4*>(x);
  uint2* qp = reinterpret_cast<uint2*>(q);
  const float4* cp = reinterpret_cast<const float4*>(col);
  // the narrowest team that holds the row with four chunks per thread; eight only for the longest rows
  if (K8 <= 32 * 4) return launch_rows_rot_team<32, 4, kDivide, kRotate>(xp, M, K8, qp, s, B / 8, norm, cp, stream);
  if (K8 <= 64 * 4) return launch_rows_rot_team<64, 4, kDivide, kRotate>(xp, M, K8, qp, s, B / 8, norm, cp, stream);
  if (K8 <= 128 * 4) return launch_rows_rot_team<128, 4, kDivide, kRotate>(xp, M, K8, qp, s, B / 8, norm, cp, stream);
  if (K8 <= 256 * 4) return launch_rows_rot_team<256, 4, kDivide, kRotate>(xp, M, K8, qp, s, B / 8, norm, cp, stream);
  return launch_rows_rot_team<256, kCached, kDivide, kRotate>(xp, M, K8, qp, s, B / 8, norm, cp, stream);
}

template <int T, bool kDivide, bool kSmooth>
int launch_rows_team(const uint4* xp, int64_t M, int K8, uint2* qp, float* s, const float4* col, cudaStream_t stream) {
  constexpr int kRowsPerBlock = kThreads / T;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>((M + kRowsPerBlock - 1) / kRowsPerBlock), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (!kDivide && pdl_enabled()) ? 1 : 0;
  return cuda_status(cudaLaunchKernelEx(&cfg, quantize_rows_kernel<T, kDivide, kSmooth>, xp, M, K8, qp, s, col));
}

template <bool kDivide, bool kSmooth>
int launch_rows(const void* x, int64_t M, int64_t K, int8_t* q, float* s, const float* col, cudaStream_t stream) {
  const int K8 = static_cast<int>(K / 8);
  const uint4* xp = static_cast<const uint4*>(x);
  uint2* qp = reinterpret_cast<uint2*>(q);
  const float4* cp = reinterpret_cast<const float4*>(col);
  // The narrowest row team that still keeps the whole row in registers.  (Wider teams for short launches --
  // more loads in flight per row -- were measured and lose: the maximum then crosses warps through shared
  // memory and a block barrier; 2048 x 2048: 4.4 us with 32 threads per row, 5.2 with 128, 7.1 with 256.)
  const int T = K8 <= 32 * kCached ? 32 : (K8 <= 64 * kCached ? 64 : (K8 <= 128 * kCached ? 128 : 256));
  if (T == 32) return launch_rows_team<32, kDivide, kSmooth>(xp, M, K8, qp, s, cp, stream);
  if (T == 64) return launch_rows_team<64, kDivide, kSmooth>(xp, M, K8, qp, s, cp, stream);
  if (T == 128) return launch_rows_team<128, kDivide, kSmooth>(xp, M, K8, qp, s, cp, stream);
  return launch_rows_team<256, kDivide, kSmooth>(xp, M, K8, qp, s, cp, stream);
}

// ---------------------------------------------------------------------------- INT4
// Packed layout of one weight row: K/2 bytes; inside every run of 32 consecutive k
// (16 bytes) byte b holds code(k0 + b) in bits 0-3 and code(k0 + 16 + b) in bits 4-7,
// two's complement.  A 32-bit word w of that run then widens with two logic ops into
// four consecutive INT8 values each:  (w << 4) & 0xF0F0F0F0 -> 16 * code(k0 + 4j .. 4j+3),
// w & 0xF0F0F0F0 -> 16 * code(k0 + 16 + 4j ..).

// One warp per (output channel n, group g of 128 k).  Lane l owns bytes 2*(l%8), 2*(l%8)+1
// of 32-k run l/8, i.e. codes k0+b, k0+b+1, k0+16+b, k0+16+b+1.
// col (nullable): the column factors of Eq. 3; the group maximum and the codes are then those of S W.
__global__ void __launch_bounds__(kThreads) pack_w4_kernel(const __half* __restrict__ w, int64_t N, int K,
                                                           uint8_t* __restrict__ wp,
                                                           __half* __restrict__ s_grp,
                                                           const float* __restrict__ col) {
  const int G = K / 128;
  const int64_t warp = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
  if (warp >= N * G) return;
  const int lane = threadIdx.x & 31;
  const int64_t n = warp / G;
  const int g = static_cast<int>(warp % G);
  const int k0 = g * 128 + (lane >> 3) * 32;
  const int b = (lane & 7) * 2;
  const __half* wr = w + n * K + k0;
  const __half2 lo = *reinterpret_cast<const __half2*>(wr + b);
  const __half2 hi = *reinterpret_cast<const __half2*>(wr + 16 + b);
  float v0 = __low2float(lo), v1 = __high2float(lo), v2 = __low2float(hi), v3 = __high2float(hi);
  if (col != nullptr) {
    v0 = __fmul_rn(v0, __ldg(col + k0 + b));
    v1 = __fmul_rn(v1, __ldg(col + k0 + b + 1));
    v2 = __fmul_rn(v2, __ldg(col + k0 + 16 + b));
    v3 = __fmul_rn(v3, __ldg(col + k0 + 16 + b + 1));
  }
  float a = fmaxf(fmaxf(fabsf(v0), fabsf(v1)), fmaxf(fabsf(v2), fabsf(v3)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  const __half s16 = __float2half_rn(__fdiv_rn(a, 7.5f));
  const float sf = __half2float(s16);
  if (lane == 0) s_grp[static_cast<int64_t>(g) * N + n] = s16;
  auto code4 = [sf](float x) -> uint32_t {
    if (sf == 0.0f) return 0u;
    int r = __float2int_rn(__fdiv_rn(x, sf));
    return static_cast<uint32_t>(max(-8, min(7, r))) & 0xfu;
  };
  const uint32_t byte0 = code4(v0) | (code4(v2) << 4);
  const uint32_t byte1 = code4(v1) | (code4(v3) << 4);
  uint8_t* out = wp + n * (K / 2) + k0 / 2 + b;
  *reinterpret_cast<uint16_t*>(out) = static_cast<uint16_t>(byte0 | (byte1 << 8));
}

// One thread per packed byte -> two row-major INT8 codes in [-8, 7].
__global__ void __launch_bounds__(kThreads) unpack_w4_kernel(const uint8_t* __restrict__ wp, int64_t N, int K,
                                                             int8_t* __restrict__ codes) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  const int K2 = K / 2;
  if (i >= N * K2) return;
  const int64_t n = i / K2;
  const int j = static_cast<int>(i % K2);
  const int k0 = (j / 16) * 32, b = j % 16;
  const uint8_t v = wp[i];
  const int lo = static_cast<int8_t>(v << 4) >> 4;
  const int hi = static_cast<int8_t>(v) >> 4;
  codes[n * K + k0 + b] = static_cast<int8_t>(lo);
  codes[n * K + k0 + 16 + b] = static_cast<int8_t>(hi);
}

// Group-wise INT4 packing of W H (Eq. 4).  One warp per (output channel n, span of 256 k): lane l holds
// k = k0 + 8 l .. + 7, rotates with its block (order 128 or 256: K is a multiple of 128), then the two
// groups of the span (lanes 0-15, 16-31) are quantized like pack_w4_kernel does and the codes are
// exchanged between lanes l and l ^ 2 to form the packed bytes (byte b of a 32-k run = code(b) |
// code(16 + b) << 4).
__global__ void __launch_bounds__(kThreads) pack_w4_rot_kernel(const __half* __restrict__ w, int64_t N, int K,
                                                               uint8_t* __restrict__ wp,
                                                               __half* __restrict__ s_grp, int chunks_per_block,
                                                               float norm) {
  const int spans = (K + 255) / 256;
  const int64_t warp = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
  if (warp >= N * spans) return;
  const int lane = threadIdx.x & 31;
  const int64_t n = warp / spans;
  const int k0 = static_cast<int>(warp % spans) * 256;
  const int k = k0 + 8 * lane;
  const bool inside = k < K;                      // K is a multiple of 128: a half-span is all in or all out
  uint4 raw = make_uint4(0u, 0u, 0u, 0u);
  if (inside) raw = *reinterpret_cast<const uint4*>(w + n * K + k);
  const __half* h = reinterpret_cast<const __half*>(&raw);
  float v[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = __half2float(h[j]);
  hadamard_chunk(v, lane, chunks_per_block, norm);
  float a = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) a = fmaxf(a, fabsf(v[j]));
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));   // over the group's 16 lanes
  const __half s16 = __float2half_rn(__fdiv_rn(a, 7.5f));
  const float sf = __half2float(s16);
  const int G = K / 128;
  if (inside && (lane & 15) == 0) s_grp[static_cast<int64_t>(k / 128) * N + n] = s16;
  uint32_t mine = 0;                               // eight 4-bit codes, code j in bits 4j .. 4j+3
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint32_t c = 0;
    if (sf != 0.0f) {
      const int r = __float2int_rn(__fdiv_rn(v[j], sf));
      c = static_cast<uint32_t>(max(-8, min(7, r))) & 0xfu;
    }
    mine |= c << (4 * j);
  }
  const uint32_t theirs = __shfl_xor_sync(0xffffffffu, mine, 2);
  if (inside && (lane & 2) == 0) {
    // this lane holds positions 8 (l % 4) .. + 7 of its 32-k run, the partner the positions 16 higher
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      lo |= (((mine >> (4 * j)) & 0xfu) | (((theirs >> (4 * j)) & 0xfu) << 4)) << (8 * j);
      hi |= (((mine >> (4 * (j + 4))) & 0xfu) | (((theirs >> (4 * (j + 4))) & 0xfu) << 4)) << (8 * j);
    }
    const int run = lane >> 2;
    uint8_t* out = wp + n * (K / 2) + k0 / 2 + run * 16 + (lane & 1) * 8;
    *reinterpret_cast<uint2*>(out) = make_uint2(lo, hi);
  }
  (void)G;
}

// Group-wise INT4 packing of W H for rows rotated as a whole (K a power of two above 256).  One block per
// output channel: the row is rotated in shared memory in FP32 by the in-place butterfly (distances 1, 2, ...,
// K/2 in this order, each step one rounded sum and one rounded difference), scaled by 1/sqrt(K), and warp w
// quantizes the groups w, w + 8, ... exactly as pack_w4_kernel does.
__global__ void __launch_bounds__(kThreads) pack_w4_rotfull_kernel(const __half* __restrict__ w, int64_t N, int K,
                                                                   uint8_t* __restrict__ wp,
                                                                   __half* __restrict__ s_grp, float norm) {
  extern __shared__ float rot_row[];
  const int64_t n = blockIdx.x;
  const int tid = threadIdx.x;
  for (int k = tid; k < K; k += kThreads) rot_row[k] = __half2float(w[n * K + k]);
  __syncthreads();
  for (int h = 1; h < K; h <<= 1) {
    for (int p = tid; p < K / 2; p += kThreads) {
      const int idx = (p / h) * 2 * h + (p % h);
      const float a = rot_row[idx], b = rot_row[idx + h];
      rot_row[idx] = __fadd_rn(a, b);
      rot_row[idx + h] = __fsub_rn(a, b);
    }
    __syncthreads();
  }
  for (int k = tid; k < K; k += kThreads) rot_row[k] = __fmul_rn(rot_row[k], norm);
  __syncthreads();
  const int lane = tid & 31;
  for (int g = tid >> 5; g < K / 128; g += kThreads / 32) {
    const int k0 = g * 128 + (lane >> 3) * 32;
    const int b = (lane & 7) * 2;
    const float v0 = rot_row[k0 + b], v1 = rot_row[k0 + b + 1], v2 = rot_row[k0 + 16 + b], v3 = rot_row[k0 + 16 + b + 1];
    float a = fmaxf(fmaxf(fabsf(v0), fabsf(v1)), fmaxf(fabsf(v2), fabsf(v3)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    const __half s16 = __float2half_rn(__fdiv_rn(a, 7.5f));
    const float sf = __half2float(s16);
    if (lane == 0) s_grp[static_cast<int64_t>(g) * N + n] = s16;
    auto code4 = [sf](float x) -> uint32_t {
      if (sf == 0.0f) return 0u;
      const int r = __float2int_rn(__fdiv_rn(x, sf));
      return static_cast<uint32_t>(max(-8, min(7, r))) & 0xfu;
    };
    const uint32_t byte0 = code4(v0) | (code4(v2) << 4);
    const uint32_t byte1 = code4(v1) | (code4(v3) << 4);
    uint8_t* out = wp + n * (K / 2) + k0 / 2 + b;
    *reinterpret_cast<uint16_t*>(out) = static_cast<uint16_t>(byte0 | (byte1 << 8));
  }
}

// Launched (plainly, stream-ordered) behind the offline weight kernels.  A GEMM that follows in
// the stream may request weight tiles before its own wait on its predecessor; with this kernel
// in between, that predecessor starts only after the packed weights are complete and visible.
__global__ void pack_fence_kernel() {}

}  // namespace

int launch_pack_fence(cudaStream_t stream) {
  pack_fence_kernel<<<1, 32, 0, stream>>>();
  return cuda_status(cudaGetLastError());
}

int launch_quantize_act(const void* x, int64_t M, int64_t K, int8_t* q, float* s, bool divide_by_scale,
                        const float* col, cudaStream_t stream) {
  if (col != nullptr) {
    if (K / 8 <= 256 * kCached) {
      // the row fits the team's registers as FP32: evaluate x * col[k] once
      return divide_by_scale ? launch_rows_f32<true, false>(x, M, K, q, s, col, stream)
                             : launch_rows_f32<false, false>(x, M, K, q, s, col, stream);
    }
    return divide_by_scale ? launch_rows<true, true>(x, M, K, q, s, col, stream)
                           : launch_rows<false, true>(x, M, K, q, s, col, stream);
  }
  return divide_by_scale ? launch_rows<true, false>(x, M, K, q, s, nullptr, stream)
                         : launch_rows<false, false>(x, M, K, q, s, nullptr, stream);
}

int launch_pack_w4(const void* w, int64_t N, int64_t K, void* wp, void* s_grp, const float* col,
                   cudaStream_t stream) {
  const int64_t warps = N * (K / 128);
  const unsigned blocks = static_cast<unsigned>((warps + kThreads / 32 - 1) / (kThreads / 32));
  pack_w4_kernel<<<blocks, kThreads, 0, stream>>>(static_cast<const __half*>(w), N, static_cast<int>(K),
                                                  static_cast<uint8_t*>(wp), static_cast<__half*>(s_grp), col);
  return cuda_status(cudaGetLastError());
}

int launch_quantize_act_hadamard(const void* x, int64_t M, int64_t K, int8_t* q, float* s, bool divide_by_scale,
                                 cudaStream_t stream) {
  return divide_by_scale ? launch_rows_f32<true, true>(x, M, K, q, s, nullptr, stream)
                         : launch_rows_f32<false, true>(x, M, K, q, s, nullptr, stream);
}

int launch_pack_w4_hadamard(const void* w, int64_t N, int64_t K, void* wp, void* s_grp, cudaStream_t stream) {
  const int B = hadamard_block_order(K);
  const float norm = 1.0f / sqrtf(static_cast<float>(B));
  if (B > 256) {
    // the row is rotated as a whole
    const int smem = static_cast<int>(K) * static_cast<int>(sizeof(float));
    if (smem > 48 * 1024) {
      static PerDeviceOnce once;
      if (const int rc = set_dynamic_smem_once(once, pack_w4_rotfull_kernel, smem > 64 * 1024 ? smem : 64 * 1024); rc != PQ_OK) return rc;
    }
    pack_w4_rotfull_kernel<<<static_cast<unsigned>(N), kThreads, smem, stream>>>(
        static_cast<const __half*>(w), N, static_cast<int>(K), static_cast<uint8_t*>(wp), static_cast<__half*>(s_grp), norm);
    return cuda_status(cudaGetLastError());
  }
  const int64_t warps = N * ((K + 255) / 256);
  const unsigned blocks = static_cast<unsigned>((warps + kThreads / 32 - 1) / (kThreads / 32));
  pack_w4_rot_kernel<<<blocks, kThreads, 0, stream>>>(static_cast<const __half*>(w), N, static_cast<int>(K),
                                                      static_cast<uint8_t*>(wp), static_cast<__half*>(s_grp), B / 8,
                                                      norm);
  return cuda_status(cudaGetLastError());
}

// ---------------------------------------------------------------------------- SwiGLU + per-token quantization
namespace {

// 1 + e^t for t in [-87, 88] as a fixed sequence of binary32 operations (every step a single correctly
// rounded operation, so that the INT8 codes decided by the result are reproducible anywhere):
// t = n ln2 + r with n = rne(t / ln2) and ln2 split into a part with 9 trailing zero bits (n * hi is
// exact) and a remainder, p = e^r by the degree-7 Taylor polynomial in Horner form with fused
// multiply-adds, result fma(p, 2^n, 1).  rne(x) for |x| < 2^22 is taken as (x + 1.5 * 2^23) - 1.5 * 2^23:
// the sum's low mantissa bits are n itself, so 2^n (n in [-126, 127]) is built from them with one
// shift-and-add and no conversion instruction.
__device__ __forceinline__ float one_plus_exp_fixed(float t) {
  const float big = __fadd_rn(__fmul_rn(t, 1.44269502162933349609375f), 12582912.0f);   // 1 / ln 2 rounded to binary32
  const float n = __fadd_rn(big, -12582912.0f);
  float r = __fmaf_rn(n, -0.693145751953125f, t);                       // ln 2, upper part
  r = __fmaf_rn(n, -1.42860676533018704503775e-06f, r);                 // ln 2, lower part
  float p = 1.98412701138295233249664e-04f;                             // 1/7!
  p = __fmaf_rn(p, r, 1.38888892251998186111450e-03f);                  // 1/6!
  p = __fmaf_rn(p, r, 8.33333376795053482055664e-03f);                  // 1/5!
  p = __fmaf_rn(p, r, 4.16666679084300994873047e-02f);                  // 1/4!
  p = __fmaf_rn(p, r, 1.66666671633720397949219e-01f);                  // 1/3!
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  // as_int(big) = 0x4B400000 + n and 0x4B400000 << 23 == 0 (mod 2^32): (n + 127) << 23
  const float two_n = __int_as_float((__float_as_int(big) << 23) + 0x3F800000);
  return __fmaf_rn(p, two_n, 1.0f);
}

// silu(g) * u, silu(g) = g / (1 + e^-g): clamp of the exponent's argument, d = 1 + e^t as above, the
// IEEE reciprocal of d, and two products.  Not rounded back to FP16.
__device__ __forceinline__ float swiglu_fixed(float g, float u) {
  const float t = fminf(fmaxf(-g, -87.0f), 88.0f);
  return __fmul_rn(__fmul_rn(g, __frcp_rn(one_plus_exp_fixed(t))), u);
}

// h = silu(gate) * up for one token row, kept in FP32 registers (I <= 8 * C * T), then the per-token
// quantizer of Eq. 1-2 on h: the MLP's gated activation and the down projection's activation quantizer
// in one pass over the gate/up outputs (4 bytes read, 1 written per element; no FP16 round trip of h).
// About 40 instructions per element (the fixed exponential and the reciprocal) next to 5 bytes of
// traffic: the kernel needs many resident warps, so long rows are spread over 512 threads with three or
// four 16-byte chunks each (<= 64 registers, 32 warps per SM) and all of a thread's loads are issued
// before its first use.
template <int BLOCK, int T, int C>
__global__ void __launch_bounds__(BLOCK, 2048 / BLOCK / 2) swiglu_quantize_kernel(const uint4* __restrict__ gate,
                                                                                const uint4* __restrict__ up, int64_t M,
                                                                                int K8, uint2* __restrict__ q,
                                                                                float* __restrict__ scale) {
  constexpr int kRowsPerBlock = BLOCK / T;
  constexpr int kWarpsPerRow = T / 32;
  __shared__ float red[BLOCK / 32];
  const int tid = threadIdx.x;
  const int t = tid % T;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kRowsPerBlock + tid / T;
  const bool live = row < M;

  grid_dep_launch();
  grid_dep_wait();   // gate and up are the outputs of the preceding GEMM

  uint4 gr[C], ur[C];
#pragma unroll
  for (int i = 0; i < C; ++i) {
    const int c = t + i * T;
    gr[i] = make_uint4(0u, 0u, 0u, 0u);   // silu(0) * 0 = 0: a chunk past the row's end adds nothing to the maximum
    ur[i] = make_uint4(0u, 0u, 0u, 0u);
    if (live && c < K8) {
      gr[i] = __ldg(gate + row * K8 + c);
      ur[i] = __ldg(up + row * K8 + c);
    }
  }
  float v[C][8];
  float a = 0.0f;
#pragma unroll
  for (int i = 0; i < C; ++i) {
    const __half* gh = reinterpret_cast<const __half*>(&gr[i]);
    const __half* uh = reinterpret_cast<const __half*>(&ur[i]);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      v[i][j] = swiglu_fixed(__half2float(gh[j]), __half2float(uh[j]));
      a = fmaxf(a, fabsf(v[i][j]));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  if constexpr (kWarpsPerRow > 1) {
    if ((tid & 31) == 0) red[tid >> 5] = a;
    __syncthreads();
    const int w0 = (tid / T) * kWarpsPerRow;
#pragma unroll
    for (int w = 0; w < kWarpsPerRow; ++w) a = fmaxf(a, red[w0 + w]);
  }
  if (!live) return;
  const float s = __fdiv_rn(a, 127.5f);
  const float f = (a == 0.0f) ? 0.0f : __fdiv_rn(127.5f, a);
  if (t == 0) scale[row] = s;
  uint2* qr = q + row * K8;
#pragma unroll
  for (int i = 0; i < C; ++i) {
    const int c = t + i * T;
    if (c < K8) {
      qr[c] = make_uint2(codes4<false>(v[i][0], v[i][1], v[i][2], v[i][3], f),
                         codes4<false>(v[i][4], v[i][5], v[i][6], v[i][7], f));
    }
  }
}

template <int BLOCK, int T, int C>
int launch_swiglu_team(const void* gate, const void* up, int64_t M, int K8, int8_t* q, float* s, cudaStream_t stream) {
  constexpr int kRowsPerBlock = BLOCK / T;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>((M + kRowsPerBlock - 1) / kRowsPerBlock), 1, 1);
  cfg.blockDim = dim3(BLOCK, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cuda_status(cudaLaunchKernelEx(&cfg, swiglu_quantize_kernel<BLOCK, T, C>, static_cast<const uint4*>(gate),
                                        static_cast<const uint4*>(up), M, K8, reinterpret_cast<uint2*>(q), s));
}

}  // namespace

int launch_swiglu_quantize(const void* gate, const void* up, int64_t M, int64_t I, int8_t* q, float* s_tok,
                           cudaStream_t stream) {
  const int K8 = static_cast<int>(I / 8);
  if (K8 > 512 * 4) return PQ_ERR_SHAPE;   // the row has to fit the team's registers
  // the narrowest team that holds the row with at most four chunks per thread
  if (K8 <= 32 * 4) return launch_swiglu_team<256, 32, 4>(gate, up, M, K8, q, s_tok, stream);
  if (K8 <= 64 * 4) return launch_swiglu_team<256, 64, 4>(gate, up, M, K8, q, s_tok, stream);
  if (K8 <= 128 * 4) return launch_swiglu_team<256, 128, 4>(gate, up, M, K8, q, s_tok, stream);
  if (K8 <= 256 * 3) return launch_swiglu_team<256, 256, 3>(gate, up, M, K8, q, s_tok, stream);
  if (K8 <= 256 * 4) return launch_swiglu_team<256, 256, 4>(gate, up, M, K8, q, s_tok, stream);
  if (K8 <= 512 * 3) return launch_swiglu_team<512, 512, 3>(gate, up, M, K8, q, s_tok, stream);
  return launch_swiglu_team<512, 512, 4>(gate, up, M, K8, q, s_tok, stream);
}

// ---------------------------------------------------------------------------- static activation scale
namespace {

// Eq. 1 against ONE calibrated scale (no maximum pass): a thread owns a 16-byte chunk of 8 elements.
// *s_ptr is the scale; the token scale vector is filled with it so that the GEMMs run unchanged.
__global__ void __launch_bounds__(kThreads) quantize_static_kernel(const uint4* __restrict__ x, int64_t M, int K8,
                                                                   uint2* __restrict__ q, float* __restrict__ s_tok,
                                                                   const float* __restrict__ s_ptr) {
  grid_dep_launch();
  grid_dep_wait();   // x (and possibly the scale) come from the preceding kernel
  const float s = __ldg(s_ptr);
  const float sc = s > 0.0f ? s : 0.0f;
  const float inv = s > 0.0f ? __fdiv_rn(1.0f, s) : 0.0f;
  const int64_t total = M * K8;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * kThreads) {
    q[i] = quantize8<false, false>(__ldg(x + i), inv, nullptr, 0);
    if (i % K8 == 0) s_tok[i / K8] = sc;
  }
}

// The same with one calibrated scale per feature channel, given as reciprocals inv_s[k]: one product per
// element; a reciprocal that is not positive gives code 0.  Token scales are 1 (the channel scales belong
// into the weights).
__global__ void __launch_bounds__(kThreads) quantize_static_channel_kernel(const uint4* __restrict__ x, int64_t M, int K8,
                                                                           uint2* __restrict__ q,
                                                                           float* __restrict__ s_tok,
                                                                           const float4* __restrict__ inv_s) {
  grid_dep_launch();
  grid_dep_wait();
  const int64_t total = M * K8;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * kThreads) {
    const int c = static_cast<int>(i % K8);
    float4 f0 = __ldg(inv_s + 2 * c), f1 = __ldg(inv_s + 2 * c + 1);
    f0.x = fmaxf(f0.x, 0.0f); f0.y = fmaxf(f0.y, 0.0f); f0.z = fmaxf(f0.z, 0.0f); f0.w = fmaxf(f0.w, 0.0f);
    f1.x = fmaxf(f1.x, 0.0f); f1.y = fmaxf(f1.y, 0.0f); f1.z = fmaxf(f1.z, 0.0f); f1.w = fmaxf(f1.w, 0.0f);
    const uint4 v = __ldg(x + i);
    const __half* h = reinterpret_cast<const __half*>(&v);
    q[i] = make_uint2(
        codes4<false>(__fmul_rn(__half2float(h[0]), f0.x), __fmul_rn(__half2float(h[1]), f0.y),
                      __fmul_rn(__half2float(h[2]), f0.z), __fmul_rn(__half2float(h[3]), f0.w), 1.0f),
        codes4<false>(__fmul_rn(__half2float(h[4]), f1.x), __fmul_rn(__half2float(h[5]), f1.y),
                      __fmul_rn(__half2float(h[6]), f1.z), __fmul_rn(__half2float(h[7]), f1.w), 1.0f));
    if (c == 0) s_tok[i / K8] = 1.0f;
  }
}

}  // namespace

int launch_quantize_act_static_channel(const void* x, const float* inv_s, int64_t M, int64_t K, int8_t* q, float* s_tok,
                                       cudaStream_t stream) {
  const int K8 = static_cast<int>(K / 8);
  const int64_t total = M * K8;
  int64_t blocks = (total + kThreads - 1) / kThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 16;
  if (blocks > cap) blocks = cap;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cuda_status(cudaLaunchKernelEx(&cfg, quantize_static_channel_kernel, static_cast<const uint4*>(x), M, K8,
                                        reinterpret_cast<uint2*>(q), s_tok, reinterpret_cast<const float4*>(inv_s)));
}

int launch_quantize_act_static(const void* x, const float* s_ptr, int64_t M, int64_t K, int8_t* q, float* s_tok,
                               cudaStream_t stream) {
  const int K8 = static_cast<int>(K / 8);
  const int64_t total = M * K8;
  int64_t blocks = (total + kThreads - 1) / kThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 16;   // grid-stride beyond a few waves
  if (blocks > cap) blocks = cap;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cuda_status(cudaLaunchKernelEx(&cfg, quantize_static_kernel, static_cast<const uint4*>(x), M, K8,
                                        reinterpret_cast<uint2*>(q), s_tok, s_ptr));
}

// ---------------------------------------------------------------------------- Eq. 3 calibration
namespace {

// Column maxima of |A| for A FP16 [R,K]: a thread owns 8 adjacent columns (one 16-byte chunk) of a
// strip of rows; non-negative floats order like their bit patterns, so strips merge with atomicMax
// on the patterns.  out must be zero when the kernel starts.
constexpr int kStripRows = 64;
__global__ void __launch_bounds__(kThreads) col_absmax_kernel(const uint4* __restrict__ a, int64_t R, int K8,
                                                              unsigned int* __restrict__ out) {
  const int c = blockIdx.x * kThreads + threadIdx.x;
  if (c >= K8) return;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kStripRows;
  const int64_t r1 = r0 + kStripRows < R ? r0 + kStripRows : R;
  __half2 m[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) m[i] = __float2half2_rn(0.0f);
  for (int64_t r = r0; r < r1; ++r) {
    const uint4 v = __ldg(a + r * K8 + c);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) m[i] = __hmax2(m[i], __habs2(h[i]));
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    atomicMax(out + 8 * c + 2 * i, __float_as_uint(__low2float(m[i])));
    atomicMax(out + 8 * c + 2 * i + 1, __float_as_uint(__high2float(m[i])));
  }
}

// Eq. 3 with alpha = 1/2, literally: sqrt(max|X_j|) / sqrt(max|W_j|), and its reciprocal; three and
// one correctly rounded FP32 operations.  A channel with a zero maximum keeps s = 1.
// x^(a/4) for a = 0 ... 4 out of correctly rounded square roots and at most one rounded product.
__device__ __forceinline__ float quarter_power(float x, int a) {
  const float r2 = __fsqrt_rn(x);
  switch (a) {
    case 0: return 1.0f;
    case 1: return __fsqrt_rn(r2);
    case 2: return r2;
    case 3: return __fmul_rn(r2, __fsqrt_rn(r2));
    default: return x;
  }
}

// alpha = a / 4: s = x^alpha / w^(1 - alpha); a = 2 is Eq. 3 as the paper sets it.
__global__ void __launch_bounds__(kThreads) smooth_scales_kernel(const float* __restrict__ xa,
                                                                 const float* __restrict__ wa, int64_t K, int a,
                                                                 float* __restrict__ s, float* __restrict__ s_inv) {
  const int64_t k = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  if (k >= K) return;
  const float x = xa[k], w = wa[k];
  float sv = 1.0f, si = 1.0f;
  if (x > 0.0f && w > 0.0f) {
    sv = __fdiv_rn(quarter_power(x, a), quarter_power(w, 4 - a));
    si = __fdiv_rn(1.0f, sv);
  }
  s[k] = sv;
  s_inv[k] = si;
}

}  // namespace

int launch_col_absmax(const void* a, int64_t R, int64_t K, float* out, cudaStream_t stream) {
  if (cudaMemsetAsync(out, 0, static_cast<size_t>(K) * sizeof(float), stream) != cudaSuccess) return PQ_ERR_CUDA;
  const int K8 = static_cast<int>(K / 8);
  const dim3 grid(static_cast<unsigned>((K8 + kThreads - 1) / kThreads),
                  static_cast<unsigned>((R + kStripRows - 1) / kStripRows), 1);
  col_absmax_kernel<<<grid, kThreads, 0, stream>>>(static_cast<const uint4*>(a), R, K8,
                                                   reinterpret_cast<unsigned int*>(out));
  return cuda_status(cudaGetLastError());
}

int launch_smooth_scales(const float* xa, const float* wa, int64_t K, int alpha_quarters, float* s, float* s_inv,
                         cudaStream_t stream) {
  const unsigned blocks = static_cast<unsigned>((K + kThreads - 1) / kThreads);
  smooth_scales_kernel<<<blocks, kThreads, 0, stream>>>(xa, wa, K, alpha_quarters, s, s_inv);
  return cuda_status(cudaGetLastError());
}

int launch_unpack_w4(const void* wp, int64_t N, int64_t K, int8_t* codes, cudaStream_t stream) {
  const int64_t n = N * (K / 2);
  const unsigned blocks = static_cast<unsigned>((n + kThreads - 1) / kThreads);
  unpack_w4_kernel<<<blocks, kThreads, 0, stream>>>(static_cast<const uint8_t*>(wp), N, static_cast<int>(K), codes);
  return cuda_status(cudaGetLastError());
}

}  // namespace pq
