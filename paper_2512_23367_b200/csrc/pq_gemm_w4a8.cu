// W4A8 prefill GEMM for sm_100a.  Packed INT4 weights are widened to INT8 inside the kernel,
// multiplied with the INT8 activation codes on the tensor cores one K-group (128) at a time,
// and every group's INT32 accumulator is dequantized with its own scale into an FP32 running
// sum:   R[m,n] += float(ACC_g[m,n]) * s_grp[g,n];   Y = fp16(R * s_tok[m]).
//
// Warp roles of the persistent CTA (one per SM, tile 128 x 128):
//   warp 0      TMA producer: Q tile (128-byte swizzle), packed weight tile and the group's
//               FP16 scales -> stage ring
//   warp 1      MMA issuer: four 128x128x32 kind::i8 steps per group into a ring of four
//               TMEM accumulators (a fresh accumulator per group)
//   warps 2-3   unpack: nibbles -> INT8 (as 16 x code, two logic ops per four codes) written in
//               the swizzled K-major layout the MMA reads; scales -> FP32 (x 1/16)
//   warps 4-7   promotion/epilogue: tcgen05.ld, INT32 -> FP32, FMA with the group scale into
//               128 running sums per thread; after the last group x token scale -> FP16 store
// The widened weights are 16 x code (the nibble sits in the high half of the byte, which keeps
// two's complement without sign-extension work); 1/16 is folded into the FP32 scale, exactly.
#include <cuda_fp16.h>

#include "pq_internal.h"
#include "pq_ptx.cuh"

namespace pq {
namespace {

constexpr int BM = 128, BN = 128, BK = 128, UMMA_K = 32;
constexpr int STAGES = 5;       // Q + packed-weight + scale stages
constexpr int B8_SLOTS = 3;     // widened weight tiles
constexpr int SC_SLOTS = 6;     // FP32 scale rows
constexpr int ACC_SLOTS = 4;    // TMEM accumulators of BN columns
constexpr int kNumThreads = 256;
constexpr int kUnpackThreads = 64;

constexpr int kABytes = BM * BK;          // 16 KB
constexpr int kPBytes = BN * BK / 2;      // 8 KB packed
constexpr int kSBytes = BN * 2;           // FP16 scales of one group
constexpr int kStageBytes = kABytes + kPBytes + 1024;  // scales padded to keep 1024-B alignment
constexpr int kTxBytes = kABytes + kPBytes + kSBytes;
constexpr int kB8Bytes = BN * BK;         // 16 KB
constexpr int kB8Off = STAGES * kStageBytes;
constexpr int kScOff = kB8Off + B8_SLOTS * kB8Bytes;
constexpr int kBarOff = kScOff + SC_SLOTS * BN * 4;
constexpr int kNumBars = 2 * STAGES + 2 * B8_SLOTS + 2 * SC_SLOTS + 2 * ACC_SLOTS;
constexpr int kMiscOff = kBarOff + kNumBars * 8;
constexpr int kDynamicSmem = kMiscOff + 16 + 1024;

struct W4Args {
  const float* s_tok;
  __half* y;
  int32_t* acc_g;  // [G, M, N] when exporting
  int* status;
  int M, N, K;
  int m_blocks, n_blocks, k_blocks;
};

template <bool kExportAcc>
__global__ void __launch_bounds__(kNumThreads, 1)
gemm_w4a8_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_w,
                 const __grid_constant__ CUtensorMap tm_s, const W4Args p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_full = smem_base + kBarOff;            // stage landed (TMA bytes)
  const uint32_t bar_empty = bar_full + STAGES * 8;         // stage free: MMA read Q + unpack read weights
  const uint32_t bar_b8_full = bar_empty + STAGES * 8;      // widened tile written
  const uint32_t bar_b8_empty = bar_b8_full + B8_SLOTS * 8; // MMA finished reading it
  const uint32_t bar_sc_full = bar_b8_empty + B8_SLOTS * 8; // FP32 scales written
  const uint32_t bar_sc_empty = bar_sc_full + SC_SLOTS * 8; // promotion warps read them
  const uint32_t bar_acc_full = bar_sc_empty + SC_SLOTS * 8;
  const uint32_t bar_acc_empty = bar_acc_full + ACC_SLOTS * 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kMiscOff + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.m_blocks * p.n_blocks;
  constexpr uint32_t kTmemCols = ACC_SLOTS * BN;  // 512

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + s * 8, 1);
      mbar_init(bar_empty + s * 8, 1 + kUnpackThreads / 32);
    }
    for (int s = 0; s < B8_SLOTS; ++s) {
      mbar_init(bar_b8_full + s * 8, kUnpackThreads / 32);
      mbar_init(bar_b8_empty + s * 8, 1);
    }
    for (int s = 0; s < SC_SLOTS; ++s) {
      mbar_init(bar_sc_full + s * 8, kUnpackThreads / 32);
      mbar_init(bar_sc_empty + s * 8, 4);
    }
    for (int s = 0; s < ACC_SLOTS; ++s) {
      mbar_init(bar_acc_full + s * 8, 1);
      mbar_init(bar_acc_empty + s * 8, 4);
    }
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_w);
    tma_prefetch_desc(&tm_s);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % p.m_blocks) * BM;
        const int n0 = (tile / p.m_blocks) * BN;
        for (int g = 0; g < p.k_blocks; ++g, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_empty + s * 8, ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = smem_base + s * kStageBytes;
          mbar_arrive_expect_tx(bar_full + s * 8, kTxBytes);
          tma_load_2d(dst, &tm_q, bar_full + s * 8, g * BK, m0);
          tma_load_2d(dst + kABytes, &tm_w, bar_full + s * 8, g * (BK / 2), n0);
          tma_load_2d(dst + kABytes + kPBytes, &tm_s, bar_full + s * 8, n0, g);
        }
      }
      if (!ok) {
        const uint32_t first = it >= static_cast<uint32_t>(STAGES) ? it - STAGES : 0u;
        for (uint32_t j = first; j < it; ++j) {
          const uint32_t s = j % STAGES, ph = (j / STAGES) & 1u;
          for (uint32_t i = 0; i < (1u << 16) && !mbar_try_wait(bar_full + s * 8, ph); ++i) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_s8(BM, BN);
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        for (int g = 0; g < p.k_blocks; ++g, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          const uint32_t u = it % B8_SLOTS, uph = (it / B8_SLOTS) & 1u;
          const uint32_t a = it % ACC_SLOTS, aph = (it / ACC_SLOTS) & 1u;
          if (!mbar_wait(bar_acc_empty + a * 8, aph ^ 1u, abort_flag) ||
              !mbar_wait(bar_full + s * 8, ph, abort_flag) ||
              !mbar_wait(bar_b8_full + u * 8, uph, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          const uint64_t a_desc = umma_desc_k_sw128(smem_base + s * kStageBytes);
          const uint64_t b_desc = umma_desc_k_sw128(smem_base + kB8Off + u * kB8Bytes);
          const uint32_t d_tmem = tmem_base + a * BN;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) umma_i8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0);
          umma_commit(bar_empty + s * 8);
          umma_commit(bar_b8_empty + u * 8);
          umma_commit(bar_acc_full + a * 8);
        }
      }
    }
  } else if (warp < 4) {
    // ------------------------------------------------------------ unpack (warps 2, 3)
    const int ut = threadIdx.x - 64;  // 0..63
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      for (int g = 0; g < p.k_blocks; ++g, ++it) {
        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
        const uint32_t u = it % B8_SLOTS, uph = (it / B8_SLOTS) & 1u;
        const uint32_t v = it % SC_SLOTS, vph = (it / SC_SLOTS) & 1u;
        bool w = mbar_wait(bar_full + s * 8, ph, abort_flag);
        w = w && mbar_wait(bar_b8_empty + u * 8, uph ^ 1u, abort_flag);
        w = w && mbar_wait(bar_sc_empty + v * 8, vph ^ 1u, abort_flag);
        ok = __all_sync(0xffffffffu, w);
        if (!ok) break;
        const uint8_t* stage = smem + s * kStageBytes;
        const uint4* packed = reinterpret_cast<const uint4*>(stage + kABytes);
        uint8_t* b8 = smem + kB8Off + u * kB8Bytes;
#pragma unroll
        for (int i = 0; i < (BN * 4) / kUnpackThreads; ++i) {
          const int idx = ut + i * kUnpackThreads;
          const int r = idx >> 2, j = idx & 3;  // weight row in the tile, 32-k run of the group
          const uint4 w4 = packed[idx];
          uint4 lo, hi;
          lo.x = (w4.x << 4) & 0xF0F0F0F0u; hi.x = w4.x & 0xF0F0F0F0u;
          lo.y = (w4.y << 4) & 0xF0F0F0F0u; hi.y = w4.y & 0xF0F0F0F0u;
          lo.z = (w4.z << 4) & 0xF0F0F0F0u; hi.z = w4.z & 0xF0F0F0F0u;
          lo.w = (w4.w << 4) & 0xF0F0F0F0u; hi.w = w4.w & 0xF0F0F0F0u;
          uint8_t* row = b8 + r * 128;
          const int sw = r & 7;  // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
          *reinterpret_cast<uint4*>(row + (((2 * j) ^ sw) << 4)) = lo;       // k = 32j .. 32j+15
          *reinterpret_cast<uint4*>(row + (((2 * j + 1) ^ sw) << 4)) = hi;   // k = 32j+16 .. 32j+31
        }
        const __half* sh = reinterpret_cast<const __half*>(stage + kABytes + kPBytes);
        float* sc = reinterpret_cast<float*>(smem + kScOff) + v * BN;
        for (int c = ut; c < BN; c += kUnpackThreads) sc[c] = __half2float(sh[c]) * 0.0625f;
        fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor-core (async) proxy
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_b8_full + u * 8);
          mbar_arrive(bar_sc_full + v * 8);
          mbar_arrive(bar_empty + s * 8);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ promotion + epilogue (warps 4..7)
    const int quad = warp & 3;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile % p.m_blocks) * BM;
      const int n0 = (tile / p.m_blocks) * BN;
      const int row = m0 + quad * 32 + lane;
      float R[BN];
#pragma unroll
      for (int j = 0; j < BN; ++j) R[j] = 0.0f;
      for (int g = 0; g < p.k_blocks; ++g, ++it) {
        const uint32_t a = it % ACC_SLOTS, aph = (it / ACC_SLOTS) & 1u;
        const uint32_t v = it % SC_SLOTS, vph = (it / SC_SLOTS) & 1u;
        bool w = mbar_wait(bar_acc_full + a * 8, aph, abort_flag);
        w = w && mbar_wait(bar_sc_full + v * 8, vph, abort_flag);
        ok = __all_sync(0xffffffffu, w);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + a * BN;
        const float* sc = reinterpret_cast<const float*>(smem + kScOff) + v * BN;
#pragma unroll
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t r[32];
          tmem_ld_32x32(t_addr + c0, r);
          tmem_ld_wait();
          if constexpr (kExportAcc) {
            if (row < p.M) {
              int32_t* dst = p.acc_g + (static_cast<int64_t>(g) * p.M + row) * p.N + n0 + c0;
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                if (n0 + c0 + j < p.N) {
                  *reinterpret_cast<int4*>(dst + j) =
                      make_int4(static_cast<int32_t>(r[j]) >> 4, static_cast<int32_t>(r[j + 1]) >> 4,
                                static_cast<int32_t>(r[j + 2]) >> 4, static_cast<int32_t>(r[j + 3]) >> 4);
                }
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 s4 = *reinterpret_cast<const float4*>(sc + c0 + j);
              R[c0 + j + 0] = fmaf(__int2float_rn(static_cast<int32_t>(r[j + 0])), s4.x, R[c0 + j + 0]);
              R[c0 + j + 1] = fmaf(__int2float_rn(static_cast<int32_t>(r[j + 1])), s4.y, R[c0 + j + 1]);
              R[c0 + j + 2] = fmaf(__int2float_rn(static_cast<int32_t>(r[j + 2])), s4.z, R[c0 + j + 2]);
              R[c0 + j + 3] = fmaf(__int2float_rn(static_cast<int32_t>(r[j + 3])), s4.w, R[c0 + j + 3]);
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_acc_empty + a * 8);
          mbar_arrive(bar_sc_empty + v * 8);
        }
      }
      if constexpr (!kExportAcc) {
        if (ok && row < p.M) {
          const float st = __ldg(p.s_tok + row);
          __half* dst = p.y + static_cast<int64_t>(row) * p.N + n0;
#pragma unroll
          for (int j = 0; j < BN; j += 8) {
            if (n0 + j < p.N) {
              uint32_t o[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const __half2 h = __floats2half2_rn(R[j + 2 * i] * st, R[j + 2 * i + 1] * st);
                o[i] = *reinterpret_cast<const uint32_t*>(&h);
              }
              *reinterpret_cast<uint4*>(dst + j) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
        }
      }
    }
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, static_cast<int>(PQ_ERR_TIMEOUT));
}

template <bool kExportAcc>
int launch_w4(const CUtensorMap& tq, const CUtensorMap& tw, const CUtensorMap& ts, const W4Args& a,
              cudaStream_t stream) {
  auto kern = gemm_w4a8_kernel<kExportAcc>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynamicSmem) != cudaSuccess)
      return PQ_ERR_CUDA;
    configured = true;
  }
  const int tiles = a.m_blocks * a.n_blocks;
  const int grid = tiles < sm_count() ? tiles : sm_count();
  kern<<<grid, kNumThreads, kDynamicSmem, stream>>>(tq, tw, ts, a);
  return cuda_status(cudaGetLastError());
}

}  // namespace

int launch_gemm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M,
                     int64_t N, int64_t K, void* y, int32_t* acc_g, cudaStream_t stream) {
  CUtensorMap tq, tw, ts;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), BM, BK, 1, 128);
  if (rc != PQ_OK) return rc;
  rc = make_tmap_2d(&tw, wp, static_cast<uint64_t>(N), static_cast<uint64_t>(K / 2), BN, BK / 2, 1, 0);
  if (rc != PQ_OK) return rc;
  // Group scales [K/128, N] FP16; the accumulator-export variant has none and reads a dummy map of Q.
  if (s_grp != nullptr) {
    rc = make_tmap_2d(&ts, s_grp, static_cast<uint64_t>(K / 128), static_cast<uint64_t>(N), 1, BN, 2, 0);
  } else {
    rc = make_tmap_2d(&ts, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K / 2), 1, BN, 2, 0);
  }
  if (rc != PQ_OK) return rc;
  W4Args a;
  a.s_tok = s_tok;
  a.y = static_cast<__half*>(y);
  a.acc_g = acc_g;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.N = static_cast<int>(N);
  a.K = static_cast<int>(K);
  a.m_blocks = static_cast<int>((M + BM - 1) / BM);
  a.n_blocks = static_cast<int>((N + BN - 1) / BN);
  a.k_blocks = static_cast<int>(K / BK);
  return acc_g != nullptr ? launch_w4<true>(tq, tw, ts, a, stream) : launch_w4<false>(tq, tw, ts, a, stream);
}

}  // namespace pq
