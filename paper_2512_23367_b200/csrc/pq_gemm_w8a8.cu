// W8A8 prefill GEMM for sm_100a:  ACC = Q * Wq^T in INT32 on the 5th-generation tensor
// cores (tcgen05.mma kind::i8), fused dequantization  Y = fp16(float(ACC) * s_tok[m] * s_ch[n]).
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: 128-byte-swizzled Q and Wq tiles -> shared-memory ring
//   warp 1      MMA issuer (one elected thread): 128 x BN x 32 INT8 steps into a TMEM
//               accumulator; two accumulators so tile i's epilogue overlaps tile i+1's main loop
//   warps 2-5   epilogue: tcgen05.ld INT32 -> FP32 x token scale x channel scale -> FP16 stores
// Ragged M, N and K need no special main-loop code: TMA fills out-of-range bytes with zeros
// (which add nothing to an integer dot product) and the epilogue predicates its stores.
#include <cuda_fp16.h>

#include <cstdlib>

#include "pq_internal.h"
#include "pq_ptx.cuh"

namespace pq {
namespace {

constexpr int BM = 128;   // rows of Q per tile (= TMEM lanes)
constexpr int BK = 128;   // K bytes per pipeline stage (= one 128-byte swizzle row)
constexpr int UMMA_K = 32;
constexpr int kNumThreads = 192;
constexpr int kEpilogueThreads = 128;

struct GemmArgs {
  const float* s_tok;
  const float* s_ch;
  __half* y;
  int32_t* acc;
  int* status;
  int M, N, K;
  int m_blocks, n_blocks, k_blocks;
};

template <int BN, int STAGES>
struct Smem {
  static constexpr int kABytes = BM * BK;
  static constexpr int kBBytes = BN * BK;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kScaleOff = STAGES * kStageBytes;            // BN floats per epilogue warp
  static constexpr int kBarOff = kScaleOff + 4 * BN * 4;            // barriers (8 B each)
  static constexpr int kNumBars = 2 * STAGES + 4;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;           // tmem base, abort flag
  static constexpr int kTotal = kMiscOff + 16;
  static constexpr int kDynamic = kTotal + 1024;                    // slack for 1024-B alignment
};

template <int BN, int STAGES, bool kExportAcc>
__global__ void __launch_bounds__(kNumThreads, 1)
gemm_w8a8_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_w,
                 const GemmArgs p) {
  using L = Smem<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  float* s_ch_smem = reinterpret_cast<float*>(smem + L::kScaleOff);
  const uint32_t bar_full = smem_base + L::kBarOff;
  const uint32_t bar_empty = bar_full + STAGES * 8;
  const uint32_t bar_tfull = bar_empty + STAGES * 8;
  const uint32_t bar_tempty = bar_tfull + 2 * 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.m_blocks * p.n_blocks;
  constexpr uint32_t kTmemCols = 2 * BN;  // 256 or 512: a power of two

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + s * 8, 1);
      mbar_init(bar_empty + s * 8, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + b * 8, 1);
      mbar_init(bar_tempty + b * 8, kEpilogueThreads / 32);
    }
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_w);
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
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_empty + s * 8, ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t a_dst = smem_base + s * L::kStageBytes;
          mbar_arrive_expect_tx(bar_full + s * 8, L::kStageBytes);
          tma_load_2d(a_dst, &tm_q, bar_full + s * 8, kb * BK, m0);
          tma_load_2d(a_dst + L::kABytes, &tm_w, bar_full + s * 8, kb * BK, n0);
        }
      }
      if (!ok) {
        // Giving up: let the loads already issued land before the CTA may exit.
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
      uint32_t it = 0, t = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
        const uint32_t b = t & 1u;
        if (!mbar_wait(bar_tempty + b * 8, ((t >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + b * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_full + s * 8, ph, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_base + s * L::kStageBytes;
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + L::kABytes);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing K by 32 bytes inside the swizzled 128-byte row: +2 in 16-byte units
            umma_i8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
          }
          umma_commit(bar_empty + s * 8);  // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(bar_tfull + b * 8);  // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;           // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
    float* sc_warp = s_ch_smem + (warp - 2) * BN;  // this warp's own copy of the tile's channel scales
    uint32_t t = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
      const uint32_t b = t & 1u;
      const int m0 = (tile % p.m_blocks) * BM;
      const int n0 = (tile / p.m_blocks) * BN;
      const int row = m0 + quad * 32 + lane;
      float st = 0.0f;
      if constexpr (!kExportAcc) {
        __syncwarp();  // the previous tile's reads of sc_warp are done
        for (int c = lane; c < BN; c += 32) sc_warp[c] = (n0 + c < p.N) ? __ldg(p.s_ch + n0 + c) : 0.0f;
        if (row < p.M) st = __ldg(p.s_tok + row);
        __syncwarp();
      }
      // one decision for the whole warp: the loop below holds warp-collective instructions
      ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + b * 8, (t >> 1) & 1u, abort_flag));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + b * BN;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32(t_addr + c0, r);
        tmem_ld_wait();
        if (row < p.M) {
          if constexpr (kExportAcc) {
            int32_t* dst = p.acc + static_cast<int64_t>(row) * p.N + n0 + c0;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              if (n0 + c0 + j < p.N)
                *reinterpret_cast<uint4*>(dst + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
            }
          } else {
            const float* sc = sc_warp + c0;
            __half* dst = p.y + static_cast<int64_t>(row) * p.N + n0 + c0;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              if (n0 + c0 + j < p.N) {
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const float2 s2 = *reinterpret_cast<const float2*>(sc + j + 2 * i);
                  const float v0 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int32_t>(r[j + 2 * i])), st), s2.x);
                  const float v1 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int32_t>(r[j + 2 * i + 1])), st), s2.y);
                  const __half2 h = __floats2half2_rn(v0, v1);
                  o[i] = *reinterpret_cast<const uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(dst + j) = make_uint4(o[0], o[1], o[2], o[3]);
              }
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + b * 8);
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

template <int BN, int STAGES, bool kExportAcc>
int launch_cfg(const CUtensorMap& tq, const CUtensorMap& tw, const GemmArgs& a, cudaStream_t stream) {
  using L = Smem<BN, STAGES>;
  auto kern = gemm_w8a8_kernel<BN, STAGES, kExportAcc>;
  static bool configured = false;  // attribute is per function; setting it repeatedly is harmless
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic) != cudaSuccess)
      return PQ_ERR_CUDA;
    configured = true;
  }
  const int tiles = a.m_blocks * a.n_blocks;
  const int grid = tiles < sm_count() ? tiles : sm_count();
  kern<<<grid, kNumThreads, L::kDynamic, stream>>>(tq, tw, a);
  return cuda_status(cudaGetLastError());
}

}  // namespace

int launch_gemm_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M,
                     int64_t N, int64_t K, void* y, int32_t* acc, cudaStream_t stream) {
  // Tile width.  The main loop is bound by the bytes each SM pulls from L2 per multiply-add
  // (48 KB per 128x256x128 step against 32 KB per 128x128x128 step), so the cost of a
  // configuration is (waves of tiles over the SMs) x (bytes per tile step).
  const int sms = sm_count();
  const int64_t mb = (M + BM - 1) / BM;
  const int64_t t256 = mb * ((N + 255) / 256), t128 = mb * ((N + 127) / 128);
  auto waves = [sms](int64_t tiles) { return (tiles + sms - 1) / sms; };
  bool use128 = (N <= 128) || (waves(t128) * 32 < waves(t256) * 48);
  if (const char* e = getenv("PQ_W8A8_BN")) {  // ablation knob: force the tile width
    if (e[0] == '1') use128 = true;
    if (e[0] == '2') use128 = false;
  }
  const int BN = use128 ? 128 : 256;

  CUtensorMap tq, tw;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), BM, BK, 1, 128);
  if (rc != PQ_OK) return rc;
  rc = make_tmap_2d(&tw, wq, static_cast<uint64_t>(N), static_cast<uint64_t>(K), static_cast<uint32_t>(BN), BK, 1, 128);
  if (rc != PQ_OK) return rc;

  GemmArgs a;
  a.s_tok = s_tok;
  a.s_ch = s_ch;
  a.y = static_cast<__half*>(y);
  a.acc = acc;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.N = static_cast<int>(N);
  a.K = static_cast<int>(K);
  a.m_blocks = static_cast<int>(mb);
  a.n_blocks = static_cast<int>((N + BN - 1) / BN);
  a.k_blocks = static_cast<int>((K + BK - 1) / BK);
  if (acc != nullptr) {
    return use128 ? launch_cfg<128, 6, true>(tq, tw, a, stream) : launch_cfg<256, 4, true>(tq, tw, a, stream);
  }
  return use128 ? launch_cfg<128, 6, false>(tq, tw, a, stream) : launch_cfg<256, 4, false>(tq, tw, a, stream);
}

}  // namespace pq
