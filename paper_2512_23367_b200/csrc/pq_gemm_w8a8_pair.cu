// W8A8 prefill GEMM on CTA pairs (tcgen05 cta_group::2) for sm_100a.
//
// The single-CTA kernel is bound by the bytes every SM pulls from L2 per multiply-add.  Here
// two CTAs of a cluster share one 256 x BN output tile: each loads its own 128 rows of Q and
// only HALF of the weight tile (BN/2 rows); one tcgen05.mma issued by the leader CTA reads both
// halves from the two CTAs' shared memory and writes each CTA's 128 x BN accumulator into that
// CTA's tensor memory.  Per 128 x 256 x 128 step a CTA now loads 32 KB instead of 48 KB, and the
// smaller stages allow a six-deep ring.
//
// Roles per CTA (192 threads): warp 0 TMA producer (its loads are counted on the LEADER's
// barrier), warp 1 MMA issuer (leader CTA only; also owns TMEM allocation in both CTAs),
// warps 2-5 epilogue (tcgen05.ld -> x token scale x channel scale -> FP16 stores) for the CTA's
// own 128 rows.  Two TMEM accumulators overlap tile i's epilogue with tile i+1's main loop.
#include <cuda_fp16.h>

#include <cstdlib>

#include "pq_internal.h"
#include "pq_ptx.cuh"

namespace pq {
namespace {

constexpr int BM_CTA = 128;       // rows of Q per CTA
constexpr int BM_PAIR = 256;      // rows of Q per tile
constexpr int BK = 128;
constexpr int UMMA_K = 32;
constexpr int kNumThreads = 192;

struct PairArgs {
  const float* s_tok;
  const float* s_ch;
  __half* y;
  int32_t* acc;
  int* status;
  int M, N, K;
  int m_blocks, n_blocks, k_blocks;
};

template <int BN, int STAGES>
struct PairSmem {
  static constexpr int kABytes = BM_CTA * BK;
  static constexpr int kBBytes = (BN / 2) * BK;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kScaleOff = STAGES * kStageBytes;   // BN floats per epilogue warp
  static constexpr int kBarOff = kScaleOff + 4 * BN * 4;
  static constexpr int kNumBars = 2 * STAGES + 4;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kDynamic = kMiscOff + 16 + 1024;
};

template <int BN, int STAGES, bool kExportAcc>
__global__ void __launch_bounds__(kNumThreads, 1)
gemm_w8a8_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_w,
                      const PairArgs p) {
  using L = PairSmem<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  float* s_ch_smem = reinterpret_cast<float*>(smem + L::kScaleOff);
  const uint32_t bar_full = smem_base + L::kBarOff;     // used in the leader: both CTAs' loads landed
  const uint32_t bar_empty = bar_full + STAGES * 8;     // per CTA: the pair's MMAs released the stage
  const uint32_t bar_tfull = bar_empty + STAGES * 8;    // per CTA: accumulator complete
  const uint32_t bar_tempty = bar_tfull + 2 * 8;        // used in the leader: both epilogues drained it
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();              // 0 = leader, 1 = peer
  const int pair_id = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;
  const int num_tiles = p.m_blocks * p.n_blocks;
  constexpr uint32_t kTmemCols = 2 * BN;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + s * 8, 1);    // the leader's producer posts the byte count of BOTH CTAs
      mbar_init(bar_empty + s * 8, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + b * 8, 1);
      mbar_init(bar_tempty + b * 8, 8);  // four epilogue warps in each CTA
    }
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_w);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      const uint32_t full0 = mapa_u32(bar_full, 0);  // the leader's ring of "stage landed" barriers
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
        const int m0 = (tile % p.m_blocks) * BM_PAIR + static_cast<int>(rank) * BM_CTA;
        const int n0 = (tile / p.m_blocks) * BN + static_cast<int>(rank) * (BN / 2);
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_empty + s * 8, ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = smem_base + s * L::kStageBytes;
          // Only the leader arrives (plain CTA-scope arrive; a cluster-scope release per K block
          // would serialise the ring).  The peer's bytes may land first: the transaction count
          // then runs negative until the leader's expect_tx, which is allowed.
          if (rank == 0) mbar_arrive_expect_tx(bar_full + s * 8, 2 * L::kStageBytes);
          tma_load_2d_pair(dst, &tm_q, full0 + s * 8, kb * BK, m0);
          tma_load_2d_pair(dst + L::kABytes, &tm_w, full0 + s * 8, kb * BK, n0);
        }
      }
      (void)ok;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_s8(BM_PAIR, BN);
      uint32_t it = 0, t = 0;
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs, ++t) {
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
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_i8_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
          umma_commit_pair_mcast(bar_empty + s * 8, 0x3);   // frees the stage in both CTAs
        }
        if (ok) umma_commit_pair_mcast(bar_tfull + b * 8, 0x3);  // accumulator ready in both CTAs
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int quad = warp & 3;
    float* sc_warp = s_ch_smem + (warp - 2) * BN;
    const uint32_t tempty0 = mapa_u32(bar_tempty, 0);
    uint32_t t = 0;
    bool ok = true;
    for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs, ++t) {
      const uint32_t b = t & 1u;
      const int m0 = (tile % p.m_blocks) * BM_PAIR + static_cast<int>(rank) * BM_CTA;
      const int n0 = (tile / p.m_blocks) * BN;
      const int row = m0 + quad * 32 + lane;
      float st = 0.0f;
      if constexpr (!kExportAcc) {
        __syncwarp();
        for (int c = lane; c < BN; c += 32) sc_warp[c] = (n0 + c < p.N) ? __ldg(p.s_ch + n0 + c) : 0.0f;
        if (row < p.M) st = __ldg(p.s_tok + row);
        __syncwarp();
      }
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
      if (lane == 0) mbar_arrive_cluster_addr(tempty0 + b * 8);
    }
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();  // neither CTA leaves while its peer may still signal or read it
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, static_cast<int>(PQ_ERR_TIMEOUT));
}

template <int BN, int STAGES, bool kExportAcc>
int launch_pair_cfg(const CUtensorMap& tq, const CUtensorMap& tw, const PairArgs& a, cudaStream_t stream) {
  using L = PairSmem<BN, STAGES>;
  auto kern = gemm_w8a8_pair_kernel<BN, STAGES, kExportAcc>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic) != cudaSuccess)
      return PQ_ERR_CUDA;
    configured = true;
  }
  const int tiles = a.m_blocks * a.n_blocks;
  const int max_pairs = sm_count() / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs), 1, 1);
  cfg.blockDim = dim3(kNumThreads, 1, 1);
  cfg.dynamicSmemBytes = L::kDynamic;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cuda_status(cudaLaunchKernelEx(&cfg, kern, tq, tw, a));
}

}  // namespace

int launch_gemm_w8a8_pair(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M,
                          int64_t N, int64_t K, void* y, int32_t* acc, cudaStream_t stream) {
  // Tile width by the same cost model as the single-CTA kernel: waves of pair tiles over the
  // SM pairs x bytes a CTA loads per K block (16 KB of Q + BN/2 rows of weights).
  const int pairs = sm_count() / 2;
  const int64_t mb = (M + BM_PAIR - 1) / BM_PAIR;
  const int64_t t256 = mb * ((N + 255) / 256), t128 = mb * ((N + 127) / 128);
  auto waves = [pairs](int64_t tiles) { return (tiles + pairs - 1) / pairs; };
  bool use128 = (N <= 128) || (waves(t128) * 24 < waves(t256) * 32);
  if (const char* e = getenv("PQ_W8A8_BN")) {  // ablation knob: force the tile width
    if (e[0] == '1') use128 = true;
    if (e[0] == '2') use128 = false;
  }
  const int BN = use128 ? 128 : 256;

  CUtensorMap tq, tw;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), BM_CTA, BK, 1, true);
  if (rc != PQ_OK) return rc;
  rc = make_tmap_2d(&tw, wq, static_cast<uint64_t>(N), static_cast<uint64_t>(K), static_cast<uint32_t>(BN / 2), BK, 1, true);
  if (rc != PQ_OK) return rc;

  PairArgs a;
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
    return use128 ? launch_pair_cfg<128, 8, true>(tq, tw, a, stream) : launch_pair_cfg<256, 6, true>(tq, tw, a, stream);
  }
  return use128 ? launch_pair_cfg<128, 8, false>(tq, tw, a, stream) : launch_pair_cfg<256, 6, false>(tq, tw, a, stream);
}

}  // namespace pq
