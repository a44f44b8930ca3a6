// W4A8 prefill GEMM on CTA pairs (tcgen05 cta_group::2) for sm_100a.  Packed INT4 weights are
// widened to INT8 inside the kernel, multiplied with the INT8 activation codes on the tensor
// cores one K-group (128) at a time, and every group's INT32 accumulator is dequantized with
// its own scale into an FP32 running sum:
//     R[m,n] += float(ACC_g[m,n]) * s_grp[g,n];     Y = fp16(R * s_tok[m]).
//
// Two CTAs share a 256 x 256 output tile.  Each loads its own 128 rows of Q, HALF of the packed
// weight tile (128 rows x 64 bytes per group) and the group's 256 scales; it widens its half of
// the weights into the swizzled K-major INT8 layout; the leader's tcgen05.mma (M = 256, N = 256)
// reads both halves and leaves each CTA's 128 x 256 group accumulator in that CTA's tensor
// memory.  Shared-memory traffic per group and CTA: 32 KB read by the tensor core + 8 KB read and
// 16 KB written by the widening, under the 64 KB the SM can move in the 512 cycles the four
// MMAs of a group take (a lone CTA with a 128 x 128 tile needs 56 KB per 256 cycles).
//
// The per-group dequantization is CUDA-core work proportional to M*N*K/128: one conversion and
// one fused multiply-add per accumulator element, 2 x 32768 instructions per group and CTA against
// 4 x 512 issue slots -- the arithmetic limit of this kernel sits at the tensor-core time.  It runs
// on eight warps (two per TMEM lane quadrant, 128 columns each) that keep their 128 running
// sums in registers and have the next tcgen05.ld in flight while 16 columns are processed.
//
// Warp roles (512 threads; register budgets moved with setmaxnreg):
//   warp 0        TMA producer (Q tile counted on the LEADER's barrier; packed weights + scales
//                 on a local one, and requested before the wait on the preceding kernel)
//   warp 1        MMA issuer (leader CTA only; owns TMEM allocation in both CTAs)
//   warps 4-7     widen nibbles -> INT8 (16 x code: the nibble sits in the high half of the byte,
//                 which keeps two's complement; 1/16 is folded exactly into the FP32 scale).
//                 Warp w takes every fourth K-group whole, so that the proxy fence that ends a
//                 group (generic writes -> tensor-core reads, several hundred cycles) overlaps
//                 with the other three warps' work
//   warps 8-15    promotion, and after the last group x token scale -> FP16 -> TMA store
#include <cuda_fp16.h>

#include "pq_internal.h"
#include "pq_ptx.cuh"

namespace pq {
namespace {

constexpr int BM_CTA = 128, BM_PAIR = 256, BN = 256, BK = 128, UMMA_K = 32;
constexpr int STAGES = 5;       // Q + packed-weight + scale stages
constexpr int B8_SLOTS = 4;     // widened weight tiles (this CTA's half)
constexpr int SC_SLOTS = 4;     // FP32 scale rows
constexpr int ACC_SLOTS = 2;    // TMEM accumulators of BN columns
constexpr int kNumThreads = 512;
constexpr int kUnpackWarps = 4;
constexpr int kPromoteWarps = 8;
constexpr int kRegsCtl = 64, kRegsUnpack = 64, kRegsPromote = 192;   // x128, x128, x256 threads = 64 Ki

constexpr int kABytes = BM_CTA * BK;            // 16 KB of codes
constexpr int kPBytes = (BN / 2) * BK / 2;      // 8 KB packed weights (this CTA's 128 rows)
constexpr int kSBytes = BN * 2;                 // FP16 scales of one group
constexpr int kStageBytes = kABytes + kPBytes + 1024;  // scales padded to keep 1024-B alignment
constexpr int kTxP = kPBytes + kSBytes;
constexpr int kB8Bytes = (BN / 2) * BK;         // 16 KB
constexpr int kOutBoxBytes = 32 * 32 * 2;
constexpr int kB8Off = STAGES * kStageBytes;
constexpr int kScOff = kB8Off + B8_SLOTS * kB8Bytes;
constexpr int kOutOff = kScOff + SC_SLOTS * BN * 4;
constexpr int kBarOff = kOutOff + kPromoteWarps * kOutBoxBytes;
constexpr int kNumBars = 3 * STAGES + 2 * B8_SLOTS + 2 * SC_SLOTS + 2 * ACC_SLOTS;
constexpr int kMiscOff = kBarOff + kNumBars * 8;
constexpr int kDynamicSmem = kMiscOff + 16 + 1024;
static_assert(kDynamicSmem <= 232448, "exceeds the shared memory of one CTA");
static_assert(BK / UMMA_K == 4, "the MMA issuer is unrolled for four steps per group");
static_assert(128 * kRegsCtl + 128 * kRegsUnpack + 256 * kRegsPromote <= 65536, "register budget");

struct W4Args {
  const float* s_tok;
  int32_t* acc_g;  // [G, M, N] when exporting
  int* status;
  int M, N, K;
  int m_blocks, n_blocks, k_blocks;
};

template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

template <bool kExportAcc>
__global__ void __launch_bounds__(kNumThreads, 1)
gemm_w4a8_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_w,
                 const __grid_constant__ CUtensorMap tm_s, const __grid_constant__ CUtensorMap tm_y,
                 const W4Args p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_fullA = smem_base + kBarOff;             // LEADER: both CTAs' Q tiles landed
  const uint32_t bar_fullP = bar_fullA + STAGES * 8;          // local: packed weights + scales landed
  const uint32_t bar_empty = bar_fullP + STAGES * 8;          // local: MMAs read Q, widening read the rest
  const uint32_t bar_b8_full = bar_empty + STAGES * 8;        // LEADER: both halves of the widened tile written
  const uint32_t bar_b8_empty = bar_b8_full + B8_SLOTS * 8;   // local: the pair's MMAs finished reading it
  const uint32_t bar_sc_full = bar_b8_empty + B8_SLOTS * 8;   // local: FP32 scales written
  const uint32_t bar_sc_empty = bar_sc_full + SC_SLOTS * 8;   // local: promotion warps read them
  const uint32_t bar_acc_full = bar_sc_empty + SC_SLOTS * 8;  // local: group accumulator complete
  const uint32_t bar_acc_empty = bar_acc_full + ACC_SLOTS * 8;  // LEADER: both CTAs' promotion drained it
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kMiscOff + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair_id = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;
  const int num_tiles = p.m_blocks * p.n_blocks;
  constexpr uint32_t kTmemCols = ACC_SLOTS * BN;  // 512

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_fullA + s * 8, 1);
      mbar_init(bar_fullP + s * 8, 1);
      mbar_init(bar_empty + s * 8, 2);    // the MMAs' commit + the widening warp of this group
    }
    for (int s = 0; s < B8_SLOTS; ++s) {
      mbar_init(bar_b8_full + s * 8, 2);  // one widening warp in each CTA
      mbar_init(bar_b8_empty + s * 8, 1);
    }
    for (int s = 0; s < SC_SLOTS; ++s) {
      mbar_init(bar_sc_full + s * 8, 1);
      mbar_init(bar_sc_empty + s * 8, kPromoteWarps);
    }
    for (int s = 0; s < ACC_SLOTS; ++s) {
      mbar_init(bar_acc_full + s * 8, 1);
      mbar_init(bar_acc_empty + s * 8, 2 * kPromoteWarps);
    }
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_w);
    tma_prefetch_desc(&tm_s);
    if constexpr (!kExportAcc) tma_prefetch_desc(&tm_y);
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

  grid_dep_launch();   // nothing above touched global data; the successor may begin its set-up

  if (warp < 4) {
    setmaxnreg_dec<kRegsCtl>();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------- TMA producer (both CTAs)
      const uint32_t fullA0 = mapa_u32(bar_fullA, 0);
      auto load_weights = [&](uint32_t s, int g, int n_tile) {
        const uint32_t dst = smem_base + s * kStageBytes;
        mbar_arrive_expect_tx(bar_fullP + s * 8, kTxP);
        tma_load_2d(dst + kABytes, &tm_w, bar_fullP + s * 8, g * (BK / 2), n_tile + static_cast<int>(rank) * (BN / 2));
        tma_load_2d(dst + kABytes + kPBytes, &tm_s, bar_fullP + s * 8, n_tile, g);
      };
      auto load_codes = [&](uint32_t s, int g, int m0) {
        // Only the leader arrives; the peer's bytes may land first (the count then runs negative).
        if (rank == 0) mbar_arrive_expect_tx(bar_fullA + s * 8, 2 * kABytes);
        tma_load_2d_pair(smem_base + s * kStageBytes, &tm_q, fullA0 + s * 8, g * BK, m0);
      };
      // First ring pass of the first tile: weights and scales (constants) before the wait on the
      // preceding kernel, the codes it may have produced after it.
      int pre = 0;
      if (pair_id < num_tiles) {
        pre = p.k_blocks < STAGES ? p.k_blocks : STAGES;
        for (int g = 0; g < pre; ++g) load_weights(static_cast<uint32_t>(g), g, (pair_id / p.m_blocks) * BN);
      }
      grid_dep_wait();
      if (pair_id < num_tiles) {
        const int m0 = (pair_id % p.m_blocks) * BM_PAIR + static_cast<int>(rank) * BM_CTA;
        for (int g = 0; g < pre; ++g) load_codes(static_cast<uint32_t>(g), g, m0);
      }
      uint32_t it = static_cast<uint32_t>(pre);
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
        const int m0 = (tile % p.m_blocks) * BM_PAIR + static_cast<int>(rank) * BM_CTA;
        const int n_tile = (tile / p.m_blocks) * BN;
        for (int g = (tile == pair_id ? pre : 0); g < p.k_blocks; ++g, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_empty + s * 8, ph ^ 1u, abort_flag)) { ok = false; break; }
          load_weights(s, g, n_tile);
          load_codes(s, g, m0);
        }
      }
      (void)ok;
    } else if (warp == 1 && lane == 0 && rank == 0) {
      // ---------------------------------------------------------- MMA issuer (leader only)
      constexpr uint32_t idesc = umma_idesc_s8(BM_PAIR, BN);
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
        for (int g = 0; g < p.k_blocks; ++g, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          const uint32_t u = it % B8_SLOTS, uph = (it / B8_SLOTS) & 1u;
          const uint32_t a = it % ACC_SLOTS, aph = (it / ACC_SLOTS) & 1u;
          // This one thread shares its scheduler with three busy warps, so every instruction between
          // a barrier opening and the MMAs leaving costs tens of cycles: operands are prepared
          // before the waits, and the wait most likely to open last comes last.
          const uint64_t a_desc = umma_desc_k_sw128(smem_base + s * kStageBytes);
          const uint64_t b_desc = umma_desc_k_sw128(smem_base + kB8Off + u * kB8Bytes);
          const uint32_t d_tmem = tmem_base + a * BN;
          if (!mbar_wait(bar_fullA + s * 8, ph, abort_flag) ||
              !mbar_wait_cluster(bar_b8_full + u * 8, uph, abort_flag) ||
              !mbar_wait_cluster(bar_acc_empty + a * 8, aph ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          umma_i8_pair_imm<0>(d_tmem, a_desc, b_desc, idesc);
          umma_i8_pair_imm<1>(d_tmem, a_desc + 2, b_desc + 2, idesc);
          umma_i8_pair_imm<1>(d_tmem, a_desc + 4, b_desc + 4, idesc);
          umma_i8_pair_imm<1>(d_tmem, a_desc + 6, b_desc + 6, idesc);
          umma_commit_pair_mcast(bar_acc_full + a * 8, 0x3);
          umma_commit_pair_mcast(bar_empty + s * 8, 0x3);
          umma_commit_pair_mcast(bar_b8_empty + u * 8, 0x3);
        }
      }
    }
  } else if (warp < 8) {
    // ------------------------------------------------------------ widen nibbles (warps 4..7)
    setmaxnreg_dec<kRegsUnpack>();
    const uint32_t uw = static_cast<uint32_t>(warp - 4);
    const uint32_t b8_full0 = mapa_u32(bar_b8_full, 0);
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
      for (int g = 0; g < p.k_blocks; ++g, ++it) {
        if ((it & (kUnpackWarps - 1)) != uw) continue;   // another warp's group
        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
        const uint32_t u = it % B8_SLOTS, uph = (it / B8_SLOTS) & 1u;
        const uint32_t v = it % SC_SLOTS, vph = (it / SC_SLOTS) & 1u;
        bool w = mbar_wait(bar_fullP + s * 8, ph, abort_flag);
        w = w && mbar_wait(bar_b8_empty + u * 8, uph ^ 1u, abort_flag);
        w = w && mbar_wait(bar_sc_empty + v * 8, vph ^ 1u, abort_flag);
        ok = __all_sync(0xffffffffu, w);
        if (!ok) break;
        const uint8_t* stage = smem + s * kStageBytes;
        const uint4* packed = reinterpret_cast<const uint4*>(stage + kABytes);
        uint8_t* b8 = smem + kB8Off + u * kB8Bytes;
#pragma unroll 4
        for (int i = 0; i < (BN / 2 * 4) / 32; ++i) {
          const int idx = lane + i * 32;
          const int r = idx >> 2, j = idx & 3;  // weight row in this CTA's half, 32-k run of the group
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
        const __half2* sh = reinterpret_cast<const __half2*>(stage + kABytes + kPBytes);
        float2* sc = reinterpret_cast<float2*>(smem + kScOff + v * BN * 4);
#pragma unroll
        for (int i = 0; i < BN / 64; ++i) {
          const float2 f = __half22float2(sh[lane + 32 * i]);
          sc[lane + 32 * i] = make_float2(f.x * 0.0625f, f.y * 0.0625f);
        }
        fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor-core (async) proxy
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster_addr(b8_full0 + u * 8);
          mbar_arrive(bar_sc_full + v * 8);
          mbar_arrive(bar_empty + s * 8);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ promotion + epilogue (warps 8..15)
    setmaxnreg_inc<kRegsPromote>();
    grid_dep_wait();                    // token scales come from the preceding kernel; Y is overwritten
    constexpr int HC = BN / 2;          // columns per promotion warp
    constexpr int NCH = HC / 32;        // 32-column boxes of the final store
    constexpr int CH = 16, NLD = HC / CH;   // 16 columns per tcgen05.ld
    const int pw = warp - 8;
    const int quad = warp & 3;
    const int half = pw >> 2;
    const uint32_t acc_empty0 = mapa_u32(bar_acc_empty, 0);
    uint8_t* out_warp = smem + kOutOff + pw * kOutBoxBytes;
    const uint32_t out_warp_u32 = smem_base + kOutOff + pw * kOutBoxBytes;
    const int sw = (lane >> 1) & 3;     // 64-byte swizzle of the staging buffer
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
      const int row0 = (tile % p.m_blocks) * BM_PAIR + static_cast<int>(rank) * BM_CTA + quad * 32;
      const int n0 = (tile / p.m_blocks) * BN + half * HC;
      const int row = row0 + lane;
      float R[HC];
#pragma unroll
      for (int j = 0; j < HC; ++j) R[j] = 0.0f;
      for (int g = 0; g < p.k_blocks; ++g, ++it) {
        const uint32_t a = it % ACC_SLOTS, aph = (it / ACC_SLOTS) & 1u;
        const uint32_t v = it % SC_SLOTS, vph = (it / SC_SLOTS) & 1u;
        bool w = mbar_wait(bar_acc_full + a * 8, aph, abort_flag);
        w = w && mbar_wait(bar_sc_full + v * 8, vph, abort_flag);
        ok = __all_sync(0xffffffffu, w);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + a * BN + half * HC;
        const uint32_t sc_addr = smem_base + kScOff + v * BN * 4 + half * HC * 4;
        uint32_t r[2][CH];
        tmem_ld_32x16(t_addr, r[0]);
#pragma unroll
        for (int c = 0; c < NLD; ++c) {
          tmem_ld_wait();
          if (c + 1 < NLD) {
            tmem_ld_32x16(t_addr + (c + 1) * CH, r[(c + 1) & 1]);
          } else {
            // The whole slice is in registers: hand the accumulator back before the arithmetic.
            // (Relaxed arrive: the data moved through tensor memory, ordered by the tcgen05 fence.)
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_addr_relaxed(acc_empty0 + a * 8);
          }
          const uint32_t(&x)[CH] = r[c & 1];
          if constexpr (kExportAcc) {
            if (row < p.M) {
              int32_t* dst = p.acc_g + (static_cast<int64_t>(g) * p.M + row) * p.N + n0 + c * CH;
#pragma unroll
              for (int j = 0; j < CH; j += 4) {
                if (n0 + c * CH + j < p.N) {
                  *reinterpret_cast<int4*>(dst + j) =
                      make_int4(static_cast<int32_t>(x[j]) >> 4, static_cast<int32_t>(x[j + 1]) >> 4,
                                static_cast<int32_t>(x[j + 2]) >> 4, static_cast<int32_t>(x[j + 3]) >> 4);
                }
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < CH; j += 4) {
              float4 s4;   // scales of columns j..j+3
              asm("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                  : "=f"(s4.x), "=f"(s4.y), "=f"(s4.z), "=f"(s4.w)
                  : "r"(sc_addr + (c * CH + j) * 4));
              R[c * CH + j + 0] = fmaf(__int2float_rn(static_cast<int32_t>(x[j + 0])), s4.x, R[c * CH + j + 0]);
              R[c * CH + j + 1] = fmaf(__int2float_rn(static_cast<int32_t>(x[j + 1])), s4.y, R[c * CH + j + 1]);
              R[c * CH + j + 2] = fmaf(__int2float_rn(static_cast<int32_t>(x[j + 2])), s4.z, R[c * CH + j + 2]);
              R[c * CH + j + 3] = fmaf(__int2float_rn(static_cast<int32_t>(x[j + 3])), s4.w, R[c * CH + j + 3]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sc_empty + v * 8);
      }
      if constexpr (!kExportAcc) {
        if (ok) {
          const float st = (row < p.M) ? __ldg(p.s_tok + row) : 0.0f;
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            if (lane == 0) tma_store_wait_read<0>();   // the previous store has read the staging buffer
            __syncwarp();
            uint8_t* dst = out_warp + lane * 64;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t o[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const __half2 h = __floats2half2_rn(R[c * 32 + 8 * j + 2 * i] * st, R[c * 32 + 8 * j + 2 * i + 1] * st);
                o[i] = *reinterpret_cast<const uint32_t*>(&h);
              }
              *reinterpret_cast<uint4*>(dst + ((j ^ sw) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (n0 + c * 32 < p.N && row0 < p.M) tma_store_2d(&tm_y, out_warp_u32, n0 + c * 32, row0);
              tma_store_commit();
            }
          }
        }
      }
    }
    if constexpr (!kExportAcc) {
      if (lane == 0) tma_store_wait_read<0>();
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

template <bool kExportAcc>
int launch_w4(const CUtensorMap& tq, const CUtensorMap& tw, const CUtensorMap& ts, const CUtensorMap& ty,
              const W4Args& a, cudaStream_t stream) {
  auto kern = gemm_w4a8_kernel<kExportAcc>;
  static int configured = 0;  // 0 = not yet, 1 = ok, -1 = unusable
  if (configured == 0) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return PQ_ERR_CUDA;
    // The promotion warps raise their register budget with setmaxnreg; that only terminates if the
    // CTA's allocation (registers per thread at launch x 512) holds the sum of the three budgets.
    if (fa.numRegs * kNumThreads < 128 * kRegsCtl + 128 * kRegsUnpack + 256 * kRegsPromote) {
      configured = -1;
    } else if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynamicSmem) != cudaSuccess) {
      return PQ_ERR_CUDA;
    } else {
      configured = 1;
    }
  }
  if (configured < 0) return PQ_ERR_CUDA;
  const int tiles = a.m_blocks * a.n_blocks;
  const int max_pairs = sm_count() / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs), 1, 1);
  cfg.blockDim = dim3(kNumThreads, 1, 1);
  cfg.dynamicSmemBytes = kDynamicSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  return cuda_status(cudaLaunchKernelEx(&cfg, kern, tq, tw, ts, ty, a));
}

}  // namespace

int launch_gemm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M,
                     int64_t N, int64_t K, void* y, int32_t* acc_g, cudaStream_t stream) {
  CUtensorMap tq, tw, ts, ty;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), BM_CTA, BK, 1, 128);
  if (rc != PQ_OK) return rc;
  rc = make_tmap_2d(&tw, wp, static_cast<uint64_t>(N), static_cast<uint64_t>(K / 2), BN / 2, BK / 2, 1, 0);
  if (rc != PQ_OK) return rc;
  // Group scales [K/128, N] FP16; the accumulator-export variant has none and reads a dummy map of Q.
  if (s_grp != nullptr) {
    rc = make_tmap_2d(&ts, s_grp, static_cast<uint64_t>(K / 128), static_cast<uint64_t>(N), 1, BN, 2, 0);
  } else {
    rc = make_tmap_2d(&ts, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K / 2), 1, BN, 2, 0);
  }
  if (rc != PQ_OK) return rc;
  if (y != nullptr) {
    rc = make_tmap_2d(&ty, y, static_cast<uint64_t>(M), static_cast<uint64_t>(N), 32, 32, 2, 64);
    if (rc != PQ_OK) return rc;
  } else {
    ty = tq;  // not used by the accumulator export
  }
  W4Args a;
  a.s_tok = s_tok;
  a.acc_g = acc_g;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.N = static_cast<int>(N);
  a.K = static_cast<int>(K);
  a.m_blocks = static_cast<int>((M + BM_PAIR - 1) / BM_PAIR);
  a.n_blocks = static_cast<int>((N + BN - 1) / BN);
  a.k_blocks = static_cast<int>(K / BK);
  return acc_g != nullptr ? launch_w4<true>(tq, tw, ts, ty, a, stream) : launch_w4<false>(tq, tw, ts, ty, a, stream);
}

}  // namespace pq
