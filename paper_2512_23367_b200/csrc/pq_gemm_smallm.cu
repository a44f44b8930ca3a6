// Small-M (decode-shaped; M <= 128) linear for sm_100a: a weight-streaming schedule
// that computes the same result as the prefill kernels.
//
// The roles of the two operands are swapped: a tile of 128 WEIGHT rows is the 128-lane operand
// of tcgen05.mma and the (zero-padded) tokens are the narrow N dimension (16, 32, 64 or 128), so one
// instruction consumes 4 KB of weights and the tensor pipe stays far below its limit while the
// weights stream from HBM exactly once.  The K dimension is split over the CTAs of a thread-block
// cluster (up to 8) so that ~2 CTAs per SM pull weights concurrently; the partial results are
// reduced through distributed shared memory in a fixed order (exact for the INT32 accumulators
// of W8A8, deterministic for the FP32 group sums of W4A8) and the cluster's CTAs share the
// dequantize + FP16 store work.  No global scratch memory is used.
//
//   warp 0      TMA producer (weights + token tile per 128-deep K block)
//   warp 1      MMA issuer
//   warps 2-3, 8-9   W4 only: nibble -> INT8 widening into the swizzled operand layout; the two
//               pairs of warps take the K blocks in turn (even / odd), each into its own slot, so
//               that one pair's proxy fence and hand-over overlap with the other pair's work
//   warps 4-7   TMEM -> registers (W4: per-group promotion with the row's own group scale),
//               cross-CTA reduction, dequantization, FP16 store
#include <cuda_fp16.h>

#include <cstdlib>

#include "pq_internal.h"
#include "pq_ptx.cuh"

namespace pq {
namespace {

constexpr int BW = 128;   // weight rows per tile (TMEM lanes)
constexpr int BK = 128;   // K per block = one W4 group
constexpr int UMMA_K = 32;
constexpr int kUnpackThreads = 64;    // per K block (one pair of warps)
constexpr int kMaxSplit = 8;  // portable cluster size

template <int MPAD, bool kW4>
struct Cfg {
  static constexpr int kWBytes = kW4 ? BW * BK / 2 : BW * BK;    // weight tile as loaded
  static constexpr int kQBytes = MPAD * BK;                      // token tile (128-byte swizzle)
  static constexpr int kSBytes = kW4 ? BW * 2 : 0;               // FP16 group scales of the tile
  static constexpr int kStageBytes = kWBytes + kQBytes + (kW4 ? 1024 : 0);
  static constexpr int kTxBytes = kWBytes + kQBytes + kSBytes;
  // Short rings and small footprints: three or four CTAs fit on an SM, so the CTAs of the NEXT
  // launch become resident (and stream their weights) while this launch reduces and stores.
  static constexpr int STAGES = (kW4 && MPAD > 64) ? 6 : ((kW4 || MPAD == 64) ? 4 : 3);
  // W4: two pairs of widening warps, except at 64 tokens (that variant needs its registers for the 64
  // per-thread partial results and keeps one pair and two co-resident CTAs).  At 128 tokens one CTA
  // owns the SM: a six-deep ring, four widened slots, eight epilogue warps.
  static constexpr int kUnpackPairs = (kW4 && MPAD != 64) ? 2 : 1;
  // Warps: 0 producer, 1 MMA issuer, 2-3 first widening pair, then the epilogue warps (W4 at 128 tokens:
  // two per TMEM lane quadrant, 64 token columns each, so that a thread keeps 64 partial results), then
  // the second widening pair.
  static constexpr int kEpiWarps = (kW4 && MPAD > 64) ? 8 : 4;
  static constexpr int kEpiEnd = 4 + kEpiWarps;                  // first warp after the epilogue warps
  static constexpr int kEpiCols = MPAD / (kEpiWarps / 4);        // token columns per epilogue warp
  static constexpr int kThreads = 32 * (kEpiEnd + (kUnpackPairs == 2 ? 2 : 0));
  static constexpr int kMinCtasPerSm = (kW4 && MPAD > 64) ? 1 : (MPAD >= 64 ? 2 : (kW4 ? 2 : 4));
  static constexpr int A8_SLOTS = kW4 ? (MPAD > 64 ? 4 : 2) : 0;                   // widened weight tiles: one per pair of widening warps
  static constexpr int kA8Bytes = BW * BK;
  static constexpr int SC_SLOTS = kW4 ? 6 : 0;                   // FP32 scale rows (128 floats)
  static constexpr int ACC_SLOTS = kW4 ? 4 : 1;
  static constexpr int kA8Off = STAGES * kStageBytes;
  static constexpr int kScOff = kA8Off + A8_SLOTS * kA8Bytes;
  static constexpr int kRingEnd = kScOff + SC_SLOTS * BW * 4;
  static constexpr int kRedBytes = MPAD * BW * 4;                // aliases the stage ring
  static constexpr int kBarOff = (kRingEnd > kRedBytes ? kRingEnd : kRedBytes);
  // A barrier's phases are told apart by one parity bit, so a warp may only wait on barriers whose every
  // phase it sees in turn: with two widening pairs alternating over the K blocks, each ring's length is even.
  static_assert(!kW4 || (STAGES % kUnpackPairs == 0 && A8_SLOTS % kUnpackPairs == 0 && SC_SLOTS % kUnpackPairs == 0),
                "ring lengths and widening pairs");
  static constexpr int kNumBars = 2 * STAGES + 2 * A8_SLOTS + 2 * SC_SLOTS + 2 * ACC_SLOTS + 1;   // + the MMA issuer's drain barrier
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  // A CTA that takes all 512 TMEM columns must be alone on its SM (a second one would block in
  // tcgen05.alloc): its shared-memory request is raised past half an SM's so that it always is.
  static constexpr int kNeeded = kMiscOff + 16 + 1024;
  static constexpr int kDynamic = (ACC_SLOTS * MPAD > 256 && kNeeded < 117 * 1024) ? 117 * 1024 : kNeeded;
  static constexpr uint32_t kTmemCols = (ACC_SLOTS * MPAD) < 32 ? 32 : (ACC_SLOTS * MPAD);
};

struct SmallArgs {
  const float* s_tok;
  const float* s_ch[kMaxGroup];   // W8, per member
  __half* y[kMaxGroup];           // per member
  int N[kMaxGroup];               // per member
  int tile_end[kMaxGroup];        // 128-channel tiles of members 0..g (running total); INT_MAX past the last
  int count;                      // members in this launch (linears over the same tokens)
  int32_t* acc;          // export (single member): W8 [M,N]; W4 [G,M,N]
  int* status;
  int M, K;
  int k_blocks, splits;
  uint32_t wait_limit;   // poll bound of every wait
};

// Tensor maps of the members' weights (and W4 group scales), indexed by member.
struct SmallMaps {
  CUtensorMap w[kMaxGroup];
  CUtensorMap s[kMaxGroup];
};

__device__ __forceinline__ uint4 ld_dsmem_v4(uint32_t local_addr, uint32_t rank) {
  uint4 v;
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %4, %5;\n\t"
      "ld.shared::cluster.v4.b32 {%0, %1, %2, %3}, [ra];\n\t}"
      : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
      : "r"(local_addr), "r"(rank)
      : "memory");
  return v;
}

template <int MPAD>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[MPAD]) {
  if constexpr (MPAD == 16) {
    tmem_ld_32x16(taddr, r);
  } else if constexpr (MPAD == 32) {
    tmem_ld_32x32(taddr, r);
  } else {
    uint32_t(&lo)[32] = *reinterpret_cast<uint32_t(*)[32]>(&r[0]);
    uint32_t(&hi)[32] = *reinterpret_cast<uint32_t(*)[32]>(&r[32]);
    tmem_ld_32x32(taddr, lo);
    tmem_ld_32x32(taddr + 32, hi);
  }
}

template <int MPAD, bool kW4, bool kExportAcc>
__global__ void __launch_bounds__(Cfg<MPAD, kW4>::kThreads, Cfg<MPAD, kW4>::kMinCtasPerSm)
smallm_kernel(const __grid_constant__ SmallMaps maps, const __grid_constant__ CUtensorMap tm_q, const SmallArgs p) {
  using C = Cfg<MPAD, kW4>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_full = smem_base + C::kBarOff;
  const uint32_t bar_empty = bar_full + C::STAGES * 8;
  const uint32_t bar_a8_full = bar_empty + C::STAGES * 8;
  const uint32_t bar_a8_empty = bar_a8_full + C::A8_SLOTS * 8;
  const uint32_t bar_sc_full = bar_a8_empty + C::A8_SLOTS * 8;
  const uint32_t bar_sc_empty = bar_sc_full + C::SC_SLOTS * 8;
  const uint32_t bar_acc_full = bar_sc_empty + C::SC_SLOTS * 8;
  const uint32_t bar_acc_empty = bar_acc_full + C::ACC_SLOTS * 8;
  const uint32_t bar_drain = bar_acc_empty + C::ACC_SLOTS * 8;   // give-up path of the MMA issuer only
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::kMiscOff + 4);
  const WaitCtx wc{abort_flag, p.wait_limit};

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // This CTA's member and first channel inside it (grid.x runs over the tiles of all members).
  int member = 0, tile = static_cast<int>(blockIdx.x);
  if (p.count > 1) {
    const int e0 = p.tile_end[0], e1 = p.tile_end[1], e2 = p.tile_end[2];
    if (tile >= e2) { member = 3; tile -= e2; }
    else if (tile >= e1) { member = 2; tile -= e1; }
    else if (tile >= e0) { member = 1; tile -= e0; }
  }
  const int n0 = tile * BW;
  const int N_mem = member == 0 ? p.N[0] : (member == 1 ? p.N[1] : (member == 2 ? p.N[2] : p.N[3]));
  const float* s_ch_mem = member == 0 ? p.s_ch[0] : (member == 1 ? p.s_ch[1] : (member == 2 ? p.s_ch[2] : p.s_ch[3]));
  __half* y_mem = member == 0 ? p.y[0] : (member == 1 ? p.y[1] : (member == 2 ? p.y[2] : p.y[3]));
  const CUtensorMap* tm_w = &maps.w[member];
  const CUtensorMap* tm_s = &maps.s[member];
  const int split = blockIdx.y;                       // == rank in the cluster (cluster = all of grid.y)
  const int m0 = static_cast<int>(blockIdx.z) * MPAD;  // first token of this CTA (grid.z runs over blocks of MPAD tokens)
  const int m_live = p.M - m0 < MPAD ? p.M - m0 : MPAD;
  const int kb0 = static_cast<int>(static_cast<int64_t>(p.k_blocks) * split / p.splits);
  const int kb1 = static_cast<int>(static_cast<int64_t>(p.k_blocks) * (split + 1) / p.splits);
  const int nkb = kb1 - kb0;

  // The j-th K block of this CTA goes into stage j % STAGES.  Weights (and W4 group scales) are
  // constants of the model and may be requested before the wait on the preceding kernel; the
  // token codes may be its output and are requested after it.
  auto issue_weights = [&](int j) {
    const uint32_t s = static_cast<uint32_t>(j) % C::STAGES;
    const uint32_t dst = smem_base + s * C::kStageBytes;
    const int kb = kb0 + j;
    mbar_arrive_expect_tx(bar_full + s * 8, C::kTxBytes);
    tma_load_2d(dst, tm_w, bar_full + s * 8, kW4 ? kb * (BK / 2) : kb * BK, n0);
    if constexpr (kW4) tma_load_2d(dst + C::kWBytes + C::kQBytes, tm_s, bar_full + s * 8, n0, kb);
  };
  auto issue_codes = [&](int j) {
    const uint32_t s = static_cast<uint32_t>(j) % C::STAGES;
    tma_load_2d(smem_base + s * C::kStageBytes + C::kWBytes, &tm_q, bar_full + s * 8, (kb0 + j) * BK, m0);
  };

  if (threadIdx.x == 64) {
    tma_prefetch_desc(tm_w);
    tma_prefetch_desc(&tm_q);
    if constexpr (kW4) tma_prefetch_desc(tm_s);
  }
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar_drain, 1);
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(bar_full + s * 8, 1);
      mbar_init(bar_empty + s * 8, kW4 ? 1 + kUnpackThreads / 32 : 1);
    }
    for (int s = 0; s < C::A8_SLOTS; ++s) {
      mbar_init(bar_a8_full + s * 8, kUnpackThreads / 32);
      mbar_init(bar_a8_empty + s * 8, 1);
    }
    for (int s = 0; s < C::SC_SLOTS; ++s) {
      mbar_init(bar_sc_full + s * 8, kUnpackThreads / 32);
      mbar_init(bar_sc_empty + s * 8, C::kEpiWarps);
    }
    for (int s = 0; s < C::ACC_SLOTS; ++s) {
      mbar_init(bar_acc_full + s * 8, 1);
      mbar_init(bar_acc_empty + s * 8, C::kEpiWarps);
    }
    fence_mbar_init();
    // Start the weight stream at once: the first ring pass needs no wait, neither on a stage
    // nor on the preceding kernel.
    const int first = nkb < C::STAGES ? nkb : C::STAGES;
    for (int j = 0; j < first; ++j) issue_weights(j);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // The successor may now become resident and start streaming its own weights.  Only now: every CTA of this
  // launch holds its tensor memory before a later launch's CTA can ask for any (a CTA that took all columns
  // of an SM and then waited for this launch, while a CTA of this launch still waited for columns, would never
  // be released).
  grid_dep_launch();

  // W4: per-thread partial results of the epilogue warps, P[m] for weight row n0 + 32*quad + lane.
  // (W8 copies its one accumulator from tensor memory straight into the reduction tile.)
  constexpr int kPartials = kW4 ? C::kEpiCols : 1;
  uint32_t P[kPartials];
#pragma unroll
  for (int m = 0; m < kPartials; ++m) P[m] = 0u;
  bool ok = true;
  int issued = 0;   // producer thread: K blocks it has requested (for the give-up path)

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (remaining blocks)
    if (lane == 0) {
      grid_dep_wait();   // the token codes may come from the preceding kernel
      const int first = nkb < C::STAGES ? nkb : C::STAGES;
      for (int j = 0; j < first; ++j) issue_codes(j);
      int j = C::STAGES;
      for (; j < nkb; ++j) {
        const uint32_t s = static_cast<uint32_t>(j) % C::STAGES, ph = (static_cast<uint32_t>(j) / C::STAGES) & 1u;
        if (!mbar_wait(bar_empty + s * 8, ph ^ 1u, wc)) { ok = false; break; }
        issue_weights(j);
        issue_codes(j);
      }
      issued = j < nkb ? j : nkb;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_s8(BW, MPAD);
      for (int j = 0; j < nkb; ++j) {
        const uint32_t it = static_cast<uint32_t>(j);
        const uint32_t s = it % C::STAGES, ph = (it / C::STAGES) & 1u;
        const uint32_t stage = smem_base + s * C::kStageBytes;
        uint64_t w_desc;
        uint32_t d_tmem = tmem_base;
        if constexpr (kW4) {
          const uint32_t u = it % C::A8_SLOTS, uph = (it / C::A8_SLOTS) & 1u;
          const uint32_t a = it % C::ACC_SLOTS, aph = (it / C::ACC_SLOTS) & 1u;
          w_desc = umma_desc_k_sw128(smem_base + C::kA8Off + u * C::kA8Bytes);
          d_tmem = tmem_base + a * MPAD;
          // (the three waits share their round trips)
          if (!mbar_wait3(bar_full + s * 8, ph, bar_a8_full + u * 8, uph, bar_acc_empty + a * 8, aph ^ 1u,
                          wc)) { ok = false; break; }
        } else {
          if (!mbar_wait(bar_full + s * 8, ph, wc)) { ok = false; break; }
          w_desc = umma_desc_k_sw128(stage);
        }
        tc_fence_after_sync();
        const uint64_t q_desc = umma_desc_k_sw128(stage + C::kWBytes);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          const uint32_t accumulate = kW4 ? (k != 0) : ((j | k) != 0);
          umma_i8(d_tmem, w_desc + 2 * k, q_desc + 2 * k, idesc, accumulate);
        }
        umma_commit(bar_empty + s * 8);
        if constexpr (kW4) {
          umma_commit(bar_a8_empty + (it % C::A8_SLOTS) * 8);
          umma_commit(bar_acc_full + (it % C::ACC_SLOTS) * 8);
        }
      }
      if constexpr (!kW4) {
        if (ok) umma_commit(bar_acc_full);
      }
    }
  } else if (warp < 4 || warp >= C::kEpiEnd) {
    // ------------------------------------------------------------ W4: widen nibbles to INT8
    if constexpr (kW4) {
      const int pair = warp >= C::kEpiEnd ? 1 : 0;             // warps 2-3: even K blocks, the last two warps: odd ones
      const int ut = threadIdx.x - (pair ? C::kEpiEnd * 32 : 64);
      for (int j = pair; j < nkb; j += C::kUnpackPairs) {
        const uint32_t it = static_cast<uint32_t>(j);
        const uint32_t s = it % C::STAGES, ph = (it / C::STAGES) & 1u;
        const uint32_t u = it % C::A8_SLOTS, uph = (it / C::A8_SLOTS) & 1u;
        const uint32_t v = it % C::SC_SLOTS, vph = (it / C::SC_SLOTS) & 1u;
        const bool w = mbar_wait3(bar_full + s * 8, ph, bar_a8_empty + u * 8, uph ^ 1u, bar_sc_empty + v * 8,
                                  vph ^ 1u, wc);
        ok = __all_sync(0xffffffffu, w);
        if (!ok) break;
        const uint8_t* stage = smem + s * C::kStageBytes;
        const uint4* packed = reinterpret_cast<const uint4*>(stage);
        uint8_t* a8 = smem + C::kA8Off + u * C::kA8Bytes;
#pragma unroll
        for (int i = 0; i < (BW * 4) / kUnpackThreads; ++i) {
          const int idx = ut + i * kUnpackThreads;
          const int r = idx >> 2, c = idx & 3;
          const uint4 w4 = packed[idx];
          uint4 lo, hi;
          lo.x = (w4.x << 4) & 0xF0F0F0F0u; hi.x = w4.x & 0xF0F0F0F0u;
          lo.y = (w4.y << 4) & 0xF0F0F0F0u; hi.y = w4.y & 0xF0F0F0F0u;
          lo.z = (w4.z << 4) & 0xF0F0F0F0u; hi.z = w4.z & 0xF0F0F0F0u;
          lo.w = (w4.w << 4) & 0xF0F0F0F0u; hi.w = w4.w & 0xF0F0F0F0u;
          uint8_t* row = a8 + r * 128;
          const int sw = r & 7;
          *reinterpret_cast<uint4*>(row + (((2 * c) ^ sw) << 4)) = lo;
          *reinterpret_cast<uint4*>(row + (((2 * c + 1) ^ sw) << 4)) = hi;
        }
        const __half* sh = reinterpret_cast<const __half*>(stage + C::kWBytes + C::kQBytes);
        float* sc = reinterpret_cast<float*>(smem + C::kScOff) + v * BW;
        for (int c = ut; c < BW; c += kUnpackThreads) sc[c] = __half2float(sh[c]) * 0.0625f;
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_a8_full + u * 8);
          mbar_arrive(bar_sc_full + v * 8);
          mbar_arrive(bar_empty + s * 8);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ TMEM -> registers
    grid_dep_wait();   // token scales come from the preceding kernel; outputs are overwritten
    const int quad = warp & 3;
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const int n_local = quad * 32 + lane;
    if constexpr (kW4) {
      const int col0 = ((warp - 4) >> 2) * C::kEpiCols;   // this warp's first token column
      constexpr int CH = MPAD < 32 ? MPAD : 32;  // columns promoted per tcgen05.ld
      for (int j = 0; j < nkb; ++j) {
        const uint32_t it = static_cast<uint32_t>(j);
        const uint32_t a = it % C::ACC_SLOTS, aph = (it / C::ACC_SLOTS) & 1u;
        const uint32_t v = it % C::SC_SLOTS, vph = (it / C::SC_SLOTS) & 1u;
        const bool w = mbar_wait2(bar_acc_full + a * 8, aph, bar_sc_full + v * 8, vph, wc);
        ok = __all_sync(0xffffffffu, w);
        if (!ok) break;
        tc_fence_after_sync();
        const float sg = (reinterpret_cast<const float*>(smem + C::kScOff) + v * BW)[n_local];
#pragma unroll
        for (int c0 = 0; c0 < C::kEpiCols; c0 += CH) {
          uint32_t r[CH];
          tmem_ld_cols<CH>(lane_addr + a * MPAD + col0 + c0, r);
          tmem_ld_wait();
          if constexpr (kExportAcc) {
            const int n = n0 + n_local;
#pragma unroll
            for (int m = 0; m < CH; ++m) {
              if (col0 + c0 + m < m_live && n < N_mem)
                p.acc[(static_cast<int64_t>(kb0 + j) * p.M + m0 + col0 + c0 + m) * N_mem + n] = static_cast<int32_t>(r[m]) >> 4;
            }
          } else {
#pragma unroll
            for (int m = 0; m < CH; ++m)
              P[c0 + m] = __float_as_uint(fmaf(__int2float_rn(static_cast<int32_t>(r[m])), sg, __uint_as_float(P[c0 + m])));
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_acc_empty + a * 8);
          mbar_arrive(bar_sc_empty + v * 8);
        }
      }
    } else {
      // All K blocks of this CTA are consumed once the accumulator is complete, so the stage ring is
      // free: the partial tile goes there as red[m][n] (32-bit words), 32 token columns at a time.
      uint32_t* red_w8 = reinterpret_cast<uint32_t*>(smem);
      if (nkb > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full, 0u, wc));
      if (ok) tc_fence_after_sync();
      constexpr int CW = MPAD < 32 ? MPAD : 32;
#pragma unroll
      for (int c0 = 0; c0 < MPAD; c0 += CW) {
        uint32_t r[CW];
        if (ok && nkb > 0) {
          tmem_ld_cols<CW>(lane_addr + c0, r);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int m = 0; m < CW; ++m) r[m] = 0u;
        }
#pragma unroll
        for (int m = 0; m < CW; ++m) red_w8[(c0 + m) * BW + n_local] = r[m];
      }
      tc_fence_before_sync();
    }
  }

  // ------------------------------------------------------------ cross-CTA reduction + store
  // All K blocks of this CTA are consumed (the epilogue warps saw the last accumulator), so the
  // stage ring is free and holds this CTA's partial tile as red[m][n] (32-bit words).
  uint32_t* red = reinterpret_cast<uint32_t*>(smem);
  const bool do_reduce = !(kW4 && kExportAcc);
  if (do_reduce && kW4 && warp >= 4 && warp < C::kEpiEnd) {
    const int n_local = (warp & 3) * 32 + lane;
    const int col0 = ((warp - 4) >> 2) * C::kEpiCols;
#pragma unroll
    for (int m = 0; m < kPartials; ++m) red[(col0 + m) * BW + n_local] = P[m];
  }
  tc_fence_before_sync();
  __syncwarp();
  cluster_sync_all();
  if (*abort_flag) {
    // Some role of this CTA gave up (every role is past its loop here).  Work already handed to the
    // hardware still completes by itself and must have done so before this CTA's shared and tensor
    // memory go away: the producer's loads and the issuer's MMAs.  (The other threads go on to the
    // reduction, whose result is unspecified after a give-up, and meet these two at the next barrier.)
    if (threadIdx.x == 0) {
      const int first = issued > C::STAGES ? issued - C::STAGES : 0;
      for (int i = first; i < issued; ++i)
        mbar_drain(bar_full + (static_cast<uint32_t>(i) % C::STAGES) * 8, (static_cast<uint32_t>(i) / C::STAGES) & 1u);
    } else if (threadIdx.x == 32) {
      umma_commit(bar_drain);
      mbar_drain(bar_drain, 0u);
    }
  }
  if (do_reduce && warp >= 4 && warp < C::kEpiEnd) {
    // Thread t owns four consecutive output channels (one 16-byte word of every part's partial
    // tile) for the rows m = rank + splits * (t / 32 + kEpiWarps i): the remote loads of all parts of a row
    // are issued together, so a row costs one distributed-shared-memory round trip, not `splits`.
    const int t = threadIdx.x - 128;
    const int nq = t & 31, msub = t >> 5;
    const int n = n0 + 4 * nq;
    const uint32_t my_rank = cluster_ctarank();
    float sc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (!kW4 && !kExportAcc && n < N_mem) {
#pragma unroll
      for (int j = 0; j < 4; ++j) sc[j] = __ldg(s_ch_mem + n + j);   // N is a multiple of 8: n < N covers n + 3
    }
    for (int m = static_cast<int>(my_rank) + p.splits * msub; m < m_live; m += C::kEpiWarps * p.splits) {
      const uint32_t addr = smem_base + static_cast<uint32_t>(m * BW + 4 * nq) * 4u;
      uint4 part[kMaxSplit];
#pragma unroll
      for (int r = 0; r < kMaxSplit; ++r) {
        if (r < p.splits) part[r] = ld_dsmem_v4(addr, static_cast<uint32_t>(r));
      }
      if (n >= N_mem) continue;
      if constexpr (kW4) {
        float tot[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int r = 0; r < kMaxSplit; ++r) {
          if (r < p.splits) {
            tot[0] += __uint_as_float(part[r].x); tot[1] += __uint_as_float(part[r].y);
            tot[2] += __uint_as_float(part[r].z); tot[3] += __uint_as_float(part[r].w);
          }
        }
        const float st = __ldg(p.s_tok + m0 + m);
        const __half2 h01 = __floats2half2_rn(tot[0] * st, tot[1] * st), h23 = __floats2half2_rn(tot[2] * st, tot[3] * st);
        *reinterpret_cast<uint2*>(y_mem + static_cast<int64_t>(m0 + m) * N_mem + n) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
      } else {
        int32_t tot[4] = {0, 0, 0, 0};
#pragma unroll
        for (int r = 0; r < kMaxSplit; ++r) {
          if (r < p.splits) {
            tot[0] += static_cast<int32_t>(part[r].x); tot[1] += static_cast<int32_t>(part[r].y);
            tot[2] += static_cast<int32_t>(part[r].z); tot[3] += static_cast<int32_t>(part[r].w);
          }
        }
        if constexpr (kExportAcc) {
          *reinterpret_cast<int4*>(p.acc + static_cast<int64_t>(m0 + m) * N_mem + n) = make_int4(tot[0], tot[1], tot[2], tot[3]);
        } else {
          const float st = __ldg(p.s_tok + m0 + m);
          float v[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) v[j] = __fmul_rn(__fmul_rn(__int2float_rn(tot[j]), st), sc[j]);
          const __half2 h01 = __floats2half2_rn(v[0], v[1]), h23 = __floats2half2_rn(v[2], v[3]);
          *reinterpret_cast<uint2*>(y_mem + static_cast<int64_t>(m0 + m) * N_mem + n) =
              make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
        }
      }
    }
  }
  __syncwarp();
  cluster_sync_all();  // nobody leaves while a peer may still read its shared memory
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, C::kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, static_cast<int>(PQ_ERR_TIMEOUT));
}

template <int MPAD, bool kW4, bool kExportAcc>
int launch_cfg(const SmallMaps& maps, const CUtensorMap& tq, const SmallArgs& a, int n_tiles, int m_blocks,
               cudaStream_t stream) {
  using C = Cfg<MPAD, kW4>;
  auto kern = smallm_kernel<MPAD, kW4, kExportAcc>;
  static PerDeviceOnce once;   // one per kernel variant
  if (const int rc = set_dynamic_smem_once(once, kern, C::kDynamic); rc != PQ_OK) return rc;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(n_tiles), static_cast<unsigned>(a.splits), static_cast<unsigned>(m_blocks));
  cfg.blockDim = dim3(C::kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kDynamic;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = static_cast<unsigned>(a.splits);
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  return cuda_status(cudaLaunchKernelEx(&cfg, kern, maps, tq, a));
}

// `count` linears over the same tokens in one launch: grid.x runs over the 128-channel tiles of all
// members.  w / s_ch / s_grp / N / y are host arrays of `count` entries; acc (export) only with count == 1.
template <bool kW4>
int launch_smallm(const int8_t* q, const float* s_tok, int count, const void* const* w, const float* const* s_ch,
                  const void* const* s_grp, const int64_t* N, void* const* y, int64_t M, int64_t K, int32_t* acc,
                  cudaStream_t stream) {
  if (count < 1 || count > kMaxGroup || (acc != nullptr && count != 1)) return PQ_ERR_SHAPE;
  const int mpad = M <= 16 ? 16 : (M <= 32 ? 32 : (M <= 64 ? 64 : 128));
  const int m_blocks = static_cast<int>((M + mpad - 1) / mpad);   // > 1 only beyond 128 tokens
  const int k_blocks = static_cast<int>((K + BK - 1) / BK);

  CUtensorMap tq;
  SmallMaps maps;
  SmallArgs a;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), static_cast<uint32_t>(mpad), BK, 1, 128);
  if (rc != PQ_OK) return rc;
  int64_t n_tiles = 0;
  for (int g = 0; g < kMaxGroup; ++g) {
    const int src = g < count ? g : 0;   // unused slots repeat member 0 (never selected)
    if (kW4) {
      rc = make_tmap_2d(&maps.w[g], w[src], static_cast<uint64_t>(N[src]), static_cast<uint64_t>(K / 2), BW, BK / 2, 1, 0);
    } else {
      rc = make_tmap_2d(&maps.w[g], w[src], static_cast<uint64_t>(N[src]), static_cast<uint64_t>(K), BW, BK, 1, 128);
    }
    if (rc != PQ_OK) return rc;
    if (kW4 && acc == nullptr) {
      rc = make_tmap_2d(&maps.s[g], s_grp[src], static_cast<uint64_t>(K / 128), static_cast<uint64_t>(N[src]), 1, BW, 2, 0);
    } else if (kW4) {
      // the W4 accumulator export has no scales: it reads (and ignores) token bytes instead
      rc = make_tmap_2d(&maps.s[g], q, static_cast<uint64_t>(M), static_cast<uint64_t>(K / 2), 1, BW, 2, 0);
    } else {
      maps.s[g] = tq;  // unused by W8
    }
    if (rc != PQ_OK) return rc;
    a.s_ch[g] = kW4 ? nullptr : s_ch[src];
    a.y[g] = static_cast<__half*>(acc == nullptr ? y[src] : nullptr);
    a.N[g] = static_cast<int>(N[src]);
    if (g < count) n_tiles += (N[g] + BW - 1) / BW;
    a.tile_end[g] = g < count ? static_cast<int>(n_tiles) : 0x7fffffff;
  }
  if (n_tiles > 0x3fffffff) return PQ_ERR_SHAPE;

  // Aim at two resident CTAs per SM; the split is the cluster size (<= 8) and <= K blocks.
  const int64_t units = n_tiles * m_blocks;   // (channel tile, token block) pairs, each split over a cluster
  int splits = static_cast<int>((2 * sm_count()) / units);
  splits = splits < 1 ? 1 : (splits > kMaxSplit ? kMaxSplit : splits);
  // Variants with two CTAs per SM have no room to spare: a cluster has to fit one GPC, so a grid that
  // nearly fills the device leaves clusters for a second wave (2048 -> 6144 at M = 64: 12.8 us with
  // clusters of 6, 7.4 us with clusters of 4).  Stay below 90 % of the resident capacity, and off the
  // cluster sizes 5 and 7.
  const int ctas_per_sm = (kW4 && mpad > 64) ? 1 : (mpad >= 64 ? 2 : (kW4 ? 2 : 4));
  while (splits > 1 && units * splits * 10 > static_cast<int64_t>(ctas_per_sm) * sm_count() * 9) --splits;
  if (splits == 5 || splits == 7) --splits;
  // ablation knob, read once: force the number of K parts (cluster size)
  static const int force_splits = [] { const char* e = getenv("PQ_SMALLM_SPLITS"); return e ? atoi(e) : 0; }();
  if (force_splits >= 1 && force_splits <= kMaxSplit) splits = force_splits;
  if (splits > k_blocks) splits = k_blocks;

  a.count = count;
  a.s_tok = s_tok;
  a.acc = acc;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.K = static_cast<int>(K);
  a.k_blocks = k_blocks;
  a.splits = splits;
  a.wait_limit = wait_limit();
  const bool ex = acc != nullptr;
  const int nt = static_cast<int>(n_tiles);
  switch (mpad) {
    case 16: return ex ? launch_cfg<16, kW4, true>(maps, tq, a, nt, m_blocks, stream) : launch_cfg<16, kW4, false>(maps, tq, a, nt, m_blocks, stream);
    case 32: return ex ? launch_cfg<32, kW4, true>(maps, tq, a, nt, m_blocks, stream) : launch_cfg<32, kW4, false>(maps, tq, a, nt, m_blocks, stream);
    case 64: return ex ? launch_cfg<64, kW4, true>(maps, tq, a, nt, m_blocks, stream) : launch_cfg<64, kW4, false>(maps, tq, a, nt, m_blocks, stream);
    default: return ex ? launch_cfg<128, kW4, true>(maps, tq, a, nt, m_blocks, stream) : launch_cfg<128, kW4, false>(maps, tq, a, nt, m_blocks, stream);
  }
}

}  // namespace

int launch_smallm_w8a8_group(const int8_t* q, const float* s_tok, int count, const void* const* wq,
                             const float* const* s_ch, const int64_t* N, void* const* y, int64_t M, int64_t K,
                             int32_t* acc, cudaStream_t stream) {
  return launch_smallm<false>(q, s_tok, count, wq, s_ch, nullptr, N, y, M, K, acc, stream);
}

int launch_smallm_w4a8_group(const int8_t* q, const float* s_tok, int count, const void* const* wp,
                             const void* const* s_grp, const int64_t* N, void* const* y, int64_t M, int64_t K,
                             int32_t* acc_g, cudaStream_t stream) {
  return launch_smallm<true>(q, s_tok, count, wp, nullptr, s_grp, N, y, M, K, acc_g, stream);
}

int launch_smallm_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M,
                       int64_t N, int64_t K, void* y, int32_t* acc, cudaStream_t stream) {
  return launch_smallm_w8a8_group(q, s_tok, 1, &wq, &s_ch, &N, &y, M, K, acc, stream);
}

int launch_smallm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M,
                       int64_t N, int64_t K, void* y, int32_t* acc_g, cudaStream_t stream) {
  return launch_smallm_w4a8_group(q, s_tok, 1, &wp, &s_grp, &N, &y, M, K, acc_g, stream);
}

}  // namespace pq
