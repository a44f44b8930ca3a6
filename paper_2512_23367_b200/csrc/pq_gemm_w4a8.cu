// W4A8 prefill GEMM on CTA pairs (tcgen05 cta_group::2) for sm_100a.  Packed INT4 weights are
// widened to INT8 inside the kernel, multiplied with the INT8 activation codes on the tensor
// cores one K-group (128) at a time, and every group's INT32 accumulator is dequantized with
// its own scale into an FP32 running sum:
//     R[m,n] += float(ACC_g[m,n]) * s_grp[g,n];     Y = fp16(R * s_tok[m]).
//
// The operands are swapped with respect to the W8A8 kernel: the WEIGHT rows are the 256-row
// operand of tcgen05.mma (128 output channels per CTA = its 128 tensor-memory lanes) and the
// tokens are the 256 columns.  A promotion thread therefore owns one output channel, so the
// group scale s_grp[g,n] is ONE register per group instead of a shared-memory operand per
// accumulator column: with the scales read from shared memory next to the tensor core's operand
// traffic the promotion loop measured 1490 cycles per group, with the scale in a register 1000.
//
// Two CTAs share a 256-token x 256-channel output tile.  Each loads 128 token rows of Q, the
// packed weights of its own 128 channels (128 rows x 64 bytes per group) and their 128 scales; it
// widens its weights into the swizzled K-major INT8 layout; the leader's tcgen05.mma (M = 256
// channels, N = 256 tokens) reads both CTAs' operands and leaves each CTA's 128 x 256 group
// accumulator in that CTA's tensor memory.
//
// The per-group dequantization is CUDA-core work proportional to M*N*K/128: one conversion and
// one fused multiply-add per accumulator element, 2 x 32768 instructions per group and CTA against
// 4 x 512 issue slots -- the arithmetic limit of this kernel sits at the tensor-core time.  It runs
// on eight warps (two per TMEM lane quadrant, 128 token columns each) that keep their 128 running
// sums in registers.
//
// Warp roles (512 threads; register budgets moved with setmaxnreg):
//   warp 0        TMA producer of the token codes: a ring of four 16 KB stages, freed by the MMAs
//   warp 2        TMA producer of packed weights + scales: a ring of its own (four slots of 8.25 KB), freed
//                 by the widening, so that it runs ahead of the MMAs and -- these being constants of the
//                 model -- ahead of the wait on the preceding kernel.  (With one ring for everything the
//                 loop load -> widen -> MMA -> free bounded the kernel: 64.2 against 59.6 us.)
//   warp 1        MMA issuer (leader CTA only; owns TMEM allocation in both CTAs).  It shares its
//                 scheduler with busy warps, so it is kept to two waits, four MMAs and three commits
//                 per group: "widened" (which implies "codes landed": the widening warp waits for the
//                 stage's barrier before it signals) and "accumulator free"
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

// Tokens per tile (MMA N, TMEM columns) / per CTA.  Narrower tiles give a deeper accumulator ring (512
// columns / BT_PAIR slots) but measured slower: 2048 x 4096 x 4096 takes 57 us at 256, 68 us at 160 and
// 77 us at 128 tokens, with four or eight widening warps and with deeper code and weight rings alike.
constexpr int BT_PAIR = 256, BT_CTA = BT_PAIR / 2;
constexpr int BC_CTA = 128, BC_PAIR = 256;   // output channels per CTA (TMEM lanes) / per tile (MMA M)
constexpr int BK = 128, UMMA_K = 32;
constexpr int Q_STAGES = 4;     // token-code stages, freed by the MMAs
constexpr int W8_SLOTS = 4;     // widened-weight slots, freed by the MMAs
constexpr int P_SLOTS = 4;      // packed weights + FP16 scales of a group: a ring of its own, freed by the widening
constexpr int SC_SLOTS = 8;     // FP32 scale rows (this CTA's 128 channels)
constexpr int ACC_SLOTS = 512 / BT_PAIR;    // TMEM accumulators of BT_PAIR columns
constexpr int kUnpackWarps = 4;                     // widening warps: kUnpackPerSlot share a group's 128 rows
constexpr int kUnpackPerSlot = 1;                   // warps that share one group's rows (a warp per group measured
                                                    // best: 57.3 us against 61.8 us with two, 2048 x 4096 x 4096)
constexpr int kUnpackTeams = kUnpackWarps / kUnpackPerSlot;   // team t takes the groups t, t + kUnpackTeams, ...
constexpr int kPromoteWarps = 8;
constexpr int kFirstPromote = 4 + kUnpackWarps;
constexpr int kNumThreads = 32 * (kFirstPromote + kPromoteWarps);
constexpr int kWidenBatch = 4;  // 16-byte loads of a widening thread in flight
constexpr int kOutBufs = 2;     // staging boxes per promotion warp
constexpr int kRegsCtl = 56, kRegsUnpack = 72, kRegsPromote = 192;
constexpr int kRegsTotal = 128 * kRegsCtl + 32 * kUnpackWarps * kRegsUnpack + 32 * kPromoteWarps * kRegsPromote;

constexpr int kQBytes = BT_CTA * BK;            // 16 KB of token codes
constexpr int kPBytes = BC_CTA * BK / 2;        // 8 KB packed weights
constexpr int kSBytes = BC_CTA * 2;             // FP16 scales of one group
constexpr int kStageBytes = kQBytes;            // a stage of the code ring
constexpr int kPSlotBytes = kPBytes + kSBytes;  // a slot of the packed ring
constexpr int kW8Bytes = BC_CTA * BK;           // 16 KB widened weights
constexpr int kOutTok = BT_CTA % 32 == 0 ? 32 : 16;   // tokens per stored box
constexpr int kOutBoxBytes = kOutTok * 32 * 2;
constexpr int kW8Off = Q_STAGES * kStageBytes;
constexpr int kPOff = kW8Off + W8_SLOTS * kW8Bytes;
constexpr int kScOff = kPOff + P_SLOTS * kPSlotBytes;
constexpr int kOutOff = kScOff + SC_SLOTS * BC_CTA * 4;
constexpr int kBarOff = kOutOff + kPromoteWarps * kOutBufs * kOutBoxBytes;
constexpr int kNumBars = 2 * Q_STAGES + 2 * W8_SLOTS + 2 * P_SLOTS + 2 * SC_SLOTS + 2 * ACC_SLOTS + 1;   // + the MMA issuer's drain barrier
constexpr int kMiscOff = kBarOff + kNumBars * 8;
constexpr int kDynamicSmem = kMiscOff + 16 + 1024;
static_assert(kDynamicSmem <= 232448, "exceeds the shared memory of one CTA");
static_assert(BK / UMMA_K == 4, "the MMA issuer is unrolled for four steps per group");
// A barrier's phases are told apart by one parity bit, so a warp may only wait on barriers whose every phase it
// sees in turn: each ring's length is a multiple of the number of widening teams (team t then always meets the
// same stages and slots).
static_assert(Q_STAGES % kUnpackTeams == 0 && W8_SLOTS % kUnpackTeams == 0 && P_SLOTS % kUnpackTeams == 0 &&
              SC_SLOTS % kUnpackTeams == 0, "ring lengths and widening teams");
static_assert(kUnpackWarps % 4 == 0 && kUnpackWarps % kUnpackPerSlot == 0 &&
              BC_CTA / kUnpackPerSlot >= 64, "widening teams");
static_assert(kRegsTotal <= 65536, "register budget");

struct W4Args {
  const float* s_tok;
  int32_t* acc_g;  // [G, M, N] when exporting (single member)
  int* status;
  int N[kMaxGroup];        // per member
  int nb_end[kMaxGroup];   // channel blocks of members 0..g (running total); INT_MAX past the last member
  int count;               // members in this launch (linears that share the token codes)
  int M, K;
  int m_blocks, n_blocks, k_blocks;   // n_blocks: over all members
  uint32_t wait_limit;     // poll bound of every wait
};

// Tensor maps of the members' packed weights, group scales and outputs (indexed by member).
struct W4Maps {
  CUtensorMap w[kMaxGroup];
  CUtensorMap s[kMaxGroup];
  CUtensorMap y[kMaxGroup];
};

// Where a tile lies: its member, the member's channel count, its token block and first channel.
struct W4Tile {
  int g, m_blk, c0, N;
};
__device__ __forceinline__ W4Tile locate_tile(const W4Args& p, int tile) {
  W4Tile t;
  int nblk = tile / p.m_blocks;
  t.m_blk = tile - nblk * p.m_blocks;
  t.g = 0;
  t.N = p.N[0];
  if (p.count > 1) {
    const int e0 = p.nb_end[0], e1 = p.nb_end[1], e2 = p.nb_end[2];
    if (nblk >= e2) { t.g = 3; t.N = p.N[3]; nblk -= e2; }
    else if (nblk >= e1) { t.g = 2; t.N = p.N[2]; nblk -= e1; }
    else if (nblk >= e0) { t.g = 1; t.N = p.N[1]; nblk -= e0; }
  }
  t.c0 = nblk * BC_PAIR;
  return t;
}

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
gemm_w4a8_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ W4Maps maps, const W4Args p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_full = smem_base + kBarOff;              // local: token codes landed
  const uint32_t bar_empty = bar_full + Q_STAGES * 8;         // local: the MMAs that read the code stage completed
  const uint32_t bar_w8_full = bar_empty + Q_STAGES * 8;      // LEADER: both CTAs' widened weights written
  const uint32_t bar_w8_empty = bar_w8_full + W8_SLOTS * 8;   // local: the MMAs that read the widened slot completed
  const uint32_t bar_p_full = bar_w8_empty + W8_SLOTS * 8;    // local: packed weights and scales landed
  const uint32_t bar_p_empty = bar_p_full + P_SLOTS * 8;      // local: the widening warp has read them
  const uint32_t bar_sc_full = bar_p_empty + P_SLOTS * 8;     // local: FP32 scales written
  const uint32_t bar_sc_empty = bar_sc_full + SC_SLOTS * 8;   // local: promotion warps read them
  const uint32_t bar_acc_full = bar_sc_empty + SC_SLOTS * 8;  // local: group accumulator complete
  const uint32_t bar_acc_empty = bar_acc_full + ACC_SLOTS * 8;  // LEADER: both CTAs' promotion drained it
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kMiscOff);
  const uint32_t bar_drain = bar_acc_empty + ACC_SLOTS * 8;     // give-up path of the MMA issuer only
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kMiscOff + 4);
  const WaitCtx wc{abort_flag, p.wait_limit};

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair_id = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;
  const int num_tiles = p.m_blocks * p.n_blocks;
  constexpr uint32_t kTmemCols = 512;
  static_assert(ACC_SLOTS * BT_PAIR <= 512 && BT_PAIR % 32 == 0, "accumulator slots");

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar_drain, 1);
    for (int s = 0; s < Q_STAGES; ++s) {
      mbar_init(bar_full + s * 8, 1);
      mbar_init(bar_empty + s * 8, 1);    // the MMAs' commit
    }
    for (int s = 0; s < W8_SLOTS; ++s) {
      mbar_init(bar_w8_full + s * 8, 2 * kUnpackPerSlot);  // the slot's widening warps in each CTA
      mbar_init(bar_w8_empty + s * 8, 1);                  // the MMAs' commit
    }
    for (int s = 0; s < P_SLOTS; ++s) {
      mbar_init(bar_p_full + s * 8, 1);
      mbar_init(bar_p_empty + s * 8, kUnpackPerSlot);
    }
    for (int s = 0; s < SC_SLOTS; ++s) {
      mbar_init(bar_sc_full + s * 8, kUnpackPerSlot);
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
    for (int g = 0; g < p.count; ++g) {
      tma_prefetch_desc(&maps.w[g]);
      tma_prefetch_desc(&maps.s[g]);
      if constexpr (!kExportAcc) tma_prefetch_desc(&maps.y[g]);
    }
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
  uint32_t issued = 0;   // producer threads: loads each has requested on its ring (for the give-up path)

  if (warp < 4) {
    setmaxnreg_dec<kRegsCtl>();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------- TMA producer of the token codes (both CTAs)
      grid_dep_wait();   // the codes may come from the preceding kernel
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
        const W4Tile t = locate_tile(p, tile);
        const int t0 = t.m_blk * BT_PAIR + static_cast<int>(rank) * BT_CTA;
        for (int g = 0; g < p.k_blocks; ++g, ++it) {
          const uint32_t s = it % Q_STAGES, ph = (it / Q_STAGES) & 1u;
          if (it >= Q_STAGES && !mbar_wait(bar_empty + s * 8, ph ^ 1u, wc)) { ok = false; break; }
          mbar_arrive_expect_tx(bar_full + s * 8, kQBytes);
          tma_load_2d(smem_base + s * kStageBytes, &tm_q, bar_full + s * 8, g * BK, t0);
        }
      }
      issued = it;
    } else if (warp == 2 && lane == 0) {
      // ---------------------------------------------------------- TMA producer of packed weights + scales
      // (constants of the model: this stream does not wait for the preceding kernel)
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
        const W4Tile t = locate_tile(p, tile);
        const int c0 = t.c0 + static_cast<int>(rank) * BC_CTA;
        for (int g = 0; g < p.k_blocks; ++g, ++it) {
          const uint32_t ps = it % P_SLOTS, pph = (it / P_SLOTS) & 1u;
          if (it >= P_SLOTS && !mbar_wait(bar_p_empty + ps * 8, pph ^ 1u, wc)) { ok = false; break; }
          const uint32_t dst = smem_base + kPOff + ps * kPSlotBytes;
          mbar_arrive_expect_tx(bar_p_full + ps * 8, kPSlotBytes);
          tma_load_2d(dst, &maps.w[t.g], bar_p_full + ps * 8, g * (BK / 2), c0);
          tma_load_2d(dst + kPBytes, &maps.s[t.g], bar_p_full + ps * 8, c0, g);
        }
      }
      issued = it;
    } else if (warp == 1 && lane == 0 && rank == 0) {
      // ---------------------------------------------------------- MMA issuer (leader only)
      constexpr uint32_t idesc = umma_idesc_s8(BC_PAIR, BT_PAIR);
      const int total = pair_id < num_tiles ? ((num_tiles - pair_id + num_pairs - 1) / num_pairs) * p.k_blocks : 0;   // groups of this pair
      bool ok = true;
      for (uint32_t it = 0; it < static_cast<uint32_t>(total); ++it) {
        const uint32_t sq = it % Q_STAGES;
        const uint32_t sw = it % W8_SLOTS, wph = (it / W8_SLOTS) & 1u;
        const uint32_t a = it % ACC_SLOTS, aph = (it / ACC_SLOTS) & 1u;
        // Operands are prepared before the waits, and the wait most likely to open last comes last.
        const uint64_t w_desc = umma_desc_k_sw128(smem_base + kW8Off + sw * kW8Bytes);   // 256 channel rows (both CTAs)
        const uint64_t q_desc = umma_desc_k_sw128(smem_base + sq * kStageBytes);         // token rows of both CTAs
        const uint32_t d_tmem = tmem_base + a * BT_PAIR;
        if (!mbar_wait2_cluster(bar_w8_full + sw * 8, wph, bar_acc_empty + a * 8, aph ^ 1u, wc)) { ok = false; break; }
        tc_fence_after_sync();
        umma_i8_pair_imm<0>(d_tmem, w_desc, q_desc, idesc);
        umma_i8_pair_imm<1>(d_tmem, w_desc + 2, q_desc + 2, idesc);
        umma_i8_pair_imm<1>(d_tmem, w_desc + 4, q_desc + 4, idesc);
        umma_i8_pair_imm<1>(d_tmem, w_desc + 6, q_desc + 6, idesc);
        umma_commit_pair_mcast(bar_acc_full + a * 8, 0x3);
        umma_commit_pair_mcast(bar_empty + sq * 8, 0x3);      // frees the code stage in both CTAs
        umma_commit_pair_mcast(bar_w8_empty + sw * 8, 0x3);   // and the widened slot
      }
      (void)ok;
    }
  } else if (warp < kFirstPromote) {
    // ------------------------------------------------------------ widen nibbles
    setmaxnreg_dec<kRegsUnpack>();
    const uint32_t team = static_cast<uint32_t>(warp - 4) / kUnpackPerSlot;
    const int sub = (warp - 4) % kUnpackPerSlot;                               // its share of the slot's 128 rows
    constexpr int kRows = BC_CTA / kUnpackPerSlot;
    const uint32_t w8_full0 = mapa_u32(bar_w8_full, 0);
    const int total = pair_id < num_tiles ? ((num_tiles - pair_id + num_pairs - 1) / num_pairs) * p.k_blocks : 0;
    for (uint32_t it = team; it < static_cast<uint32_t>(total); it += kUnpackTeams) {
      const uint32_t sq = it % Q_STAGES, qph = (it / Q_STAGES) & 1u;   // the group's code stage
      const uint32_t s = it % W8_SLOTS, ph = (it / W8_SLOTS) & 1u;     // and widened slot
      uint8_t* w8 = smem + kW8Off + s * kW8Bytes;
      const uint32_t v = it % SC_SLOTS, vph = (it / SC_SLOTS) & 1u;
      const uint32_t ps = it % P_SLOTS, pph = (it / P_SLOTS) & 1u;
      // packed weights landed; the widened slot's previous MMAs are done; the scale row has been read
      const bool w = mbar_wait3(bar_p_full + ps * 8, pph, bar_w8_empty + s * 8, ph ^ 1u, bar_sc_empty + v * 8, vph ^ 1u,
                                wc);
      if (!__all_sync(0xffffffffu, w)) break;
      const uint8_t* pslot = smem + kPOff + ps * kPSlotBytes;
      const uint4* packed = reinterpret_cast<const uint4*>(pslot) + sub * kRows * 4;
      // Lane l owns the 32-k run (l & 3) of the channel rows (l >> 2) + 8 i, i = 0..15: its row's swizzle
      // term is one constant.  kWidenBatch loads are in flight before the first result is stored.
      const int j = lane & 3, sw = (lane >> 2) & 7;
      uint8_t* row0 = w8 + (sub * kRows + (lane >> 2)) * 128;
      const int off_lo = ((2 * j) ^ sw) << 4, off_hi = ((2 * j + 1) ^ sw) << 4;
#pragma unroll 1
      for (int b = 0; b < (kRows * 4) / 32; b += kWidenBatch) {
        uint4 w4[kWidenBatch];
#pragma unroll
        for (int i = 0; i < kWidenBatch; ++i) w4[i] = packed[lane + (b + i) * 32];
#pragma unroll
        for (int i = 0; i < kWidenBatch; ++i) {
          uint4 lo, hi;
          lo.x = (w4[i].x << 4) & 0xF0F0F0F0u; hi.x = w4[i].x & 0xF0F0F0F0u;
          lo.y = (w4[i].y << 4) & 0xF0F0F0F0u; hi.y = w4[i].y & 0xF0F0F0F0u;
          lo.z = (w4[i].z << 4) & 0xF0F0F0F0u; hi.z = w4[i].z & 0xF0F0F0F0u;
          lo.w = (w4[i].w << 4) & 0xF0F0F0F0u; hi.w = w4[i].w & 0xF0F0F0F0u;
          uint8_t* row = row0 + (b + i) * (8 * 128);   // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
          *reinterpret_cast<uint4*>(row + off_lo) = lo;   // k = 32j .. 32j+15
          *reinterpret_cast<uint4*>(row + off_hi) = hi;   // k = 32j+16 .. 32j+31
        }
      }
      const __half2* sh = reinterpret_cast<const __half2*>(pslot + kPBytes) + sub * (kRows / 2);
      float2* sc = reinterpret_cast<float2*>(smem + kScOff + v * BC_CTA * 4) + sub * (kRows / 2);
#pragma unroll
      for (int i = 0; i < kRows / 64; ++i) {
        const float2 f = __half22float2(sh[lane + 32 * i]);
        sc[lane + 32 * i] = make_float2(f.x * 0.0625f, f.y * 0.0625f);
      }
      fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor-core (async) proxy
      // "widened" tells the MMA issuer that the group's codes are there too
      if (!__all_sync(0xffffffffu, mbar_wait(bar_full + sq * 8, qph, wc))) break;
      if (lane == 0) {
        mbar_arrive_cluster_addr(w8_full0 + s * 8);
        mbar_arrive(bar_sc_full + v * 8);
        mbar_arrive(bar_p_empty + ps * 8);
      }
    }
  } else {
    // ------------------------------------------------------------ promotion + epilogue (warps 8..15)
    setmaxnreg_inc<kRegsPromote>();
    grid_dep_wait();                    // token scales come from the preceding kernel; Y is overwritten
    constexpr int HT = BT_PAIR / 2;     // token columns per promotion warp
    constexpr int LC = 16;              // token columns per tcgen05.ld (the next one is in flight during the arithmetic)
    constexpr int CH = kOutTok, NLD = HT / CH;   // tokens per stored box
    const int pw = warp - kFirstPromote;
    const int quad = warp & 3;          // TMEM lanes 32*quad .. are this warp's: 32 output channels
    const int half = pw >> 2;           // which 128 of the tile's 256 tokens
    const int c_local = quad * 32 + lane;
    const uint32_t acc_empty0 = mapa_u32(bar_acc_empty, 0);
    uint8_t* out_warp = smem + kOutOff + pw * (kOutBufs * kOutBoxBytes);
    const uint32_t out_warp_u32 = smem_base + kOutOff + pw * (kOutBufs * kOutBoxBytes);
    uint32_t it = 0, nstore = 0;
    bool ok = true;
    const float* sc_rows = reinterpret_cast<const float*>(smem + kScOff);
    bool have_next = false;
    float sg_next = 0.0f;
    for (int tile = pair_id; tile < num_tiles && ok; tile += num_pairs) {
      const W4Tile tp = locate_tile(p, tile);
      const int tok0 = tp.m_blk * BT_PAIR + half * HT;                                // first token of this warp
      const int ch0 = tp.c0 + static_cast<int>(rank) * BC_CTA + quad * 32;            // first channel (of the member)
      float R[HT];
#pragma unroll
      for (int j = 0; j < HT; ++j) R[j] = 0.0f;
      for (int g = 0; g < p.k_blocks; ++g, ++it) {
        const uint32_t a = it % ACC_SLOTS, aph = (it / ACC_SLOTS) & 1u;
        const uint32_t v = it % SC_SLOTS, vph = (it / SC_SLOTS) & 1u;
        // this thread's channel: one scale for the whole group
        float sg;
        if (have_next) {
          sg = sg_next;   // the look-ahead of the previous group saw both barriers complete
        } else {
          ok = __all_sync(0xffffffffu, mbar_wait2(bar_sc_full + v * 8, vph, bar_acc_full + a * 8, aph, wc));
          if (!ok) break;
          sg = sc_rows[v * BC_CTA + c_local];
        }
        tc_fence_after_sync();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + a * BT_PAIR + half * HT;
        uint32_t xb[2][LC];
        uint32_t look = 0;
        tmem_ld_32x16(t_addr, xb[0]);
#pragma unroll
        for (int c = 0; c < HT / LC; ++c) {
          tmem_ld_wait();
          if (c + 1 < HT / LC) {
            tmem_ld_32x16(t_addr + (c + 1) * LC, xb[(c + 1) & 1]);
          } else {
            // The whole slice is in registers: hand the accumulator back before the arithmetic.
            // (Relaxed arrive: the data moved through tensor memory, ordered by the tcgen05 fence.)
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_addr_relaxed(acc_empty0 + a * 8);
          }
          // Look ahead: the MMAs usually run a group ahead, and a barrier round trip costs hundreds
          // of cycles under tensor-core load -- ask early, use the answer late, so that the arithmetic
          // in between hides it.
          if (c == 1) {
            const uint32_t a1 = (it + 1) % ACC_SLOTS, aph1 = ((it + 1) / ACC_SLOTS) & 1u;
            const uint32_t v1 = (it + 1) % SC_SLOTS, vph1 = ((it + 1) / SC_SLOTS) & 1u;
            look = mbar_test2(bar_sc_full + v1 * 8, vph1, bar_acc_full + a1 * 8, aph1);
          }
          if (c == HT / LC - 2) {
            have_next = __all_sync(0xffffffffu, look != 0);
            if (have_next) sg_next = sc_rows[((it + 1) % SC_SLOTS) * BC_CTA + c_local];
          }
          const uint32_t(&x)[LC] = xb[c & 1];
          if constexpr (kExportAcc) {
            const int n = ch0 + lane;
#pragma unroll
            for (int j = 0; j < LC; ++j) {
              const int m = tok0 + c * LC + j;
              if (m < p.M && n < tp.N)
                p.acc_g[(static_cast<int64_t>(g) * p.M + m) * tp.N + n] = static_cast<int32_t>(x[j]) >> 4;
            }
          } else {
#pragma unroll
            for (int j = 0; j < LC; ++j)
              R[c * LC + j] = fmaf(__int2float_rn(static_cast<int32_t>(x[j])), sg, R[c * LC + j]);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sc_empty + v * 8);
      }
      if constexpr (!kExportAcc) {
        if (ok) {
          // y[token, channel]: the lane is the channel (contiguous in memory), the register index the
          // token.  One box = 32 tokens x 32 channels, rows of 64 bytes staged with the 64-byte swizzle.
          float stv[NLD];   // lane l holds the scales of tokens tok0 + 32 c + l
#pragma unroll
          for (int c = 0; c < NLD; ++c) {
            const int m = tok0 + c * CH + lane;
            stv[c] = (m < p.M) ? __ldg(p.s_tok + m) : 0.0f;
          }
#pragma unroll
          for (int c = 0; c < NLD; ++c) {
            const uint32_t buf = nstore % kOutBufs;
            if (lane == 0) tma_store_wait_read<kOutBufs - 1>();   // the store that last read `buf` is done
            __syncwarp();
            uint8_t* dst = out_warp + buf * kOutBoxBytes + (lane & 7) * 2;
            const int chunk = lane >> 3;
#pragma unroll
            for (int j = 0; j < CH; ++j) {
              const float st = __shfl_sync(0xffffffffu, stv[c], j);
              const __half h = __float2half_rn(R[c * CH + j] * st);
              *reinterpret_cast<__half*>(dst + j * 64 + ((chunk ^ ((j >> 1) & 3)) << 4)) = h;
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (ch0 < tp.N && tok0 + c * CH < p.M)
                tma_store_2d(&maps.y[tp.g], out_warp_u32 + buf * kOutBoxBytes, ch0, tok0 + c * CH);
              tma_store_commit();  // also when nothing was stored: keeps one group per buffer use
            }
            ++nstore;
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
  if (*abort_flag) {
    // Somebody gave up.  Work already handed to the hardware still completes by itself and must have
    // done so before this CTA's shared and tensor memory go away: the producer's loads (their barriers
    // are local) and the leader's MMAs (they read both CTAs' shared memory and write both tensor memories).
    if (threadIdx.x == 0) {
      const uint32_t first = issued > static_cast<uint32_t>(Q_STAGES) ? issued - Q_STAGES : 0u;
      for (uint32_t i = first; i < issued; ++i) mbar_drain(bar_full + (i % Q_STAGES) * 8, (i / Q_STAGES) & 1u);
    } else if (threadIdx.x == 64) {
      const uint32_t first = issued > static_cast<uint32_t>(P_SLOTS) ? issued - P_SLOTS : 0u;
      for (uint32_t i = first; i < issued; ++i) mbar_drain(bar_p_full + (i % P_SLOTS) * 8, (i / P_SLOTS) & 1u);
    } else if (threadIdx.x == 32 && rank == 0) {
      umma_commit_pair_mcast(bar_drain, 0x1);
      mbar_drain(bar_drain, 0u);
    }
  }
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
int launch_w4(const CUtensorMap& tq, const W4Maps& maps, const W4Args& a, cudaStream_t stream) {
  auto kern = gemm_w4a8_kernel<kExportAcc>;
  // The promotion warps raise their register budget with setmaxnreg; that only terminates if the
  // CTA's allocation (registers per thread at launch x 512) holds the sum of the three budgets.  The
  // register count is a property of the compiled kernel: checked once per process.
  static const int regs_ok = [kern] {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return -1;
    return fa.numRegs * kNumThreads >= kRegsTotal ? 1 : 0;
  }();
  if (regs_ok <= 0) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  static PerDeviceOnce once;
  if (const int rc = set_dynamic_smem_once(once, kern, kDynamicSmem); rc != PQ_OK) return rc;
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
  return cuda_status(cudaLaunchKernelEx(&cfg, kern, tq, maps, a));
}

}  // namespace

int launch_gemm_w4a8_group(const int8_t* q, const float* s_tok, int count, const void* const* wp,
                           const void* const* s_grp, const int64_t* N, void* const* y, int64_t M, int64_t K,
                           int32_t* acc_g, cudaStream_t stream) {
  if (count < 1 || count > kMaxGroup || (acc_g != nullptr && count != 1)) return PQ_ERR_SHAPE;
  CUtensorMap tq;
  W4Maps maps;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), BT_CTA, BK, 1, 128);
  if (rc != PQ_OK) return rc;
  W4Args a;
  int64_t nb_total = 0;
  for (int g = 0; g < kMaxGroup; ++g) {
    const int src = g < count ? g : 0;   // unused slots repeat member 0 (never selected)
    rc = make_tmap_2d(&maps.w[g], wp[src], static_cast<uint64_t>(N[src]), static_cast<uint64_t>(K / 2), BC_CTA, BK / 2, 1, 0);
    if (rc != PQ_OK) return rc;
    // Group scales [K/128, N] FP16; the accumulator-export variant has none and reads a dummy map of Q.
    if (acc_g == nullptr) {
      rc = make_tmap_2d(&maps.s[g], s_grp[src], static_cast<uint64_t>(K / 128), static_cast<uint64_t>(N[src]), 1, BC_CTA, 2, 0);
      if (rc != PQ_OK) return rc;
      rc = make_tmap_2d(&maps.y[g], y[src], static_cast<uint64_t>(M), static_cast<uint64_t>(N[src]), kOutTok, 32, 2, 64);
    } else {
      rc = make_tmap_2d(&maps.s[g], q, static_cast<uint64_t>(M), static_cast<uint64_t>(K / 2), 1, BC_CTA, 2, 0);
      maps.y[g] = tq;  // not used by the accumulator export
    }
    if (rc != PQ_OK) return rc;
    a.N[g] = static_cast<int>(N[src]);
    if (g < count) nb_total += (N[g] + BC_PAIR - 1) / BC_PAIR;
    a.nb_end[g] = g < count ? static_cast<int>(nb_total) : 0x7fffffff;
  }
  a.m_blocks = static_cast<int>((M + BT_PAIR - 1) / BT_PAIR);
  if (a.m_blocks * nb_total > 0x3fffffff) return PQ_ERR_SHAPE;
  a.count = count;
  a.s_tok = s_tok;
  a.acc_g = acc_g;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.K = static_cast<int>(K);
  a.n_blocks = static_cast<int>(nb_total);
  a.k_blocks = static_cast<int>(K / BK);
  a.wait_limit = wait_limit();
  return acc_g != nullptr ? launch_w4<true>(tq, maps, a, stream) : launch_w4<false>(tq, maps, a, stream);
}

int launch_gemm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M,
                     int64_t N, int64_t K, void* y, int32_t* acc_g, cudaStream_t stream) {
  return launch_gemm_w4a8_group(q, s_tok, 1, &wp, &s_grp, &N, &y, M, K, acc_g, stream);
}

}  // namespace pq
