// W8A8 prefill GEMM on CTA pairs (tcgen05 cta_group::2) for sm_100a.
//
// Two CTAs of a cluster share one 256 x BN output tile: each loads its own 128 rows of Q and
// only HALF of the weight tile (BN/2 rows); one tcgen05.mma issued by the leader CTA reads both
// halves from the two CTAs' shared memory and writes each CTA's 128 x BN accumulator into that
// CTA's tensor memory.  Per 128 x 256 x 128 step a CTA loads 32 KB instead of the 48 KB a lone
// CTA would need, which keeps the main loop on the tensor-pipe limit instead of the L2 limit.
//
// Roles per CTA:
//   warp 0      TMA producer (its loads are counted on the LEADER's barrier)
//   warp 1      MMA issuer (leader CTA only; also owns TMEM allocation in both CTAs)
//   warps 2..   epilogue for the CTA's own 128 rows: one or two warps per TMEM lane quadrant
//               (two: each takes half of the tile's columns).  tcgen05.ld of the next 32 columns
//               is in flight while the current 32 are dequantized (x token scale x channel
//               scale), converted to FP16 and written to a swizzled staging buffer that a TMA
//               store drains (full 64-byte row segments; ragged edges are clipped by the tensor
//               map).  The accumulator is handed back to the MMA issuer as soon as its last
//               column block is in registers.
// One CTA per SM with two TMEM accumulators: a tile's epilogue overlaps the next tile's main loop.
// The weight tiles of a CTA's first ring pass are requested BEFORE the wait on the preceding
// kernel (weights are constants of the model); everything else comes after it.
//
// Grouped launch: up to kMaxGroup linears that share the token codes (q/k/v, gate/up) run as ONE
// launch.  Their column blocks are concatenated into one tile list, so the persistent scheduler
// fills its waves across the members and the per-launch fixed cost is paid once; every member
// keeps its own weights, channel scales and output tensor.
//
// Split-K (few tiles, long K -- e.g. M = 512): a work unit is (tile, K part).  Every unit writes
// its INT32 partial accumulator to global scratch, fences, and bumps the tile's arrival counter;
// the unit that arrives last adds the other parts to its own accumulator (still in tensor memory)
// and runs the normal dequantizing epilogue.  Nobody waits for anybody, integer addition makes the
// result independent of the arrival order, and the last unit puts the counter back to zero.
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
constexpr int kOutBoxBytes = 32 * 32 * 2;   // one staged store: 32 rows x 32 FP16 columns

struct PairArgs {
  const float* s_tok;
  const float* s_ch[kMaxGroup];   // per member
  int N[kMaxGroup];               // per member
  int nb_end[kMaxGroup];          // column blocks of members 0..g (running total); INT_MAX past the last member
  int count;                      // members in this launch
  int32_t* acc;
  int* status;
  int32_t* ws;              // split-K partial accumulators (global scratch), or nullptr
  unsigned int* counters;   // split-K arrival counters, one per (tile, CTA of the pair); zero between calls
  int M, K;
  int m_blocks, n_blocks, k_blocks;   // n_blocks: over all members
  int splits;               // K is cut into this many parts; 1 = no split
  uint32_t wait_limit;      // poll bound of every wait
};

// Tensor maps of the members' weights and outputs (kernel parameter, indexed by member).
struct PairMaps {
  CUtensorMap w[kMaxGroup];
  CUtensorMap y[kMaxGroup];
};

// Where a tile lies: its member, the member's column count and channel scales, its first column.
struct TilePos {
  int g, m_blk, n0, N;
  const float* s_ch;
};
template <int BN>
__device__ __forceinline__ TilePos locate_tile(const PairArgs& p, int tile) {
  TilePos t;
  int nblk = tile / p.m_blocks;
  t.m_blk = tile - nblk * p.m_blocks;
  t.g = 0;
  t.N = p.N[0];
  t.s_ch = p.s_ch[0];
  if (p.count > 1) {
    // (constant indices: the argument struct stays in the parameter bank)
    const int e0 = p.nb_end[0], e1 = p.nb_end[1], e2 = p.nb_end[2];
    if (nblk >= e2) { t.g = 3; t.N = p.N[3]; t.s_ch = p.s_ch[3]; nblk -= e2; }
    else if (nblk >= e1) { t.g = 2; t.N = p.N[2]; t.s_ch = p.s_ch[2]; nblk -= e1; }
    else if (nblk >= e0) { t.g = 1; t.N = p.N[1]; t.s_ch = p.s_ch[1]; nblk -= e0; }
  }
  t.n0 = nblk * BN;
  return t;
}

template <int BN, int STAGES, int EPI_BUFS, int EPI_WARPS>
struct PairSmem {
  static constexpr int kABytes = BM_CTA * BK;
  static constexpr int kBBytes = (BN / 2) * BK;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kOutOff = STAGES * kStageBytes;                     // staging, 2 KB boxes
  static constexpr int kScaleOff = kOutOff + EPI_WARPS * EPI_BUFS * kOutBoxBytes;
  static constexpr int kBarOff = kScaleOff + 4 * BN * 4;   // each warp's own copy of its columns' scales
  static constexpr int kNumBars = 2 * STAGES + 4 + 1;   // + the MMA issuer's drain barrier
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kDynamic = kMiscOff + 16 + 1024;
  static_assert(kDynamic <= 232448, "exceeds the shared memory of one CTA");
};

template <int BN, int STAGES, int EPI_BUFS, int ACC_BUFS, int EPI_WARPS, int MIN_CTAS, bool kExportAcc>
__global__ void __launch_bounds__(64 + 32 * EPI_WARPS, MIN_CTAS)
gemm_w8a8_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ PairMaps maps,
                      const PairArgs p) {
  using L = PairSmem<BN, STAGES, EPI_BUFS, EPI_WARPS>;
  static_assert(EPI_WARPS == 4 || EPI_WARPS == 8 || EPI_WARPS == 16, "one, two or four epilogue warps per lane quadrant");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  float* s_ch_smem = reinterpret_cast<float*>(smem + L::kScaleOff);
  const uint32_t bar_full = smem_base + L::kBarOff;     // used in the leader: both CTAs' loads landed
  const uint32_t bar_empty = bar_full + STAGES * 8;     // per CTA: the pair's MMAs released the stage
  const uint32_t bar_tfull = bar_empty + STAGES * 8;    // per CTA: accumulator complete
  const uint32_t bar_tempty = bar_tfull + ACC_BUFS * 8;        // used in the leader: both epilogues drained it
  const uint32_t bar_drain = bar_tempty + ACC_BUFS * 8;        // give-up path of the MMA issuer only
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);
  volatile int* fail_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 12);   // split-K epilogue: a warp's wait ran out
  const WaitCtx wc{abort_flag, p.wait_limit};

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();              // 0 = leader, 1 = peer
  const int pair_id = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;
  const int num_tiles = p.m_blocks * p.n_blocks;
  const int num_units = num_tiles * p.splits;     // unit u = (tile u / splits, K part u % splits)
  // (the unsplit case takes no division: these run on single threads ahead of the first load and MMA)
  auto tile_of = [&](int unit) { return p.splits == 1 ? unit : unit / p.splits; };
  auto part_of = [&](int unit) { return p.splits == 1 ? 0 : unit % p.splits; };
  auto kb_begin = [&](int unit) { return p.splits == 1 ? 0 : (p.k_blocks * part_of(unit)) / p.splits; };
  auto kb_end = [&](int unit) { return p.splits == 1 ? p.k_blocks : (p.k_blocks * (part_of(unit) + 1)) / p.splits; };
  constexpr uint32_t kTmemCols = ACC_BUFS * BN;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    *fail_flag = 0;
    mbar_init(bar_drain, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + s * 8, 1);    // the leader's producer posts the byte count of BOTH CTAs
      mbar_init(bar_empty + s * 8, 1);
    }
    for (int b = 0; b < ACC_BUFS; ++b) {
      mbar_init(bar_tfull + b * 8, 1);
      mbar_init(bar_tempty + b * 8, 2 * EPI_WARPS);  // the epilogue warps of both CTAs
    }
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    for (int g = 0; g < p.count; ++g) {
      tma_prefetch_desc(&maps.w[g]);
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

  // Everything above touched no global data.  The successor kernel may start its own set-up now.
  grid_dep_launch();
  uint32_t issued = 0;   // producer thread: ring passes it has requested (for the give-up path)

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      const uint32_t full0 = mapa_u32(bar_full, 0);  // the leader's ring of "stage landed" barriers
      // First ring pass of the first tile: weights before the wait on the preceding kernel, the
      // codes it may have produced after it.  (Only the leader arrives on the barrier -- a plain
      // CTA-scope arrive; the peer's bytes may land first, the transaction count then runs
      // negative until the leader's expect_tx, which is allowed.)
      int pre = 0;
      if (pair_id < num_units) {
        const int kb0 = kb_begin(pair_id), nkb = kb_end(pair_id) - kb0;
        pre = nkb < STAGES ? nkb : STAGES;
        const TilePos tp = locate_tile<BN>(p, tile_of(pair_id));
        const int n0 = tp.n0 + static_cast<int>(rank) * (BN / 2);
        for (int j = 0; j < pre; ++j) {
          if (rank == 0) mbar_arrive_expect_tx(bar_full + j * 8, 2 * L::kStageBytes);
          tma_load_2d_pair(smem_base + j * L::kStageBytes + L::kABytes, &maps.w[tp.g], full0 + j * 8, (kb0 + j) * BK, n0);
        }
      }
      grid_dep_wait();
      if (pair_id < num_units) {
        const int tile = tile_of(pair_id), kb0 = kb_begin(pair_id);
        const int m0 = (tile % p.m_blocks) * BM_PAIR + static_cast<int>(rank) * BM_CTA;
        for (int j = 0; j < pre; ++j)
          tma_load_2d_pair(smem_base + j * L::kStageBytes, &tm_q, full0 + j * 8, (kb0 + j) * BK, m0);
      }
      uint32_t it = static_cast<uint32_t>(pre);
      bool ok = true;
      for (int unit = pair_id; unit < num_units && ok; unit += num_pairs) {
        const TilePos tp = locate_tile<BN>(p, tile_of(unit));
        const int m0 = tp.m_blk * BM_PAIR + static_cast<int>(rank) * BM_CTA;
        const int n0 = tp.n0 + static_cast<int>(rank) * (BN / 2);
        const CUtensorMap* tm_w = &maps.w[tp.g];
        const int kb1 = kb_end(unit);
        for (int kb = kb_begin(unit) + (unit == pair_id ? pre : 0); kb < kb1; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_empty + s * 8, ph ^ 1u, wc)) { ok = false; break; }
          const uint32_t dst = smem_base + s * L::kStageBytes;
          if (rank == 0) mbar_arrive_expect_tx(bar_full + s * 8, 2 * L::kStageBytes);
          tma_load_2d_pair(dst, &tm_q, full0 + s * 8, kb * BK, m0);
          tma_load_2d_pair(dst + L::kABytes, tm_w, full0 + s * 8, kb * BK, n0);
        }
      }
      issued = it;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_s8(BM_PAIR, BN);
      uint32_t it = 0, t = 0;
      bool ok = true;
      for (int unit = pair_id; unit < num_units && ok; unit += num_pairs, ++t) {
        const uint32_t b = t % ACC_BUFS;
        if (!mbar_wait(bar_tempty + b * 8, ((t / ACC_BUFS) & 1u) ^ 1u, wc)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + b * BN;
        const int kb0 = kb_begin(unit), kb1 = kb_end(unit);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(bar_full + s * 8, ph, wc)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_base + s * L::kStageBytes;
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + L::kABytes);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_i8_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb != kb0 || k != 0) ? 1u : 0u);
          umma_commit_pair_mcast(bar_empty + s * 8, 0x3);   // frees the stage in both CTAs
        }
        if (ok) umma_commit_pair_mcast(bar_tfull + b * 8, 0x3);  // accumulator ready in both CTAs
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2.., both CTAs)
    grid_dep_wait();                       // token scales come from the preceding kernel; Y is overwritten
    constexpr int HC = BN / (EPI_WARPS / 4);   // columns per epilogue warp
    constexpr int NCH = HC / 32;           // 32-column blocks per warp and tile
    const int e = warp - 2;
    const int quad = warp & 3;             // TMEM lanes 32*quad .. 32*quad+31 are this warp's
    const int half = e >> 2;               // which part of the tile's columns
    float* sc_warp = s_ch_smem + e * HC;
    uint8_t* out_warp = smem + L::kOutOff + e * (EPI_BUFS * kOutBoxBytes);
    const uint32_t out_warp_u32 = smem_base + L::kOutOff + e * (EPI_BUFS * kOutBoxBytes);
    const uint32_t tempty0 = mapa_u32(bar_tempty, 0);
    const int sw = (lane >> 1) & 3;        // 64-byte swizzle: 16-byte chunk index XOR (row / 2) mod 4
    uint32_t t = 0, nstore = 0;
    bool ok = true;
    volatile int* last_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 8);
    for (int unit = pair_id; unit < num_units && ok; unit += num_pairs, ++t) {
      const int tile = tile_of(unit);
      const TilePos tp = locate_tile<BN>(p, tile);
      const uint32_t b = t % ACC_BUFS;
      const int row0 = tp.m_blk * BM_PAIR + static_cast<int>(rank) * BM_CTA + quad * 32;
      const int n0 = tp.n0 + half * HC;
      const int row = row0 + lane;
      float st = 0.0f;
      if constexpr (!kExportAcc) {
        __syncwarp();
        for (int c = lane; c < HC; c += 32) sc_warp[c] = (n0 + c < tp.N) ? __ldg(tp.s_ch + n0 + c) : 0.0f;
        if (row < p.M) st = __ldg(p.s_tok + row);
        __syncwarp();
      }
      const bool got = __all_sync(0xffffffffu, mbar_wait(bar_tfull + b * 8, (t / ACC_BUFS) & 1u, wc));
      const bool split_unit = !kExportAcc && p.splits > 1;
      // Without a K split a warp that gave up just leaves.  With one, the epilogue warps of the CTA meet
      // at named barriers below, so they decide TOGETHER: every warp reaches the first barrier whatever
      // its own wait said, and all leave after it if any of them failed.
      if (!got && !split_unit) { ok = false; break; }
      if (got) tc_fence_after_sync();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + b * BN + half * HC;
      // Split-K: this CTA's slice of the tile's partials, one slot per K part.  The scratch is
      // private, so it is laid out for coalescing: [4-column piece][row] of 16-byte words -- a warp's
      // store of one piece covers 512 contiguous bytes.
      const int sp = part_of(unit);
      const int64_t slot_elems = static_cast<int64_t>(BM_CTA) * BN;
      uint4* ws_tile = nullptr;
      if constexpr (!kExportAcc) {
        if (p.splits > 1) {
          ws_tile = reinterpret_cast<uint4*>(p.ws + (static_cast<int64_t>(tile) * 2 + rank) * p.splits * slot_elems) +
                    static_cast<int64_t>(half * (HC / 4)) * BM_CTA + (quad * 32 + lane);
          uint4* mine = ws_tile + sp * (slot_elems / 4);
          if (!got) {
            if (lane == 0) *fail_flag = 1;
          } else {
#pragma unroll 1
            for (int c = 0; c < NCH; ++c) {
              uint32_t v[32];
              tmem_ld_32x32(t_addr + c * 32, v);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                __stcg(mine + (c * 8 + j / 4) * BM_CTA, make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]));
            }
          }
          __threadfence();                               // the partial is visible before the arrival
          named_bar_sync(1, EPI_WARPS * 32);
          if (warp == 2 && lane == 0) {
            int last = 0;
            if (*fail_flag == 0) {
              unsigned int* ctr = p.counters + (tile * 2 + static_cast<int>(rank));
              const unsigned int old = atomicAdd(ctr, 1u);
              last = (old == static_cast<unsigned int>(p.splits - 1));
              if (last) *ctr = 0u;                       // nobody else touches it in this call; zero for the next
            }
            *last_flag = last;
          }
          named_bar_sync(1, EPI_WARPS * 32);
          if (*fail_flag != 0) { ok = false; break; }    // the same answer in every warp
          const bool last = *last_flag != 0;
          __threadfence();                               // the other parts' partials are read after the arrival count
          if (!last) {
            // Not the last part of this tile: the accumulator is saved, hand it back and move on.
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_addr_relaxed(tempty0 + b * 8);
            continue;
          }
        }
      }
      uint32_t r[2][32];
      tmem_ld_32x32(t_addr, r[0]);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        tmem_ld_wait();
        if (c + 1 < NCH) {
          tmem_ld_32x32(t_addr + (c + 1) * 32, r[(c + 1) & 1]);
        } else {
          // The whole slice is in registers: hand the accumulator back before the arithmetic.
          // (Relaxed arrive: the data moved through tensor memory, ordered by the tcgen05 fence; a
          // release at cluster scope would cost a full memory barrier here.)
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_addr_relaxed(tempty0 + b * 8);
        }
        uint32_t(&v)[32] = r[c & 1];
        const int col0 = n0 + c * 32;
        if constexpr (!kExportAcc) {
          if (p.splits > 1) {
            // add the other K parts (exact integer sums; read through L2, where they were written)
            for (int o = 0; o < p.splits; ++o) {
              if (o == sp) continue;
              const uint4* theirs = ws_tile + o * (slot_elems / 4) + c * 8 * BM_CTA;
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                const uint4 w4 = __ldcg(theirs + (j / 4) * BM_CTA);
                v[j] += w4.x; v[j + 1] += w4.y; v[j + 2] += w4.z; v[j + 3] += w4.w;
              }
            }
          }
        }
        if constexpr (kExportAcc) {
          if (row < p.M) {
            int32_t* dst = p.acc + static_cast<int64_t>(row) * tp.N + col0;   // export: single member
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              if (col0 + j < tp.N) *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            }
          }
        } else {
          const uint32_t buf = nstore % EPI_BUFS;
          if (lane == 0) tma_store_wait_read<EPI_BUFS - 1>();  // the store that last read `buf` is done
          __syncwarp();
          const float* sc = sc_warp + c * 32;
          uint8_t* dst = out_warp + buf * kOutBoxBytes + lane * 64;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 s2 = *reinterpret_cast<const float2*>(sc + 8 * j + 2 * i);
              const float v0 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int32_t>(v[8 * j + 2 * i])), st), s2.x);
              const float v1 = __fmul_rn(__fmul_rn(__int2float_rn(static_cast<int32_t>(v[8 * j + 2 * i + 1])), st), s2.y);
              const __half2 h = __floats2half2_rn(v0, v1);
              o[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
            *reinterpret_cast<uint4*>(dst + ((j ^ sw) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (col0 < tp.N && row0 < p.M) tma_store_2d(&maps.y[tp.g], out_warp_u32 + buf * kOutBoxBytes, col0, row0);
            tma_store_commit();  // also when nothing was stored: keeps one group per buffer use
          }
          ++nstore;
        }
      }
    }
    if constexpr (!kExportAcc) {
      // The staging buffers must outlive the stores' reads; the writes themselves complete with
      // the kernel.
      if (lane == 0) tma_store_wait_read<0>();
    }
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*abort_flag) {
    // Somebody gave up.  Work already handed to the hardware still completes by itself and must have
    // done so before this CTA's shared and tensor memory go away:
    if (threadIdx.x == 0) {
      // loads requested by this CTA's producer.  The leader sees them on its "stage landed" barriers;
      // the peer's loads are counted on the leader's barriers too, which it cannot poll -- it waits a
      // time that covers any load in flight.
      if (rank == 0) {
        const uint32_t first = issued > static_cast<uint32_t>(STAGES) ? issued - STAGES : 0u;
        for (uint32_t i = first; i < issued; ++i) mbar_drain(bar_full + (i % STAGES) * 8, (i / STAGES) & 1u);
      } else {
        drain_sleep_us(100);
      }
    } else if (threadIdx.x == 32 && rank == 0) {
      // MMAs issued by the leader (they read both CTAs' shared memory and write both tensor memories)
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

template <int BN, int STAGES, int EPI_BUFS, int ACC_BUFS, int EPI_WARPS, int MIN_CTAS, bool kExportAcc>
int launch_pair_cfg(const CUtensorMap& tq, const PairMaps& maps, const PairArgs& a, cudaStream_t stream) {
  using L = PairSmem<BN, STAGES, EPI_BUFS, EPI_WARPS>;
  static_assert(MIN_CTAS * (L::kDynamic + 1024) <= 233472, "co-resident CTAs exceed the SM's shared memory");
  static_assert(MIN_CTAS * ACC_BUFS * BN <= 512, "co-resident CTAs exceed the SM's tensor memory");
  auto kern = gemm_w8a8_pair_kernel<BN, STAGES, EPI_BUFS, ACC_BUFS, EPI_WARPS, MIN_CTAS, kExportAcc>;
  static PerDeviceOnce once;   // one per kernel variant
  if (const int rc = set_dynamic_smem_once(once, kern, L::kDynamic); rc != PQ_OK) return rc;
  const int units = a.m_blocks * a.n_blocks * a.splits;
  const int max_pairs = MIN_CTAS * (sm_count() / 2);
  const int pairs = units < max_pairs ? units : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs), 1, 1);
  cfg.blockDim = dim3(64 + 32 * EPI_WARPS, 1, 1);
  cfg.dynamicSmemBytes = L::kDynamic;
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

// Plan: tile width (256 or 128 columns) x number of K parts.  Cost of a plan in SM cycles:
//   waves of work units over the SM pairs x (K blocks per unit x cycles per K block + fixed cost
//   of a unit's epilogue, plus the scratch round trip when K is split: ~9000 cycles measured).
// Cycles per K block are measured figures: 512 for a 256-wide tile (the tensor-pipe time), 550
// for a 128-wide one (bound by the bytes each SM pulls per multiply-add, not faster per block).
// `scratch_bytes` = room for split-K partials (0: never split); force_* = 0 means "free choice".
// The members' column counts are N[0..count); a launch of one linear has count = 1.
// Returns the cost of the chosen plan, or -1 if the forced values admit none.
int64_t plan_w8a8_pair_group(int64_t M, const int64_t* N, int count, int64_t K, int sms, size_t scratch_bytes,
                             int force_bn, int force_splits, int* bn_out, int* splits_out) {
  const int pairs = sms / 2 > 0 ? sms / 2 : 1;
  const int64_t mb = (M + BM_PAIR - 1) / BM_PAIR;
  const int64_t kblocks = (K + BK - 1) / BK;
  auto waves = [pairs](int64_t units) { return (units + pairs - 1) / pairs; };
  int64_t n_max = 0;
  for (int g = 0; g < count; ++g) n_max = N[g] > n_max ? N[g] : n_max;
  int64_t best_cost = -1;
  for (int bn = 256; bn >= 128; bn /= 2) {
    if (force_bn != 0 && bn != force_bn) continue;
    if (bn == 256 && n_max <= 128 && force_bn == 0) continue;
    int64_t nb = 0;
    for (int g = 0; g < count; ++g) nb += (N[g] + bn - 1) / bn;
    const int64_t tiles = mb * nb;
    for (int sp = 1; sp <= 4; ++sp) {
      if (force_splits != 0 && sp != force_splits) continue;
      if (sp > 1) {
        if (kblocks / sp < 8) break;
        const size_t need = static_cast<size_t>(tiles) * 2 * sp * BM_CTA * bn * sizeof(int32_t);
        if (need > scratch_bytes || tiles * 2 > kScratchCounters) break;
      }
      const int64_t per_unit = ((kblocks + sp - 1) / sp) * (bn == 256 ? 512 : 550) + (bn == 256 ? 3000 : 1800) +
                               (sp > 1 ? 9000 : 0);   // measured: partial save + fence + reload ~ 4.7 us
      const int64_t cost = waves(tiles * sp) * per_unit;
      if (best_cost < 0 || cost < best_cost) {
        best_cost = cost;
        *bn_out = bn;
        *splits_out = sp;
      }
    }
  }
  return best_cost;
}

int64_t plan_w8a8_pair(int64_t M, int64_t N, int64_t K, int sms, size_t scratch_bytes, int force_bn,
                       int force_splits, int* bn_out, int* splits_out) {
  return plan_w8a8_pair_group(M, &N, 1, K, sms, scratch_bytes, force_bn, force_splits, bn_out, splits_out);
}

// Bytes of split-K partial sums the plan (bn, splits) needs for these members; 0 when K is not split.
size_t w8a8_pair_partial_bytes(int64_t M, const int64_t* N, int count, int bn, int splits) {
  if (splits <= 1) return 0;
  const int64_t mb = (M + BM_PAIR - 1) / BM_PAIR;
  int64_t nb = 0;
  for (int g = 0; g < count; ++g) nb += (N[g] + bn - 1) / bn;
  return static_cast<size_t>(mb * nb) * 2 * splits * BM_CTA * bn * sizeof(int32_t);
}

int launch_gemm_w8a8_pair_group(const Scratch& sc, const int8_t* q, const float* s_tok, int count,
                                const void* const* wq, const float* const* s_ch, const int64_t* N, void* const* y,
                                int64_t M, int64_t K, int32_t* acc, cudaStream_t stream) {
  if (count < 1 || count > kMaxGroup || (acc != nullptr && count != 1)) return PQ_ERR_SHAPE;
  const int64_t mb = (M + BM_PAIR - 1) / BM_PAIR;
  const int64_t kblocks = (K + BK - 1) / BK;
  // ablation knobs, read once per process
  static const int force_bn = [] { const char* e = getenv("PQ_W8A8_BN"); return e ? (e[0] == '1' ? 128 : (e[0] == '2' ? 256 : 0)) : 0; }();
  static const int force_splits = [] { const char* e = getenv("PQ_W8A8_SPLITS"); return e ? atoi(e) : 0; }();
  int best_bn = 256, best_splits = 1;
  const int64_t best_cost =
      plan_w8a8_pair_group(M, N, count, K, sm_count(), acc == nullptr && sc.partials != nullptr ? sc.partial_bytes : 0,
                           force_bn, force_splits, &best_bn, &best_splits);
  if (best_cost < 0) return PQ_ERR_SHAPE;   // only reachable through contradictory ablation knobs
  const bool use128 = best_bn == 128;
  const int BN = best_bn;

  CUtensorMap tq;
  PairMaps maps;
  int rc = make_tmap_2d(&tq, q, static_cast<uint64_t>(M), static_cast<uint64_t>(K), BM_CTA, BK, 1, 128);
  if (rc != PQ_OK) return rc;
  PairArgs a;
  int64_t nb_total = 0;
  for (int g = 0; g < kMaxGroup; ++g) {
    const int src = g < count ? g : 0;   // unused slots repeat member 0 (never selected)
    rc = make_tmap_2d(&maps.w[g], wq[src], static_cast<uint64_t>(N[src]), static_cast<uint64_t>(K),
                      static_cast<uint32_t>(BN / 2), BK, 1, 128);
    if (rc != PQ_OK) return rc;
    if (acc == nullptr) {
      // FP16 result [M, N]; stores go out as 32 x 32 boxes staged with the 64-byte swizzle.
      rc = make_tmap_2d(&maps.y[g], y[src], static_cast<uint64_t>(M), static_cast<uint64_t>(N[src]), 32, 32, 2, 64);
      if (rc != PQ_OK) return rc;
    } else {
      maps.y[g] = tq;  // the accumulator export stores directly; the map is not used
    }
    a.s_ch[g] = s_ch[src];
    a.N[g] = static_cast<int>(N[src]);
    if (g < count) nb_total += (N[g] + BN - 1) / BN;
    a.nb_end[g] = g < count ? static_cast<int>(nb_total) : 0x7fffffff;
  }
  if (mb * nb_total > 0x3fffffff) return PQ_ERR_SHAPE;

  a.count = count;
  a.s_tok = s_tok;
  a.acc = acc;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.K = static_cast<int>(K);
  a.m_blocks = static_cast<int>(mb);
  a.n_blocks = static_cast<int>(nb_total);
  a.k_blocks = static_cast<int>(kblocks);
  a.splits = best_splits;
  a.wait_limit = wait_limit();
  a.ws = best_splits > 1 ? sc.partials : nullptr;
  a.counters = best_splits > 1 ? sc.counters : nullptr;
  if (acc != nullptr) {
    return use128 ? launch_pair_cfg<128, 7, 2, 2, 8, 1, true>(tq, maps, a, stream)
                  : launch_pair_cfg<256, 5, 2, 2, 8, 1, true>(tq, maps, a, stream);
  }
  if (use128) return launch_pair_cfg<128, 7, 2, 2, 8, 1, false>(tq, maps, a, stream);
  return launch_pair_cfg<256, 5, 2, 2, 8, 1, false>(tq, maps, a, stream);
}

int launch_gemm_w8a8_pair(const Scratch& sc, const int8_t* q, const float* s_tok, const void* wq,
                          const float* s_ch, int64_t M, int64_t N, int64_t K, void* y, int32_t* acc,
                          cudaStream_t stream) {
  return launch_gemm_w8a8_pair_group(sc, q, s_tok, 1, &wq, &s_ch, &N, &y, M, K, acc, stream);
}

}  // namespace pq
