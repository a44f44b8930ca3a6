// Quantized linear for one to four tokens (the smallest decode shapes) on the CUDA cores of sm_100a.
//
// At these token counts a tensor-core tile is almost all padding and what matters is (a) that the
// weights stream from HBM once, at full rate, and (b) how much of a call's work can happen before the
// call is allowed to look at its tokens: in a chain of dependent launches every kernel waits for its
// predecessor (griddepcontrol.wait), and the time between the predecessor's last load and the moment
// that wait returns is dead time for the memory system unless somebody has loads in flight.  So:
//
//   - A CTA owns whole weight rows (no K split, no cross-CTA reduction, no tensor memory, nothing to set
//     up but a few barriers).  Rows arrive in shared memory as bulk copies of RQ consecutive rows (a
//     "row set", contiguous in memory) into a ring of slots.
//   - Weights are constants of the model: the whole ring is requested BEFORE the wait on the preceding
//     kernel.  A CTA takes at most half of an SM's shared memory and registers, so the CTAs of launch
//     i+1 become resident next to those of launch i and fill their rings while launch i computes,
//     stores and drains.  For the 4096 x 4096 shapes the ring holds the CTA's entire share.
//   - After the wait the token codes (at most 4 x K bytes) are copied into shared memory once, in a
//     layout whose 16-byte chunks are permuted inside every run of 128 k, and each of eight consumer
//     warps takes row sets in turn.
//   - Inside a warp a lane owns the 128-k blocks l, l + 32, ... of the row: for W4 that is exactly one
//     scale group, so the lane forms the group's INT32 sum with dp4a (the packed words widen to INT8
//     with two logic operations, as in the tensor-core kernels: values 16 x code, 1/16 folded into the
//     scale), converts it once and adds it to its FP32 running sum with the group's scale; for W8 the
//     lane keeps one INT32 sum per row and token.  The weights lie in shared memory as they lie in
//     global memory, so the order in which a lane walks the 16-byte chunks of its block is rotated by
//     the lane index (eight consecutive lanes then touch eight different bank groups), and the token
//     codes -- whose placement is this kernel's to choose -- are stored so that the same rotation is
//     conflict-free for them too (code_pos below).  One reduce-scatter butterfly per row set adds the
//     lanes' sums (exact for W8; a fixed order for the FP32 sums of W4).
//
// Eight warps, all of them consumers: thread 0 requests the first ring pass, and the warp that has used
// up a slot requests the row set that goes into it next (no producer role, no "slot free" barriers).
// Successive row sets of one slot are in general consumed by different warps, and an mbarrier wait names
// its phase by parity only, so a warp first waits until its row set HAS BEEN REQUESTED (a per-slot word in
// shared memory, written after the request) and only then for the slot's barrier: at that point the
// barrier cannot be more than one phase away from the one meant.
// Every wait is bounded; the give-up path lets the copies in flight land before the CTA leaves.
#include <cuda_fp16.h>

#include "pq_internal.h"
#include "pq_ptx.cuh"
#include "pq_quant_math.cuh"

namespace pq {
namespace {

constexpr int kConsumerWarps = 8;
constexpr int kThreads = 32 * kConsumerWarps;
constexpr int kMaxSlots = 32;
constexpr int kCtaBytesMax = 112 * 1024;   // ring + token codes: a CTA stays below half an SM's shared memory
constexpr int kSoloBytesMax = 216 * 1024;  // ... or takes the SM alone, when that lets the ring hold its whole share
constexpr int kCodeBytesMax = 44 * 1024;
constexpr int kFillBatch = 12;             // 16-byte chunks of codes a thread has in flight at once
constexpr int kXBatch = 6;                 // ... of FP16 activations, where the kernel quantizes them itself

struct RowArgs {
  const uint8_t* w;        // W8: [N, K] codes; W4: [N, K/2] packed
  const int8_t* q;         // [M, K]
  const __half* x;         // kFuseX: [M, K] FP16 activations instead of q and s_tok
  const float* s_tok;      // [M]
  const float* s_ch;       // W8: [N]
  const __half* s_grp;     // W4: [K/128, N]
  __half* y;               // [M, N]
  int32_t* acc;            // export: W8 [M, N]; W4 [K/128, M, N]
  int* status;
  int M, N, K;
  int row_bytes;           // K or K/2
  int slots;               // ring depth
  int n_sets;              // row sets in all: N / RQ
  int kblocks;             // ceil(K / 128)
  uint32_t wait_limit;
};

// 1-D bulk copy global -> shared, completion counted in bytes on `bar`.  Both addresses 16-byte aligned,
// size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_dst),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// Where the 16-byte chunk c (0..7) of a 128-byte block of token codes is stored inside the block, for a
// block whose index is sw modulo 8.  A lane (index sw modulo 8) reads, at step jc of its walk,
//   W8: chunk (jc + sw) & 7                       -> position (jc - sw) & 7,
//   W4: chunks 2u, 2u + 1 with u = (jc + sw/2) & 3 -> positions 2 ((jc - sw/2) & 3) + (0|1 ^ (sw & 1)),
// distinct over eight consecutive lanes in both cases; for a fixed block the map is a bijection.
template <bool kW4>
__device__ __forceinline__ int code_pos(int c, int sw) {
  if constexpr (kW4) {
    return 2 * (((c >> 1) - 2 * (sw >> 1)) & 3) + ((c ^ sw) & 1);
  } else {
    return (c - 2 * sw) & 7;
  }
}

__device__ __forceinline__ int dp4a_s8(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Sum over the 32 lanes of V values per lane (V a power of two, <= 16): a reduce-scatter butterfly.  On
// return v[0] holds, in every lane, the total of value index `which` (returned); each total lives in
// 32 / V lanes.  The association order is fixed, so FP32 sums are reproducible.
template <typename T, int V>
__device__ __forceinline__ int lane_reduce_scatter(T (&v)[V], int lane) {
  int which = 0;
  int offset = 16;
#pragma unroll
  for (int width = V; width > 1; width >>= 1, offset >>= 1) {
    const int half = width >> 1;
    const bool upper = (lane & offset) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const T send = upper ? v[i] : v[i + half];
      const T keep = upper ? v[i + half] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, offset);
    }
    if (upper) which += half;
  }
  for (; offset > 0; offset >>= 1) v[0] = v[0] + __shfl_xor_sync(0xffffffffu, v[0], offset);
  return which;
}

// kFuseX: the kernel quantizes its own tokens (Eq. 1-2, the arithmetic of the quantizer kernels) instead of
// reading codes and token scales: one launch less on the critical path of a decode step.
template <bool kW4, int MT, int RQ, bool kExportAcc, bool kFuseX = false>
__global__ void __launch_bounds__(kThreads, 2) gemv_rows_kernel(const RowArgs p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  const uint32_t smem_base = smem_u32(smem);
  const int slot_bytes = RQ * p.row_bytes;
  const int code_row = p.kblocks * 128;                           // bytes of one token's codes in shared memory
  const uint32_t ring = smem_base;
  const uint32_t codes = ring + static_cast<uint32_t>(p.slots * slot_bytes);
  const uint32_t bar_full = codes + static_cast<uint32_t>(MT * code_row);
  // per slot: the row set last requested into it (for the give-up path), then the CTA's "gave up" flag
  volatile int* last_set = reinterpret_cast<volatile int*>(smem + (bar_full - smem_base) + kMaxSlots * 8);
  volatile int* abort_flag = last_set + kMaxSlots;
  const WaitCtx wc{abort_flag, p.wait_limit};

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // This CTA's row sets: blockIdx.x, blockIdx.x + gridDim.x, ...
  const int first_set = static_cast<int>(blockIdx.x);
  const int my_sets = first_set < p.n_sets ? (p.n_sets - first_set + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;
  auto set_src = [&](int j) {
    return p.w + static_cast<int64_t>(first_set + j * static_cast<int>(gridDim.x)) * slot_bytes;
  };

  auto request = [&](int j) {   // row set j of this CTA into its slot (one thread)
    const uint32_t s = static_cast<uint32_t>(j % p.slots);
    mbar_arrive_expect_tx(bar_full + s * 8, static_cast<uint32_t>(slot_bytes));
    bulk_load(ring + s * static_cast<uint32_t>(slot_bytes), set_src(j), static_cast<uint32_t>(slot_bytes), bar_full + s * 8);
    __threadfence_block();      // the barrier is in row set j's phase before anybody can read "requested"
    last_set[s] = j;
  };
  // Row set j has landed in its slot: first "it has been requested", then its phase of the slot's barrier.
  auto wait_set = [&](int j) -> bool {
    const uint32_t s = static_cast<uint32_t>(j % p.slots);
    bool requested = false;
    for (uint32_t i = 0; i < wc.limit; ++i) {
      if (last_set[s] >= j) { requested = true; break; }
      if ((i & 255u) == 255u && *abort_flag) break;
    }
    if (!requested) {
      *abort_flag = 1;
      return false;
    }
    return mbar_wait(bar_full + s * 8, static_cast<uint32_t>(j / p.slots) & 1u, wc);
  };
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < p.slots; ++s) {
      mbar_init(bar_full + s * 8, 1);
      last_set[s] = -1;
    }
    fence_mbar_init();
    // The whole ring at once: weights are constants of the model, no wait on the preceding kernel.
    const int first = my_sets < p.slots ? my_sets : p.slots;
    for (int j = 0; j < first; ++j) request(j);
  }
  grid_dep_launch();   // the successor's CTAs may become resident and fill their own rings
  {
    // ------------------------------------------------------------ consumers (all warps)
    grid_dep_wait();   // codes and token scales come from the preceding kernel; outputs are overwritten
    // Token codes -> shared memory: token m at codes + m * code_row; inside every 128-byte block b the
    // 16-byte chunk c sits at position code_pos(c, b & 7).  Tokens >= M and bytes >= K read as zero.
    // This copy sits on the critical path of the call (nothing else can start before it), and a load
    // takes a round trip to the L2: a thread issues all its loads of a batch before it stores any.
    float st[MT];
    if constexpr (kFuseX) {
      // Pass 1: every token's largest magnitude (all of the CTA's threads over all of x; a CTA reads the
      // few KB of x by itself, from the L2).  Pass 2 reads x again (now from the L1) and writes the codes.
      __shared__ float red[kConsumerWarps][MT];
      const int x_chunks = p.K >> 3;                      // 16-byte chunks (8 values) of one token
      float amax[MT];
#pragma unroll
      for (int m = 0; m < MT; ++m) amax[m] = 0.0f;
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        if (m < p.M) {
          const uint4* xr = reinterpret_cast<const uint4*>(p.x + static_cast<int64_t>(m) * p.K);
          for (int c0 = threadIdx.x; c0 < x_chunks; c0 += kXBatch * kThreads) {
            uint4 v[kXBatch];
#pragma unroll
            for (int u = 0; u < kXBatch; ++u) {
              const int c = c0 + u * kThreads;
              v[u] = c < x_chunks ? xr[c] : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < kXBatch; ++u) amax[m] = fmaxf(amax[m], absmax8(v[u]));
          }
        }
      }
#pragma unroll
      for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax[m] = fmaxf(amax[m], __shfl_xor_sync(0xffffffffu, amax[m], o));
        if (lane == 0) red[warp][m] = amax[m];
      }
      __syncthreads();
      float fm[MT];
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        float a = 0.0f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) a = fmaxf(a, red[w][m]);
        act_scale(a, &st[m], &fm[m]);
        if (kExportAcc || m >= p.M) st[m] = 0.0f;
      }
      const int chunks_per_row = p.kblocks * 8;
      const int k_chunks = p.K >> 4;
      const int total = MT * chunks_per_row;
      for (int i = threadIdx.x; i < total; i += kThreads) {
        const int m = i / chunks_per_row, c = i - m * chunks_per_row;
        uint4 out = make_uint4(0u, 0u, 0u, 0u);
        if (m < p.M && c < k_chunks) {
          const uint4* xr = reinterpret_cast<const uint4*>(p.x + static_cast<int64_t>(m) * p.K) + 2 * c;
          const uint4 lo = xr[0], hi = xr[1];
          const __half* hl = reinterpret_cast<const __half*>(&lo);
          const __half* hh = reinterpret_cast<const __half*>(&hi);
          float f = fm[0];
#pragma unroll
          for (int j = 1; j < MT; ++j) f = (m == j) ? fm[j] : f;
          out.x = codes4<false>(__half2float(hl[0]), __half2float(hl[1]), __half2float(hl[2]), __half2float(hl[3]), f);
          out.y = codes4<false>(__half2float(hl[4]), __half2float(hl[5]), __half2float(hl[6]), __half2float(hl[7]), f);
          out.z = codes4<false>(__half2float(hh[0]), __half2float(hh[1]), __half2float(hh[2]), __half2float(hh[3]), f);
          out.w = codes4<false>(__half2float(hh[4]), __half2float(hh[5]), __half2float(hh[6]), __half2float(hh[7]), f);
        }
        const int b = c >> 3, cc = c & 7;
        *reinterpret_cast<uint4*>(smem + (codes - smem_base) + m * code_row + b * 128 + (code_pos<kW4>(cc, b & 7) << 4)) = out;
      }
    } else
    {
      const int chunks_per_row = p.kblocks * 8;
      const int k_chunks = p.K >> 4;
      const int total = MT * chunks_per_row;
      for (int i0 = threadIdx.x; i0 < total; i0 += kFillBatch * kThreads) {
        uint4 v[kFillBatch];
#pragma unroll
        for (int u = 0; u < kFillBatch; ++u) {
          const int i = i0 + u * kThreads;
          const int m = i / chunks_per_row, c = i - m * chunks_per_row;
          v[u] = make_uint4(0u, 0u, 0u, 0u);
          if (i < total && m < p.M && c < k_chunks)
            v[u] = *reinterpret_cast<const uint4*>(p.q + static_cast<int64_t>(m) * p.K + c * 16);
        }
#pragma unroll
        for (int u = 0; u < kFillBatch; ++u) {
          const int i = i0 + u * kThreads;
          if (i < total) {
            const int m = i / chunks_per_row, c = i - m * chunks_per_row;
            const int b = c >> 3, cc = c & 7;
            *reinterpret_cast<uint4*>(smem + (codes - smem_base) + m * code_row + b * 128 + (code_pos<kW4>(cc, b & 7) << 4)) = v[u];
          }
        }
      }
    }
    __syncthreads();   // the codes are in place (and the barriers exist) before anybody goes on
    if constexpr (!kFuseX) {
#pragma unroll
      for (int m = 0; m < MT; ++m) st[m] = (!kExportAcc && m < p.M) ? __ldg(p.s_tok + m) : 0.0f;
    }
    const int sw = lane & 7;                 // this lane's blocks are l, l + 32, ...: (b & 7) == (l & 7)

    for (int j = warp; j < my_sets; j += kConsumerWarps) {
      const int n0 = (first_set + j * static_cast<int>(gridDim.x)) * RQ;
      const uint32_t s = static_cast<uint32_t>(j % p.slots);
      const uint32_t slot = ring + s * static_cast<uint32_t>(slot_bytes);
      int acc[RQ][MT];
      float R[RQ][MT];
#pragma unroll
      for (int r = 0; r < RQ; ++r) {
#pragma unroll
        for (int m = 0; m < MT; ++m) { acc[r][m] = 0; R[r][m] = 0.0f; }
      }
      // W4: the group scales of this lane's first block, asked for ahead of the wait on the slot
      float sg[RQ];
      auto load_scales = [&](int b) {
#pragma unroll
        for (int r = 0; r < RQ; ++r) sg[r] = 0.0f;
        if constexpr (kW4 && !kExportAcc) {
          if (b < p.kblocks) {
            const __half* sp = p.s_grp + static_cast<int64_t>(b) * p.N + n0;
            if constexpr (RQ == 4) {
              const uint2 raw = __ldg(reinterpret_cast<const uint2*>(sp));
              const __half2 h01 = *reinterpret_cast<const __half2*>(&raw.x), h23 = *reinterpret_cast<const __half2*>(&raw.y);
              sg[0] = __low2float(h01) * 0.0625f; sg[1] = __high2float(h01) * 0.0625f;
              sg[2] = __low2float(h23) * 0.0625f; sg[3] = __high2float(h23) * 0.0625f;
            } else {
              const uint32_t raw = __ldg(reinterpret_cast<const uint32_t*>(sp));
              const __half2 h01 = *reinterpret_cast<const __half2*>(&raw);
              sg[0] = __low2float(h01) * 0.0625f; sg[1] = __high2float(h01) * 0.0625f;
            }
          }
        }
      };
      load_scales(lane);
      const bool got = __all_sync(0xffffffffu, wait_set(j));
      if (!got) break;

      for (int b = lane; b < ((p.kblocks + 31) & ~31); b += 32) {
        const bool live = b < p.kblocks;
        if (live) {
          const uint32_t qb = codes + static_cast<uint32_t>(b * 128);
          if constexpr (kW4) {
            const uint32_t wb = slot + static_cast<uint32_t>(b * 64);
            const int rot = sw >> 1;
#pragma unroll
            for (int jc = 0; jc < 4; ++jc) {
              const int pc = (jc + rot) & 3;          // 32-k run of the block handled at this step
              uint4 qa[MT], qh[MT];
#pragma unroll
              for (int m = 0; m < MT; ++m) {
                qa[m] = lds128(qb + m * code_row + (code_pos<true>(2 * pc, sw) << 4));
                qh[m] = lds128(qb + m * code_row + (code_pos<true>(2 * pc + 1, sw) << 4));
              }
#pragma unroll
              for (int r = 0; r < RQ; ++r) {
                const uint4 w4 = lds128(wb + r * p.row_bytes + (pc << 4));
                uint4 lo, hi;
                lo.x = (w4.x << 4) & 0xF0F0F0F0u; hi.x = w4.x & 0xF0F0F0F0u;
                lo.y = (w4.y << 4) & 0xF0F0F0F0u; hi.y = w4.y & 0xF0F0F0F0u;
                lo.z = (w4.z << 4) & 0xF0F0F0F0u; hi.z = w4.z & 0xF0F0F0F0u;
                lo.w = (w4.w << 4) & 0xF0F0F0F0u; hi.w = w4.w & 0xF0F0F0F0u;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                  int a = acc[r][m];
                  a = dp4a_s8(lo.x, qa[m].x, a); a = dp4a_s8(lo.y, qa[m].y, a);
                  a = dp4a_s8(lo.z, qa[m].z, a); a = dp4a_s8(lo.w, qa[m].w, a);
                  a = dp4a_s8(hi.x, qh[m].x, a); a = dp4a_s8(hi.y, qh[m].y, a);
                  a = dp4a_s8(hi.z, qh[m].z, a); a = dp4a_s8(hi.w, qh[m].w, a);
                  acc[r][m] = a;
                }
              }
            }
          } else {
            const uint32_t wb = slot + static_cast<uint32_t>(b * 128);
            const int live_chunks = min(8, (p.K >> 4) - b * 8);   // the last block of a row may be short
#pragma unroll
            for (int jc = 0; jc < 8; ++jc) {
              const int pc = (jc + sw) & 7;
              if (pc < live_chunks) {
                uint4 qa[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) qa[m] = lds128(qb + m * code_row + (code_pos<false>(pc, sw) << 4));
#pragma unroll
                for (int r = 0; r < RQ; ++r) {
                  const uint4 w8 = lds128(wb + r * p.row_bytes + (pc << 4));
#pragma unroll
                  for (int m = 0; m < MT; ++m) {
                    int a = acc[r][m];
                    a = dp4a_s8(w8.x, qa[m].x, a); a = dp4a_s8(w8.y, qa[m].y, a);
                    a = dp4a_s8(w8.z, qa[m].z, a); a = dp4a_s8(w8.w, qa[m].w, a);
                    acc[r][m] = a;
                  }
                }
              }
            }
          }
        }
        if constexpr (kW4) {
          // one INT32 per (row, token) for this lane's group: export it, or promote it with the group scale
          if constexpr (kExportAcc) {
            if (live) {
#pragma unroll
              for (int r = 0; r < RQ; ++r) {
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                  if (m < p.M) p.acc[(static_cast<int64_t>(b) * p.M + m) * p.N + n0 + r] = acc[r][m] >> 4;
                }
              }
            }
          } else {
#pragma unroll
            for (int r = 0; r < RQ; ++r) {
#pragma unroll
              for (int m = 0; m < MT; ++m) R[r][m] = fmaf(__int2float_rn(acc[r][m]), sg[r], R[r][m]);
            }
            if (b + 32 < p.kblocks) load_scales(b + 32);
          }
#pragma unroll
          for (int r = 0; r < RQ; ++r) {
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[r][m] = 0;
          }
        }
      }
      // The slot has been read by every lane: request the row set that goes into it next.  (The reads
      // went through the generic proxy, the copy writes through the async proxy: fence in between.)
      __syncwarp();
      if (lane == 0 && j + p.slots < my_sets) {
        fence_proxy_async_smem();
        request(j + p.slots);
      }

      if constexpr (kW4 && kExportAcc) continue;
      // ---- add the lanes' sums and store
      constexpr int V = RQ * MT;
      if constexpr (kW4) {
        float v[V];
#pragma unroll
        for (int r = 0; r < RQ; ++r) {
#pragma unroll
          for (int m = 0; m < MT; ++m) v[r * MT + m] = R[r][m];
        }
        const int which = lane_reduce_scatter<float, V>(v, lane);
        const int r = which / MT, m = which % MT;
        if ((lane & (32 / V - 1)) == 0 && m < p.M) {
          float stm = st[0];
#pragma unroll
          for (int i = 1; i < MT; ++i) stm = (m == i) ? st[i] : stm;
          p.y[static_cast<int64_t>(m) * p.N + n0 + r] = __float2half_rn(__fmul_rn(v[0], stm));
        }
      } else {
        int v[V];
#pragma unroll
        for (int r = 0; r < RQ; ++r) {
#pragma unroll
          for (int m = 0; m < MT; ++m) v[r * MT + m] = acc[r][m];
        }
        const int which = lane_reduce_scatter<int, V>(v, lane);
        const int r = which / MT, m = which % MT;
        if ((lane & (32 / V - 1)) == 0 && m < p.M) {
          if constexpr (kExportAcc) {
            p.acc[static_cast<int64_t>(m) * p.N + n0 + r] = v[0];
          } else {
            float stm = st[0];
#pragma unroll
            for (int i = 1; i < MT; ++i) stm = (m == i) ? st[i] : stm;
            const float sc = __ldg(p.s_ch + n0 + r);
            p.y[static_cast<int64_t>(m) * p.N + n0 + r] =
                __float2half_rn(__fmul_rn(__fmul_rn(__int2float_rn(v[0]), stm), sc));
          }
        }
      }
    }
  }

  // ------------------------------------------------------------ teardown
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // Somebody gave up: the copies already requested still land in this CTA's shared memory; stay until
    // they have.
    for (int s = 0; s < p.slots; ++s) {
      const int j = last_set[s];
      if (j >= 0) mbar_drain(bar_full + static_cast<uint32_t>(s) * 8, static_cast<uint32_t>(j / p.slots) & 1u);
    }
    atomicExch(p.status, static_cast<int>(PQ_ERR_TIMEOUT));
  }
}

template <bool kW4, int MT, int RQ, bool kExportAcc, bool kFuseX = false>
int launch_rows_cfg(const RowArgs& a, int smem_bytes, int grid, cudaStream_t stream) {
  auto kern = gemv_rows_kernel<kW4, MT, RQ, kExportAcc, kFuseX>;
  static PerDeviceOnce once;
  if (const int rc = set_dynamic_smem_once(once, kern, kSoloBytesMax + 1024); rc != PQ_OK) return rc;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cuda_status(cudaLaunchKernelEx(&cfg, kern, a));
}

template <bool kW4, int MT, bool kExportAcc, bool kFuseX = false>
int launch_rows_rq(int rq, const RowArgs& a, int smem_bytes, int grid, cudaStream_t stream) {
  return rq == 4 ? launch_rows_cfg<kW4, MT, 4, kExportAcc, kFuseX>(a, smem_bytes, grid, stream)
                 : launch_rows_cfg<kW4, MT, 2, kExportAcc, kFuseX>(a, smem_bytes, grid, stream);
}

// Shape of a launch: rows per row set, ring depth, grid, shared memory.  `fits`: the ring holds a CTA's
// whole share of the weights, so everything is requested ahead of the wait on the preceding kernel.
struct RowPlan {
  int rq, slots, grid, mt, code_bytes, smem_bytes;
  bool fits;
};
bool plan_rows_within(int cta_bytes_max, int w_bits, int64_t M, int64_t N, int64_t K, int sms, RowPlan* out);

// Two CTAs of consecutive launches per SM where a CTA's whole share fits half an SM.  Otherwise, for one
// token and a share of a few large row sets, one CTA per SM with a ring of up to 216 KB if THAT holds the
// whole share (the next launch's CTAs then start when this one's leave, and their loads run under the dead
// time between the launches: 11008 -> 4096 W4, 10.2 -> 8.1 us; with many small sets the half-SM ring with
// refills is the better one: 4096 -> 11008 W4, 8.5 against 9.2 us).  Else the half-SM ring with refills.
bool plan_rows(int w_bits, int64_t M, int64_t N, int64_t K, int sms, RowPlan* out) {
  RowPlan half, solo;
  if (!plan_rows_within(kCtaBytesMax, w_bits, M, N, K, sms, &half)) return false;
  if (!half.fits && M == 1 && plan_rows_within(kSoloBytesMax, w_bits, M, N, K, sms, &solo) && solo.fits && solo.slots <= 8)
    half = solo;
  *out = half;
  return true;
}

bool plan_rows_within(int cta_bytes_max, int w_bits, int64_t M, int64_t N, int64_t K, int sms, RowPlan* out) {
  if (M < 1 || M > 4 || N < 4 || N % 4 != 0 || sms < 1) return false;
  const int64_t row_bytes = w_bits == 4 ? K / 2 : K;
  if (row_bytes % 16 != 0 || row_bytes > cta_bytes_max) return false;
  RowPlan pl;
  pl.mt = M <= 1 ? 1 : (M <= 2 ? 2 : 4);
  const int64_t code_bytes = pl.mt * ((K + 127) / 128) * 128;
  if (code_bytes > kCodeBytesMax) return false;
  pl.code_bytes = static_cast<int>(code_bytes);
  const int ring_max = cta_bytes_max - pl.code_bytes;
  if (2 * 2 * row_bytes > ring_max) return false;                            // at least two slots of two rows
  // Row sets of four rows where three of them fit the ring, else of two.
  pl.rq = (3 * 4 * row_bytes <= ring_max) ? 4 : 2;
  const int slot_bytes = pl.rq * static_cast<int>(row_bytes);
  const int64_t n_sets = N / pl.rq;
  if (n_sets > 0x7fffffff) return false;
  pl.grid = n_sets < sms ? static_cast<int>(n_sets) : sms;
  const int sets_per_cta = static_cast<int>((n_sets + pl.grid - 1) / pl.grid);
  int slots = ring_max / slot_bytes;
  slots = slots > kMaxSlots ? kMaxSlots : slots;
  pl.fits = sets_per_cta <= slots;
  pl.slots = slots > sets_per_cta ? sets_per_cta : slots;
  pl.smem_bytes = pl.slots * slot_bytes + pl.code_bytes + kMaxSlots * 8 + kMaxSlots * 4 + 16 + 128;
  *out = pl;
  return true;
}

template <bool kW4>
int launch_rows(const int8_t* q, const float* s_tok, const void* w, const float* s_ch, const void* s_grp, int64_t M,
                int64_t N, int64_t K, void* y, int32_t* acc, cudaStream_t stream, const void* x = nullptr) {
  RowPlan pl;
  if (!plan_rows(kW4 ? 4 : 8, M, N, K, sm_count(), &pl)) return PQ_ERR_SHAPE;
  RowArgs a;
  a.row_bytes = static_cast<int>(kW4 ? K / 2 : K);
  a.w = static_cast<const uint8_t*>(w);
  a.q = q;
  a.x = static_cast<const __half*>(x);
  a.s_tok = s_tok;
  a.s_ch = s_ch;
  a.s_grp = static_cast<const __half*>(s_grp);
  a.y = static_cast<__half*>(y);
  a.acc = acc;
  a.status = device_status_ptr();
  if (a.status == nullptr) return PQ_ERR_CUDA;
  a.M = static_cast<int>(M);
  a.N = static_cast<int>(N);
  a.K = static_cast<int>(K);
  a.n_sets = static_cast<int>(N / pl.rq);
  a.kblocks = static_cast<int>((K + 127) / 128);
  a.wait_limit = wait_limit();
  a.slots = pl.slots;
  const int rq = pl.rq, grid = pl.grid, smem_bytes = pl.smem_bytes;
  const bool ex = acc != nullptr;
  if (x != nullptr) {   // the kernel quantizes its own tokens
    if (ex) return PQ_ERR_SHAPE;
    switch (pl.mt) {
      case 1: return launch_rows_rq<kW4, 1, false, true>(rq, a, smem_bytes, grid, stream);
      case 2: return launch_rows_rq<kW4, 2, false, true>(rq, a, smem_bytes, grid, stream);
      default: return launch_rows_rq<kW4, 4, false, true>(rq, a, smem_bytes, grid, stream);
    }
  }
  switch (pl.mt) {
    case 1: return ex ? launch_rows_rq<kW4, 1, true>(rq, a, smem_bytes, grid, stream) : launch_rows_rq<kW4, 1, false>(rq, a, smem_bytes, grid, stream);
    case 2: return ex ? launch_rows_rq<kW4, 2, true>(rq, a, smem_bytes, grid, stream) : launch_rows_rq<kW4, 2, false>(rq, a, smem_bytes, grid, stream);
    default: return ex ? launch_rows_rq<kW4, 4, true>(rq, a, smem_bytes, grid, stream) : launch_rows_rq<kW4, 4, false>(rq, a, smem_bytes, grid, stream);
  }
}

}  // namespace

// Whether the row kernel is the schedule for this shape: where a CTA's whole share of the weights fits its
// ring (everything is in flight before the call may look at its tokens), and for W4 with one token always.
// Measured against the tensor-core weight-streaming kernel on the 7B-class shapes (4096^2, 4096 -> 11008,
// 11008 -> 4096), one token: W4 4.4 / 8.5 / 8.1 us against 7.5 / 11.5 / 11.9 us, W8 (4096^2) 5.7 against
// 6.2 us; W4 with four tokens at 4096^2 6.5 against 7.8 us.  With a share that does not fit, W8 and the
// multi-token cases lose (the refills and the dp4a work land on the critical path behind the wait) and stay
// on the tensor cores.
bool gemv_rows_serves(int w_bits, int64_t M, int64_t N, int64_t K, int sms) {
  RowPlan pl;
  if (!plan_rows(w_bits, M, N, K, sms, &pl)) return false;
  return pl.fits || (w_bits == 4 && M == 1);
}

int launch_gemv_rows_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch, int64_t M, int64_t N,
                          int64_t K, void* y, int32_t* acc, cudaStream_t stream) {
  return launch_rows<false>(q, s_tok, wq, s_ch, nullptr, M, N, K, y, acc, stream);
}

int launch_gemv_rows_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp, int64_t M, int64_t N,
                          int64_t K, void* y, int32_t* acc_g, cudaStream_t stream) {
  return launch_rows<true>(q, s_tok, wp, nullptr, s_grp, M, N, K, y, acc_g, stream);
}

// The same from FP16 activations: the kernel quantizes them itself.
int launch_gemv_rows_w8a8_x(const void* x, const void* wq, const float* s_ch, int64_t M, int64_t N, int64_t K, void* y,
                            cudaStream_t stream) {
  return launch_rows<false>(nullptr, nullptr, wq, s_ch, nullptr, M, N, K, y, nullptr, stream, x);
}
int launch_gemv_rows_w4a8_x(const void* x, const void* wp, const void* s_grp, int64_t M, int64_t N, int64_t K, void* y,
                            cudaStream_t stream) {
  return launch_rows<true>(nullptr, nullptr, wp, nullptr, s_grp, M, N, K, y, nullptr, stream, x);
}

}  // namespace pq
