// Tensor-core E0M4 matmul over a LIST of independent problems that share M (9 <= M <= 128): one
// persistent launch streams the weights of up to 22 matrices (Section 2.2's matrix-matrix
// implementation at the token counts of batched decoding, where it is still bound by the weight
// bytes).
//
// The work of all problems is one sequence of rounds, a round being one 128-k group of one
// 128-column panel (8.7 KB of codes and scales).  The sequence is cut into equal contiguous
// ranges, one per CTA, so every SM streams the same number of bytes whatever the shapes are and
// pays pipeline fill and drain once per launch instead of once per matrix.  A range is walked as
// pieces (problem, panel, groups g0..g1).  A piece that covers its panel's whole K is converted
// and stored directly; the pieces of a panel that a range boundary cuts add fp32 partial sums
// into a scratch slot named after the first boundary inside the panel, and the CTA that brings
// the slot's group count to K/128 converts the sums and clears the slot again.
//
// Lists of more than 80 tokens run on pairs of CTAs (template argument PAIR, see the kernel).
// Both kernels also serve lists of E0M8 problems (template argument BITS = 8, 1 <= M <= 128:
// a round then carries 16.9 KB, twice the bytes for the same tensor-core time, so the list streams
// at the memory rate already at one token).
//
// The pipeline is the one of the single-problem kernel's rounds of a whole group: packed
// producer, token producer (one tensor map per problem, two boxes of 64 k per round), four
// dequantizer groups writing the A operand into tensor memory, one MMA-issuing warp (eight
// tcgen05.mma per wait and commit), four epilogue warps.  Every mbarrier wait is bounded.
#include "common.cuh"
#include "ptx.cuh"
#include "tc_common.cuh"
#include "tuning.h"

namespace tl {
namespace {

// Tensor memory: the accumulator needs at most 128 columns here (one per token), which leaves room
// for six operand slots of a whole round (64 columns = 128 k).  Four dequantizer groups share them
// in turn, so a group can expand round r + 4 while round r still waits for the tensor core.
constexpr int kBatchAccCols = 128;
constexpr int kRounds = 6;                 // rounds in flight
constexpr int kRoundCols = 2 * kAStageCols;
static_assert(kBatchAccCols + kRounds * kRoundCols <= kTmemCols, "tensor memory budget");
constexpr int kBatchGroups = 4;            // dequantizer groups of four warps (one warp per lane quadrant)
constexpr int kBatchDequantWarps = 4 * kBatchGroups;
constexpr int kBatchThreads = (kFirstDequantWarp + kBatchDequantWarps + kEpilogueWarps) * 32;

struct TcBatchProb {
  const uint8_t* packed;
  const uint8_t* scales;
  __half* y;
  int N, ng, nbs, panels;
  int units;        // what the sequence counts per group: panels, or panel pairs when two CTAs share the work
  int round_begin;  // first round of this problem in the concatenated sequence
};

struct TcBatchParams {
  CUtensorMap maps[kMaxTcBatch];   // x[M, K] of every problem: boxes of 64 k x tok rows, 128-byte swizzle
  TcBatchProb prob[kMaxTcBatch];
  unsigned int* status;
  float* ws;           // scratch slots [slot][tok][128 columns] fp32, zero on entry and left zero
  unsigned int* cnt;   // groups added to each slot so far, zero on entry and left zero
  int M, tok, count, total_rounds;
  int sx;       // token boxes (of one round) in the ring
  int pslots;   // slots of the packed ring
  int skip_copies;       // diagnostics: neither producer issues a copy, so every wait runs out
  long long wait_limit;  // SM cycles after which a bounded wait gives up
};

// A piece of a CTA's range: groups [g0, g1) of one panel of problem j.
struct Piece {
  int j, panel, g0, g1, R, ng;
};

// Walks a contiguous range of rounds piece by piece; every warp role runs its own copy.
// `step` and `rank`: with pairs a unit of the sequence is a pair of panels and this CTA takes
// panel 2 * unit + rank of it; R = 0 marks the missing partner of an odd last panel.
template <int STEP>
struct PieceWalk {
  const TcBatchParams& p;
  int j, panel, g, left, rank;
  __device__ PieceWalk(const TcBatchParams& p_, int c0, int n, int rank_) : p(p_), left(n), rank(STEP == 1 ? 0 : rank_) {
    j = 0;
    while (j + 1 < p.count && p.prob[j + 1].round_begin <= c0) ++j;
    const int off = c0 - p.prob[j].round_begin;
    panel = off / p.prob[j].ng;
    g = off - panel * p.prob[j].ng;
  }
  __device__ bool done() const { return left <= 0; }
  __device__ Piece cur() const {
    Piece w;
    const TcBatchProb& q = p.prob[j];
    w.j = j;
    w.panel = STEP == 1 ? panel : panel * STEP + rank;
    w.ng = q.ng;
    w.g0 = g;
    w.g1 = q.ng - g < left ? q.ng : g + left;
    const int rest = q.nbs - kPanelTiles * w.panel;
    w.R = rest < kPanelTiles ? (STEP == 1 || rest > 0 ? rest : 0) : kPanelTiles;
    return w;
  }
  __device__ void next() {
    const TcBatchProb& q = p.prob[j];
    const int n = q.ng - g < left ? q.ng - g : left;
    left -= n;
    g += n;
    if (g == q.ng) {
      g = 0;
      if (++panel == q.units && left > 0) {
        panel = 0;
        ++j;
      }
    }
  }
};

static_assert(sizeof(TcBatchParams) <= 4096, "tensor maps must stay within the first 4 KB of parameter space");

// One CTA per range (lists of at most 80 tokens).  This kernel is kept as its own text, not as the
// PAIR = false instantiation of the kernel below: that instantiation computes the same thing but
// measured 7 % slower (118 -> 127 us on four ChatGLM2-6B-shaped layers at 16 tokens), and the
// difference could not be attributed to any one of the generalised expressions.
// BITS = 8: E0M8 codes (tiles of 2048 bytes in chunks of 16 rows, see e0m8.cu), groups of 128.
template <int G, int BITS = 4>
__global__ void __launch_bounds__(kBatchThreads, 1)
gemm_tc_batch_kernel(const __grid_constant__ TcBatchParams p) {
  static_assert(BITS == 4 || (BITS == 8 && G == kGroup), "8-bit codes come with groups of 128");
  constexpr int kSubs = kGroup / G;
  constexpr int kSlot = tc_slot_bytes(BITS, G);
  constexpr int kTileB = BITS == 8 ? 2048 : 1024;   // bytes of a packed tile
  constexpr int kCodeBytes = kPanelTiles * kTileB;  // codes of a slot; the scale words follow them
  constexpr int SA = kRounds;
  constexpr int PM = kMaxPackedSlots;
  const int S = p.sx;
  const int P = p.pslots;
  const uint32_t x_half_bytes = (uint32_t)p.tok * kStageK * 2;  // one token box: tok rows of 64 k
  const uint32_t x_round_bytes = 2 * x_half_bytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t pk0 = smem0 + (uint32_t)S * x_round_bytes;  // the packed ring follows the token boxes
  const uint32_t bar0 = smem0 + kBarOffset;
  // Round `it` (counted over the whole launch) uses barrier pair it % SA, the operand slot
  // it % SA of tensor memory (64 columns) and token box pair it % S.
  const uint32_t ready = bar0;                  // [SA] token boxes landed and weights dequantized
  const uint32_t consumed = bar0 + 8 * SA;      // [SA] the tensor core is done with the round
  const uint32_t full_p = consumed + 8 * SA;    // [P] packed chunk has landed
  const uint32_t empty_p = full_p + 8 * PM;     // [P] dequantizers are done with the chunk
  const uint32_t acc_full = empty_p + 8 * PM;   // the piece's accumulator is complete
  const uint32_t acc_empty = acc_full + 8;      // the epilogue has drained it
  const uint32_t tmem_slot = acc_empty + 8;
  const uint32_t last_flag = tmem_slot + 4;     // this CTA completed the panel of its partial piece

  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const int lane = tid & 31;
  // this CTA's contiguous range of rounds
  const int c0 = (int)((long long)p.total_rounds * blockIdx.x / gridDim.x);
  const int c1 = (int)((long long)p.total_rounds * (blockIdx.x + 1) / gridDim.x);
  const int n_rounds = c1 - c0;

  if (tid == 0) {
    for (int s = 0; s < SA; ++s) {
      ptx::mbar_init(ready + 8 * s, 5);  // four dequantizer warps + the token producer
      ptx::mbar_init(consumed + 8 * s, 1);
    }
    for (int s = 0; s < P; ++s) {
      ptx::mbar_init(full_p + 8 * s, 1);
      ptx::mbar_init(empty_p + 8 * s, 4);
    }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, kEpilogueWarps);
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
  // Programmatic dependent launch: only weights are touched before griddepcontrol.wait (the token
  // producer waits before its first read of x, the epilogue before its first write).
  ptx::pdl_launch_dependents();

  bool ok = true;
  if (warp == 0) {
    // ------------------------------------------------- producer of packed codes and scale words
    if (lane == 0 && !p.skip_copies) {
      int ps = 0, pphase = 0, first = 1;
      for (PieceWalk<1> w(p, c0, n_rounds, 0); !w.done() && ok; w.next()) {
        const Piece wi = w.cur();
        const TcBatchProb& q = p.prob[wi.j];
        const size_t tile_base = (size_t)wi.panel * kPanelTiles * wi.ng;
        for (int g = wi.g0; g < wi.g1; ++g) {
          if (!first && !ptx::mbar_wait_bounded(empty_p + 8 * ps, pphase ^ 1, p.wait_limit)) { ok = false; break; }
          const size_t tile0 = tile_base + (size_t)g * wi.R;
          const uint32_t pk = pk0 + ps * kSlot;
          ptx::mbar_arrive_expect_tx(full_p + 8 * ps, wi.R * (kTileB + 64 * kSubs));
          ptx::bulk_g2s(pk, q.packed + tile0 * kTileB, wi.R * kTileB, full_p + 8 * ps);
          ptx::bulk_g2s(pk + kCodeBytes, q.scales + tile0 * (64 * kSubs), wi.R * 64 * kSubs, full_p + 8 * ps);
          if (++ps == P) { ps = 0; pphase ^= 1; first = 0; }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------- producer of the token boxes
    if (lane == 0 && !p.skip_copies) {
      ptx::pdl_wait();
      int s = 0, sa = 0, it = 0;   // token box and barrier of round it
      int wsa = 0, wphase = 0;     // barrier and phase of round it - S, which used the box last
      for (PieceWalk<1> w(p, c0, n_rounds, 0); !w.done() && ok; w.next()) {
        const Piece wi = w.cur();
        const CUtensorMap* map = &p.maps[wi.j];
        for (int g = wi.g0; g < wi.g1; ++g, ++it) {
          if (it >= S) {
            if (!ptx::mbar_wait_bounded(consumed + 8 * wsa, wphase, p.wait_limit)) { ok = false; break; }
            if (++wsa == SA) { wsa = 0; wphase ^= 1; }
          }
          const uint32_t bar = ready + 8 * sa;
          ptx::mbar_arrive_expect_tx(bar, x_round_bytes);
          tma_load_2d(smem0 + s * x_round_bytes, map, g * kGroup, 0, bar);
          tma_load_2d(smem0 + s * x_round_bytes + x_half_bytes, map, g * kGroup + kStageK, 0, bar);
          if (++s == S) s = 0;
          if (++sa == SA) sa = 0;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------- MMA issuer
    uint32_t leader;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
    const uint32_t t_base = __shfl_sync(0xffffffffu, tmem_base, 0);
    const uint32_t idesc = (1u << 4) | ((uint32_t)(p.tok >> 3) << 17) | ((128u >> 4) << 24);
    int s = 0, sa = 0, aphase = 0, lt = 0;
    for (PieceWalk<1> w(p, c0, n_rounds, 0); !w.done() && ok; w.next(), ++lt) {
      if (lt > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait_bounded(acc_empty, (lt - 1) & 1, p.wait_limit))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const Piece wi = w.cur();
      const int rounds = wi.g1 - wi.g0;
      for (int r = 0; r < rounds; ++r) {
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(ready + 8 * sa, aphase, p.wait_limit))) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t x_st = smem0 + s * x_round_bytes;
        const uint32_t a_t = t_base + kBatchAccCols + sa * kRoundCols;
        const uint64_t b_desc = umma_desc_sw128(x_st);
        const uint64_t b_desc2 = umma_desc_sw128(x_st + x_half_bytes);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)  // 16 k = 8 operand columns = 32 bytes of a token row
            umma_f16_ts(t_base, a_t + kk * 8, (kk < 4 ? b_desc : b_desc2) + (uint64_t)((kk & 3) * 2), idesc,
                        (r > 0 || kk > 0) ? 1u : 0u);
          umma_commit(consumed + 8 * sa);
        }
        if (++s == S) s = 0;
        if (++sa == SA) { sa = 0; aphase ^= 1; }
      }
      if (ok && leader) umma_commit(acc_full);
    }
  } else if (warp < kFirstDequantWarp + kBatchDequantWarps) {
    // ------------------------------------------------------------------------- dequantizers
    const int quad = warp & 3;                          // tensor-memory lane quadrant of this warp
    const int jg = (warp - kFirstDequantWarp) >> 2;     // this warp group takes rounds jg, jg + kBatchGroups, ...
    const int n = quad * 32 + lane;                     // weight column of the panel = operand row
    const int t_tile = n >> 4;
    const uint32_t mask_lo = reg_const(kMaskLo), exp_lo = reg_const(kExpLo);
    const uint32_t mask_hi = reg_const(kMaskHi), exp_hi = reg_const(kExpHi);
    // This group takes rounds jg, jg + kBatchGroups, ... of the CTA's range; its position in the three rings is
    // kept for the NEXT round it takes, so that the rounds of the other groups cost it nothing.
    int it0 = 0;                 // rounds before the current piece
    int next = jg;               // the next round this group takes
    int s = jg, sn = 0;          // operand slot of that round and how often the slots have wrapped
    int ps = jg % P, pphase = (jg / P) & 1;  // packed ring position and phase of that round
    for (PieceWalk<1> w(p, c0, n_rounds, 0); !w.done() && ok; w.next()) {
      const Piece wi = w.cur();
      const int R = wi.R;
      auto expand_half = [&](uint32_t pk, int h, uint32_t taddr) {
        expand_half_to_tmem<G, BITS>(pk, h, taddr, t_tile, R, n, mask_lo, exp_lo, mask_hi, exp_hi);
      };
      const int n_piece = wi.g1 - wi.g0;
      for (; next < it0 + n_piece && ok; next += kBatchGroups) {
        {
          // The tensor core must be done with the previous contents of these operand slots.  This
          // wait comes before the one for the packed slot, whose barrier changes waiters (warp
          // groups) from lap to lap: the MMAs retire in order, so it implies that the codes of every
          // round up to six rounds back have landed, and with at least six packed slots no group
          // meets a slot's barrier a whole phase early.
          if (sn > 0 && !ptx::mbar_wait_bounded(consumed + 8 * s, (sn - 1) & 1, p.wait_limit)) { ok = false; break; }
          if (!ptx::mbar_wait_bounded(full_p + 8 * ps, pphase, p.wait_limit)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t pk = pk0 + ps * kSlot;
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + kBatchAccCols + s * kRoundCols;
          expand_half(pk, 0, taddr);
          expand_half(pk, 1, taddr + kAStageCols);
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            ptx::mbar_arrive(ready + 8 * s);
            ptx::mbar_arrive(empty_p + 8 * ps);
          }
        }
        ps += kBatchGroups;
        while (ps >= P) { ps -= P; pphase ^= 1; }
        s += kBatchGroups;
        while (s >= SA) { s -= SA; ++sn; }
      }
      it0 += n_piece;
    }
  } else {
    // ------------------------------------------------------------------------- epilogue
    const int quad = warp & 3;          // the tensor-memory lane quadrant this warp may read
    const int et = tid - (kFirstDequantWarp + kBatchDequantWarps) * 32;  // 0..127 over the epilogue warps
    const int rows_here = p.M;
    const int chunk = lane & 3;         // which 8 columns of the warp's 32
    const uint32_t t_acc = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint32_t stg = smem0 + kOutStageOffset + (uint32_t)(et >> 5) * kOutStageBytes;
    const int nl = quad * 32 + lane;
    ptx::pdl_wait();
    int lt = 0;
    for (PieceWalk<1> w(p, c0, n_rounds, 0); !w.done() && ok; w.next(), ++lt) {
      const Piece wi = w.cur();
      const TcBatchProb& q = p.prob[wi.j];
      const int cols = wi.R * kTileN;
      const bool chunk_ok = quad * 32 + chunk * 8 < cols;  // cols is a multiple of 16
      const bool partial = !(wi.g0 == 0 && wi.g1 == wi.ng);
      // scratch slot of a cut panel: named after the first range boundary inside the panel
      int slot = 0;
      if (partial) {
        const long long start = (long long)q.round_begin + (long long)wi.panel * wi.ng;
        slot = (int)(start * gridDim.x / p.total_rounds);
        while ((long long)p.total_rounds * slot / gridDim.x <= start) ++slot;
      }
      float* tile_ws = p.ws + (size_t)slot * p.tok * 128;
      __half* y_chunk = q.y + (size_t)wi.panel * 128 + quad * 32 + chunk * 8;
      if (!ptx::mbar_wait_bounded(acc_full, lt & 1, p.wait_limit)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int mb = 0; mb < rows_here; mb += 32) {
        uint32_t r[32];
        tmem_ld_32x32(t_acc + mb, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (mb + 32 >= rows_here) {
          // the accumulator is in registers: hand it back before the stores
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(acc_empty);
        }
        if (!partial) {
          // r[e] = this thread's output column at token mb + e: round, transpose through the
          // staging tile and store rows mb .. mb + 31 of the warp's 32 columns, 16 bytes a thread
          __syncwarp();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const unsigned short hv = __half_as_ushort(__float2half_rn(__uint_as_float(r[e])));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(stg + e * 64 + lane * 2), "h"(hv) : "memory");
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int tok = (lane >> 2) + 8 * j;
            const uint4 v = ptx::lds128(stg + tok * 64 + chunk * 16);
            if (chunk_ok && mb + tok < rows_here) *reinterpret_cast<uint4*>(y_chunk + (size_t)(mb + tok) * q.N) = v;
          }
        } else if (nl < cols) {
          // a warp's 32 lanes add into 128 consecutive bytes of the slot
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (mb + e < rows_here) atomicAdd(tile_ws + (mb + e) * 128 + nl, __uint_as_float(r[e]));
        }
      }
      if (partial) {
        // The CTA that completes the panel converts the sums and leaves the slot zero.
        __threadfence();
        ptx::named_bar_sync(2, kEpilogueWarps * 32);
        if (et == 0) {
          const unsigned covered = (unsigned)(wi.g1 - wi.g0);
          const unsigned prev = atomicAdd(p.cnt + slot, covered);
          asm volatile("st.shared.u32 [%0], %1;" ::"r"(last_flag), "r"(prev + covered == (unsigned)wi.ng ? 1u : 0u)
                       : "memory");
        }
        ptx::named_bar_sync(2, kEpilogueWarps * 32);
        uint32_t last;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(last) : "r"(last_flag) : "memory");
        if (last) {
          __threadfence();
          // linear sweep over [rows_here][128] floats: a thread takes 4 columns of a row at a time
          float4* src = reinterpret_cast<float4*>(tile_ws);
          const int n4 = rows_here * 32;
#pragma unroll 1
          for (int i0 = 0; i0 < n4; i0 += 4 * 128) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int idx = i0 + u * 128 + et;
              v[u] = idx < n4 ? __ldcg(src + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int idx = i0 + u * 128 + et;
              if (idx < n4) {
                const int m = idx >> 5, c4 = (idx & 31) * 4;
                __stcg(src + idx, make_float4(0.0f, 0.0f, 0.0f, 0.0f));
                if (c4 < cols) {
                  const __half2 lo = __floats2half2_rn(v[u].x, v[u].y), hi = __floats2half2_rn(v[u].z, v[u].w);
                  uint2 out;
                  out.x = *reinterpret_cast<const uint32_t*>(&lo);
                  out.y = *reinterpret_cast<const uint32_t*>(&hi);
                  *reinterpret_cast<uint2*>(q.y + (size_t)m * q.N + (size_t)wi.panel * 128 + c4) = out;
                }
              }
            }
          }
          if (et == 0) p.cnt[slot] = 0;
        }
        ptx::named_bar_sync(2, kEpilogueWarps * 32);
      }
    }
  }

  if (!ok && lane == 0) atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}


// PAIR: two CTAs of a cluster (an SM pair) share every round: each dequantizes its own panel of a
// pair of panels into its own tensor memory and loads half of the token boxes, and CTA 0 issues
// tcgen05.mma.cta_group::2 (M = 256).  With few tokens an MMA costs about 71 cycles whatever N is
// (measured: the 128 x 16 weight operand has to be fetched anew for every instruction), so one
// instruction for two panels halves the tensor core's time per weight.
template <int G, bool PAIR, int BITS = 4>
__global__ void __launch_bounds__(kBatchThreads, 1)
gemm_tc_batch_pair_kernel(const __grid_constant__ TcBatchParams p) {
  static_assert(BITS == 4 || (BITS == 8 && G == kGroup), "8-bit codes come with groups of 128");
  constexpr int kTileB = BITS == 8 ? 2048 : 1024;   // bytes of a packed tile
  constexpr int kCodeBytes = kPanelTiles * kTileB;  // codes of a slot; the scale words follow them
  const int rank = PAIR ? (int)(blockIdx.x & 1u) : 0;                // CTA rank in the cluster of two
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;  // index of the CTA (pair) among its peers
  const int units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr uint32_t kLeaderMask = PAIR ? 0xFEFFFFFFu : 0xFFFFFFFFu;  // clears the CTA-rank bit of a cluster address
  constexpr int kStep = PAIR ? 2 : 1;
  constexpr int kSubs = kGroup / G;
  constexpr int kSlot = tc_slot_bytes(BITS, G);
  constexpr int SA = kRounds;
  constexpr int PM = kMaxPackedSlots;
  const int S = p.sx;
  const int P = p.pslots;
  const int box_tok = PAIR ? p.tok / 2 : p.tok;                   // token rows this CTA loads per box
  const uint32_t x_half_bytes = (uint32_t)box_tok * kStageK * 2;  // one token box: box_tok rows of 64 k
  const uint32_t x_round_bytes = 2 * x_half_bytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t pk0 = smem0 + (uint32_t)S * x_round_bytes;  // the packed ring follows the token boxes
  const uint32_t bar0 = smem0 + kBarOffset;
  // Round `it` (counted over the whole launch) uses barrier pair it % SA, the operand slot
  // it % SA of tensor memory (64 columns) and token box pair it % S.
  const uint32_t ready = bar0;                  // [SA] token boxes landed and weights dequantized
  const uint32_t consumed = bar0 + 8 * SA;      // [SA] the tensor core is done with the round
  const uint32_t full_p = consumed + 8 * SA;    // [P] packed chunk has landed
  const uint32_t empty_p = full_p + 8 * PM;     // [P] dequantizers are done with the chunk
  const uint32_t acc_full = empty_p + 8 * PM;   // the piece's accumulator is complete
  const uint32_t acc_empty = acc_full + 8;      // the epilogue has drained it
  const uint32_t tmem_slot = acc_empty + 8;
  const uint32_t last_flag = tmem_slot + 4;     // this CTA completed the panel of its partial piece

  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const int lane = tid & 31;
  // this CTA's contiguous range of rounds
  const int c0 = (int)((long long)p.total_rounds * unit / units);
  const int c1 = (int)((long long)p.total_rounds * (unit + 1) / units);
  const int n_rounds = c1 - c0;

  if (tid == 0) {
    for (int s = 0; s < SA; ++s) {
      ptx::mbar_init(ready + 8 * s, PAIR ? 9 : 5);  // four dequantizer warps (per CTA) + the token producer
      ptx::mbar_init(consumed + 8 * s, 1);
    }
    for (int s = 0; s < P; ++s) {
      ptx::mbar_init(full_p + 8 * s, 1);
      ptx::mbar_init(empty_p + 8 * s, 4);
    }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, (PAIR ? 2 : 1) * kEpilogueWarps);
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if constexpr (PAIR) {
    // both CTAs' barriers exist before either signals the other's
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
  // Programmatic dependent launch: only weights are touched before griddepcontrol.wait (the token
  // producer waits before its first read of x, the epilogue before its first write).
  ptx::pdl_launch_dependents();

  bool ok = true;
  if (warp == 0) {
    // ------------------------------------------------- producer of packed codes and scale words
    if (lane == 0 && !p.skip_copies) {
      int ps = 0, pphase = 0, first = 1;
      for (PieceWalk<kStep> w(p, c0, n_rounds, rank); !w.done() && ok; w.next()) {
        const Piece wi = w.cur();
        const TcBatchProb& q = p.prob[wi.j];
        const size_t tile_base = (size_t)wi.panel * kPanelTiles * wi.ng;
        for (int g = wi.g0; g < wi.g1; ++g) {
          if (!first && !ptx::mbar_wait_bounded(empty_p + 8 * ps, pphase ^ 1, p.wait_limit)) { ok = false; break; }
          const size_t tile0 = tile_base + (size_t)g * wi.R;
          const uint32_t pk = pk0 + ps * kSlot;
          if (wi.R > 0) {
            ptx::mbar_arrive_expect_tx(full_p + 8 * ps, wi.R * (kTileB + 64 * kSubs));
            ptx::bulk_g2s(pk, q.packed + tile0 * kTileB, wi.R * kTileB, full_p + 8 * ps);
            ptx::bulk_g2s(pk + kCodeBytes, q.scales + tile0 * (64 * kSubs), wi.R * 64 * kSubs, full_p + 8 * ps);
          } else {
            ptx::mbar_arrive(full_p + 8 * ps);  // the missing partner of an odd last panel: zeros are fed
          }
          if (++ps == P) { ps = 0; pphase ^= 1; first = 0; }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------- producer of the token boxes
    if (lane == 0 && !p.skip_copies) {
      ptx::pdl_wait();
      int s = 0, sa = 0, it = 0;   // token box and barrier of round it
      int wsa = 0, wphase = 0;     // barrier and phase of round it - S, which used the box last
      for (PieceWalk<kStep> w(p, c0, n_rounds, rank); !w.done() && ok; w.next()) {
        const Piece wi = w.cur();
        const CUtensorMap* map = &p.maps[wi.j];
        for (int g = wi.g0; g < wi.g1; ++g, ++it) {
          if (it >= S) {
            if (!ptx::mbar_wait_bounded(consumed + 8 * wsa, wphase, p.wait_limit)) { ok = false; break; }
            if (++wsa == SA) { wsa = 0; wphase ^= 1; }
          }
          const uint32_t bar = (ready + 8 * sa) & kLeaderMask;
          if constexpr (PAIR) {
            // CTA 0 announces the bytes of both CTAs' boxes; either CTA's copies complete on CTA 0's barrier
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar, 2 * x_round_bytes);
            tma_load_2d_pair(smem0 + s * x_round_bytes, map, g * kGroup, rank * box_tok, bar);
            tma_load_2d_pair(smem0 + s * x_round_bytes + x_half_bytes, map, g * kGroup + kStageK, rank * box_tok, bar);
          } else {
            ptx::mbar_arrive_expect_tx(bar, x_round_bytes);
            tma_load_2d(smem0 + s * x_round_bytes, map, g * kGroup, 0, bar);
            tma_load_2d(smem0 + s * x_round_bytes + x_half_bytes, map, g * kGroup + kStageK, 0, bar);
          }
          if (++s == S) s = 0;
          if (++sa == SA) sa = 0;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------- MMA issuer
    uint32_t leader;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
    const uint32_t t_base = __shfl_sync(0xffffffffu, tmem_base, 0);
    const uint32_t idesc = (1u << 4) | ((uint32_t)(p.tok >> 3) << 17) | (((PAIR ? 256u : 128u) >> 4) << 24);
    int s = 0, sa = 0, aphase = 0, lt = 0;
    // only CTA 0 of a pair issues
    for (PieceWalk<kStep> w(p, c0, PAIR && rank != 0 ? 0 : n_rounds, rank); !w.done() && ok; w.next(), ++lt) {
      if (lt > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait_bounded(acc_empty, (lt - 1) & 1, p.wait_limit))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const Piece wi = w.cur();
      const int rounds = wi.g1 - wi.g0;
      for (int r = 0; r < rounds; ++r) {
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(ready + 8 * sa, aphase, p.wait_limit))) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t x_st = smem0 + s * x_round_bytes;
        const uint32_t a_t = t_base + kBatchAccCols + sa * kRoundCols;
        const uint64_t b_desc = umma_desc_sw128(x_st);
        const uint64_t b_desc2 = umma_desc_sw128(x_st + x_half_bytes);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {  // 16 k = 8 operand columns = 32 bytes of a token row
            if constexpr (PAIR)
              umma_f16_ts_pair(t_base, a_t + kk * 8, (kk < 4 ? b_desc : b_desc2) + (uint64_t)((kk & 3) * 2), idesc,
                               (r > 0 || kk > 0) ? 1u : 0u);
            else
              umma_f16_ts(t_base, a_t + kk * 8, (kk < 4 ? b_desc : b_desc2) + (uint64_t)((kk & 3) * 2), idesc,
                          (r > 0 || kk > 0) ? 1u : 0u);
          }
          if constexpr (PAIR) umma_commit_pair(consumed + 8 * sa); else umma_commit(consumed + 8 * sa);
        }
        if (++s == S) s = 0;
        if (++sa == SA) { sa = 0; aphase ^= 1; }
      }
      if (ok && leader) {
        if constexpr (PAIR) umma_commit_pair(acc_full); else umma_commit(acc_full);
      }
    }
  } else if (warp < kFirstDequantWarp + kBatchDequantWarps) {
    // ------------------------------------------------------------------------- dequantizers
    const int quad = warp & 3;                          // tensor-memory lane quadrant of this warp
    const int jg = (warp - kFirstDequantWarp) >> 2;     // this warp group takes rounds jg, jg + kBatchGroups, ...
    const int n = quad * 32 + lane;                     // weight column of the panel = operand row
    const int t_tile = n >> 4;
    const uint32_t mask_lo = reg_const(kMaskLo), exp_lo = reg_const(kExpLo);
    const uint32_t mask_hi = reg_const(kMaskHi), exp_hi = reg_const(kExpHi);
    // This group takes rounds jg, jg + kBatchGroups, ... of the CTA's range; its position in the three rings is
    // kept for the NEXT round it takes, so that the rounds of the other groups cost it nothing.
    int it0 = 0;                 // rounds before the current piece
    int next = jg;               // the next round this group takes
    int s = jg, sn = 0;          // operand slot of that round and how often the slots have wrapped
    int ps = jg % P, pphase = (jg / P) & 1;  // packed ring position and phase of that round
    for (PieceWalk<kStep> w(p, c0, n_rounds, rank); !w.done() && ok; w.next()) {
      const Piece wi = w.cur();
      const int R = wi.R;
      auto expand_half = [&](uint32_t pk, int h, uint32_t taddr) {
        expand_half_to_tmem<G, BITS>(pk, h, taddr, t_tile, R, n, mask_lo, exp_lo, mask_hi, exp_hi);
      };
      const int n_piece = wi.g1 - wi.g0;
      for (; next < it0 + n_piece && ok; next += kBatchGroups) {
        {
          // The tensor core must be done with the previous contents of these operand slots.  This
          // wait comes before the one for the packed slot, whose barrier changes waiters (warp
          // groups) from lap to lap: the MMAs retire in order, so it implies that the codes of every
          // round up to six rounds back have landed, and with at least six packed slots no group
          // meets a slot's barrier a whole phase early.
          if (sn > 0 && !ptx::mbar_wait_bounded(consumed + 8 * s, (sn - 1) & 1, p.wait_limit)) { ok = false; break; }
          if (!ptx::mbar_wait_bounded(full_p + 8 * ps, pphase, p.wait_limit)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t pk = pk0 + ps * kSlot;
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + kBatchAccCols + s * kRoundCols;
          expand_half(pk, 0, taddr);
          expand_half(pk, 1, taddr + kAStageCols);
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster((ready + 8 * s) & kLeaderMask); else ptx::mbar_arrive(ready + 8 * s);
            ptx::mbar_arrive(empty_p + 8 * ps);
          }
        }
        ps += kBatchGroups;
        while (ps >= P) { ps -= P; pphase ^= 1; }
        s += kBatchGroups;
        while (s >= SA) { s -= SA; ++sn; }
      }
      it0 += n_piece;
    }
  } else {
    // ------------------------------------------------------------------------- epilogue
    const int quad = warp & 3;          // the tensor-memory lane quadrant this warp may read
    const int et = tid - (kFirstDequantWarp + kBatchDequantWarps) * 32;  // 0..127 over the epilogue warps
    const int rows_here = p.M;
    const int chunk = lane & 3;         // which 8 columns of the warp's 32
    const uint32_t t_acc = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint32_t stg = smem0 + kOutStageOffset + (uint32_t)(et >> 5) * kOutStageBytes;
    const int nl = quad * 32 + lane;
    ptx::pdl_wait();
    int lt = 0;
    for (PieceWalk<kStep> w(p, c0, n_rounds, rank); !w.done() && ok; w.next(), ++lt) {
      const Piece wi = w.cur();
      const TcBatchProb& q = p.prob[wi.j];
      const int cols = wi.R * kTileN;
      const bool chunk_ok = quad * 32 + chunk * 8 < cols;  // cols is a multiple of 16
      const bool partial = !(wi.g0 == 0 && wi.g1 == wi.ng);
      // scratch slot of a cut panel: named after the first range boundary inside the panel
      int slot = 0;
      if (partial) {
        const long long start = (long long)q.round_begin + (long long)(wi.panel / kStep) * wi.ng;
        slot = (int)(start * units / p.total_rounds);
        while ((long long)p.total_rounds * slot / units <= start) ++slot;
        slot = slot * kStep + rank;  // either CTA of a pair has its own panel, so its own slot
      }
      float* tile_ws = p.ws + (size_t)slot * p.tok * 128;
      __half* y_chunk = q.y + (size_t)wi.panel * 128 + quad * 32 + chunk * 8;
      if (!ptx::mbar_wait_bounded(acc_full, lt & 1, p.wait_limit)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int mb = 0; mb < rows_here; mb += 32) {
        uint32_t r[32];
        tmem_ld_32x32(t_acc + mb, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (mb + 32 >= rows_here) {
          // the accumulator is in registers: hand it back before the stores
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(acc_empty & kLeaderMask); else ptx::mbar_arrive(acc_empty);
          }
        }
        if (!partial) {
          // r[e] = this thread's output column at token mb + e: round, transpose through the
          // staging tile and store rows mb .. mb + 31 of the warp's 32 columns, 16 bytes a thread
          __syncwarp();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const unsigned short hv = __half_as_ushort(__float2half_rn(__uint_as_float(r[e])));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(stg + e * 64 + lane * 2), "h"(hv) : "memory");
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int tok = (lane >> 2) + 8 * j;
            const uint4 v = ptx::lds128(stg + tok * 64 + chunk * 16);
            if (chunk_ok && mb + tok < rows_here) *reinterpret_cast<uint4*>(y_chunk + (size_t)(mb + tok) * q.N) = v;
          }
        } else if (nl < cols) {
          // a warp's 32 lanes add into 128 consecutive bytes of the slot
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (mb + e < rows_here) atomicAdd(tile_ws + (mb + e) * 128 + nl, __uint_as_float(r[e]));
        }
      }
      if (partial) {
        // The CTA that completes the panel converts the sums and leaves the slot zero.
        __threadfence();
        ptx::named_bar_sync(2, kEpilogueWarps * 32);
        if (et == 0) {
          const unsigned covered = (unsigned)(wi.g1 - wi.g0);
          const unsigned prev = atomicAdd(p.cnt + slot, covered);
          asm volatile("st.shared.u32 [%0], %1;" ::"r"(last_flag), "r"(prev + covered == (unsigned)wi.ng ? 1u : 0u)
                       : "memory");
        }
        ptx::named_bar_sync(2, kEpilogueWarps * 32);
        uint32_t last;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(last) : "r"(last_flag) : "memory");
        if (last) {
          __threadfence();
          // linear sweep over [rows_here][128] floats: a thread takes 4 columns of a row at a time
          float4* src = reinterpret_cast<float4*>(tile_ws);
          const int n4 = rows_here * 32;
#pragma unroll 1
          for (int i0 = 0; i0 < n4; i0 += 4 * 128) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int idx = i0 + u * 128 + et;
              v[u] = idx < n4 ? __ldcg(src + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int idx = i0 + u * 128 + et;
              if (idx < n4) {
                const int m = idx >> 5, c4 = (idx & 31) * 4;
                __stcg(src + idx, make_float4(0.0f, 0.0f, 0.0f, 0.0f));
                if (c4 < cols) {
                  const __half2 lo = __floats2half2_rn(v[u].x, v[u].y), hi = __floats2half2_rn(v[u].z, v[u].w);
                  uint2 out;
                  out.x = *reinterpret_cast<const uint32_t*>(&lo);
                  out.y = *reinterpret_cast<const uint32_t*>(&hi);
                  *reinterpret_cast<uint2*>(q.y + (size_t)m * q.N + (size_t)wi.panel * 128 + c4) = out;
                }
              }
            }
          }
          if (et == 0) p.cnt[slot] = 0;
        }
        ptx::named_bar_sync(2, kEpilogueWarps * 32);
      }
    }
  }

  if (!ok && lane == 0) atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if constexpr (PAIR) {
    // neither CTA may free its tensor memory or leave while the other can still reach it
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if constexpr (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

namespace {

constexpr int kBatchPolicySMs = 148;  // most CTAs (and so scratch slots) of a launch
constexpr int kMinRoundsPerCta = 8;   // fewer CTAs rather than ranges too short to fill the pipeline

template <int G, bool PAIR, int BITS = 4>
cudaError_t launch_tc_batch(const TcBatchParams& p, int grid, cudaStream_t stream) {
  // lists of at most 80 tokens take the one-CTA kernel, longer ones the kernel of CTA pairs
  void (*kernel)(const TcBatchParams) = PAIR ? gemm_tc_batch_pair_kernel<G, true, BITS> : gemm_tc_batch_kernel<G, BITS>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemTotal);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kBatchThreads);
  cfg.dynamicSmemBytes = kSmemTotal;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (PAIR) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

}  // namespace

size_t gemm_tc_batch_workspace_bytes() {
  // every CTA but the last can cut one panel: a slot of 128 tokens x 128 columns per CTA, and its counter
  return ((size_t)kBatchPolicySMs * kMaxTcBatchM * 128 * sizeof(float) + (size_t)kBatchPolicySMs * sizeof(unsigned int) +
          255) & ~(size_t)255;
}

cudaError_t launch_gemm_tc_batch(const DecodeProblem* probs, int count, int M, void* workspace, unsigned int* status,
                                 cudaStream_t stream, int group, int bits) {
  if (M <= 0 || M > kMaxTcBatchM) return cudaErrorInvalidValue;
  if (bits == 8 && group != kGroup) return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (sms <= 0 || sms > kBatchPolicySMs) sms = kBatchPolicySMs;
  // Pairs of CTAs from 81 tokens on: measured on ChatGLM2-6B- and Gemma-2B-shaped lists they are
  // 3-7 % faster from 96 tokens, equal at 72-80 and 8 % slower at 32 (the cluster-wide hand-overs
  // cost what the halved MMA count saves).  tl_e0m4_tuning_set("list_pair", 0 / 1) forces the choice.
  const bool pair = tune(kTuneListPair) >= 0 ? tune(kTuneListPair) == 1 : M > 80;
  for (int j0 = 0; j0 < count; j0 += kMaxTcBatch) {
    const int n = count - j0 < kMaxTcBatch ? count - j0 : kMaxTcBatch;
    TcBatchParams p;
    p.status = status;
    p.wait_limit = wait_limit_cycles();
    p.skip_copies = tune(kTuneSkipCopies) == 1;
    p.M = M;
    p.tok = pair ? (M + 31) / 32 * 32 : (M + 15) / 16 * 16;  // the two-CTA MMA takes tokens in steps of 32
    p.count = n;
    const int box_tok = pair ? p.tok / 2 : p.tok;            // token rows of one CTA's box
    long long total = 0;
    for (int j = 0; j < n; ++j) {
      const DecodeProblem& d = probs[j0 + j];
      if (!x_tensor_map(d.x, M, d.K, box_tok, &p.maps[j])) return cudaErrorUnknown;
      TcBatchProb& q = p.prob[j];
      q.packed = reinterpret_cast<const uint8_t*>(d.packed);
      q.scales = reinterpret_cast<const uint8_t*>(d.scales);
      q.y = d.y;
      q.N = (int)d.N;
      q.ng = (int)(d.K / kGroup);
      q.nbs = (int)(d.N / kTileN);
      q.panels = (q.nbs + kPanelTiles - 1) / kPanelTiles;
      q.units = pair ? (q.panels + 1) / 2 : q.panels;
      q.round_begin = (int)total;
      total += (long long)q.units * q.ng;
      if (total > 0x7FFFFFFFLL / 512) return cudaErrorInvalidValue;
    }
    p.total_rounds = (int)total;
    const int round_bytes = box_tok * kStageK * 2 * 2;  // token bytes of one round in one CTA
    p.sx = kXRingBytes / round_bytes;
    if (p.sx > kRounds) p.sx = kRounds;               // both rings share the release barriers
    // 8-bit codes: slots of 17 KB; token boxes give way until six of them fit
    while (bits == 8 && p.sx > 2 && (kOutStageOffset - p.sx * round_bytes) / tc_slot_bytes(8, group) < kRounds) --p.sx;
    p.pslots = (kOutStageOffset - p.sx * round_bytes) / tc_slot_bytes(bits, group);
    if (p.pslots > kMaxPackedSlots) p.pslots = kMaxPackedSlots;
    if (p.pslots < kRounds) return cudaErrorInvalidConfiguration;  // the dequantizers' wait order relies on it
    const int max_units = pair ? sms / 2 : sms;
    int units = (int)((total + kMinRoundsPerCta - 1) / kMinRoundsPerCta);
    if (units > max_units) units = max_units;
    if (units < 1) units = 1;
    const int grid = pair ? 2 * units : units;
    p.ws = static_cast<float*>(workspace);
    p.cnt = reinterpret_cast<unsigned int*>(p.ws + (size_t)kBatchPolicySMs * kMaxTcBatchM * 128);
    cudaError_t e;
    if (bits == 8)
      e = pair ? launch_tc_batch<kGroup, true, 8>(p, grid, stream) : launch_tc_batch<kGroup, false, 8>(p, grid, stream);
    else if (pair)
      e = group == 32   ? launch_tc_batch<32, true>(p, grid, stream)
          : group == 64 ? launch_tc_batch<64, true>(p, grid, stream)
                        : launch_tc_batch<128, true>(p, grid, stream);
    else
      e = group == 32   ? launch_tc_batch<32, false>(p, grid, stream)
          : group == 64 ? launch_tc_batch<64, false>(p, grid, stream)
                        : launch_tc_batch<128, false>(p, grid, stream);
    count_launch();
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

}  // namespace tl
