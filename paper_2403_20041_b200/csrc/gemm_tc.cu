// Tensor-core E0M4 matmul for every M above the GEMV kernel's range (Section 2.2: the
// matrix-matrix implementation, bound by tensor-core throughput at large M).
//
// A CTA tile is one 128-column panel of W times up to 256 tokens, computed as y^T = W^T . x^T:
// the dequantized weights are the 128-row A operand of tcgen05.mma and live in TENSOR MEMORY,
// the tokens are the B operand (N = tokens of the tile, a multiple of 16) in shared memory, and
// the fp32 accumulator in tensor memory has one lane per output column and one column per token.
// Keeping the weights out of shared memory matters: with both operands in shared memory the
// tensor core's operand reads, the TMA writes and the dequantizers' stores together saturate
// the shared-memory pipe at about half of the tensor peak.  Here shared memory only carries the
// token tiles.  M is cut into equal tiles (more and smaller ones when the fewest would leave SMs
// idle); when the output tiles are still too few to fill the GPU, several CTAs share a tile along
// K and add fp32 partial sums into a self-cleaning scratch.
//
// Persistent CTAs (one per SM), 64 k per pipeline stage:
//   * warp 0    : producer of packed codes + scale words (two bulk copies per 128-k group, ring);
//   * warp 2    : producer of the token box (one TMA tensor copy per stage, 128-byte swizzle,
//                 rows beyond M read as zero), a ring of 160 KB: five boxes of 256 tokens, up to
//                 eight smaller ones;
//   * warps 3-18: dequantizers, four warps per stage (one per tensor-memory lane quadrant), four
//                 stages in flight, a ring of eight operand slots in tensor memory.  A thread owns
//                 one weight column: it expands its 32 packed bytes of the stage with the
//                 shift/mask/OR construction of Section 2.3, applies (w1 - b) * d exactly as the
//                 standalone dequantizer does, and writes the 64 fp16 values of its row with one
//                 tcgen05.st;
//   * warp 1    : one thread issues tcgen05.mma (M128 x N(tokens of the tile) x K16, A from tensor
//                 memory, B from shared memory, fp32 accumulate) and commits each stage back to
//                 both rings;
//   * warps 19-26: epilogue, two warps per tensor-memory lane quadrant taking the blocks of 32 tokens in
//                 turn.  tcgen05.ld gives a thread 32 tokens of one output column; the warp
//                 transposes 32 x 32 blocks through a small staging tile so that every thread
//                 stores 16 bytes (eight neighbouring columns of a token), and it hands the
//                 accumulator back as soon as the last block is in registers.  With split-K the
//                 partial tile is added to the scratch instead (a warp adds into 128 consecutive
//                 bytes per instruction) and the CTA that arrives last converts and clears it.
// A stage has one "ready" barrier (token box landed + four dequantizer warps) and one "consumed"
// barrier (tcgen05.commit), shared by the token ring and the weight ring, so the issuing warp does
// one wait and one commit per four MMAs; that warp runs its loop converged, with one elected
// lane issuing, so the MMA operands stay in uniform registers.
// Variants (template arguments of the kernel): SPLIT (several CTAs share a tile along K), EPI (plain
// store, fused residual add, fused SwiGLU), PAIR (two CTAs of a cluster share a work item through
// tcgen05.mma.cta_group::2; see the comment above the kernel), BIG (tiles of at most 128 tokens:
// a pipeline round is a whole 128-k group, i.e. two token boxes, two operand slots and eight MMAs
// per wait and commit, because there the single-thread roles set the pace).  Launches use programmatic dependent
// launch: only weights are touched before griddepcontrol.wait.
// Every mbarrier wait is bounded; a wait that gives up raises the device status word and the
// CTA still releases its tensor memory before it exits.
#include <type_traits>
#include "common.cuh"
#include "ptx.cuh"
#include "umma.cuh"
#include "tc_common.cuh"
#include "tuning.h"

namespace tl {
namespace {

struct TcParams {
  const uint8_t* packed;
  const uint8_t* scales;
  __half* y;
  const __half* add;   // optional fp16 [M, N] added to the product before the one rounding (may be y)
  long long add_stride;  // elements between the addend's token rows: N, or 0 for a bias row shared by all tokens
  unsigned int* status;
  int M, K, N, ng, nbs;
  int tok;      // tokens per CTA tile = N of the MMA: a multiple of 16, at most kTokTile
  int m_tiles;  // ceil(M / tok)
  int sx;       // boxes in the token ring: min(kMaxXStages, kXRingBytes / box bytes)
  int pslots;   // slots of the packed ring, which takes what the token ring leaves (6..24)
  int ksplit;   // CTAs that share one output tile along K (1 = none)
  float* ws;           // split-K scratch: [tile][tok][128 columns] fp32, zero on entry and left zero
  unsigned int* cnt;   // split-K arrival counters: [tile], zero on entry and left zero
  long long wait_limit;  // SM cycles after which a bounded wait gives up
  int skip_copies;       // diagnostics: neither producer issues a copy, so every wait runs out
};

// One unit of work: an output tile (128-column panel x tok tokens) and a slice of the k groups.
struct TcItem {
  int tile, panel, m0, R, g0, g1;
};

// PAIR: the work item belongs to two CTAs of a cluster; `rank` picks this CTA's panel of the two.
template <bool SPLIT, bool PAIR>
__device__ __forceinline__ TcItem tc_item(const TcParams& p, int item, int rank) {
  TcItem w;
  const int ksplit = SPLIT ? p.ksplit : 1;
  w.tile = SPLIT ? item / ksplit : item;
  const int ks = item - w.tile * ksplit;
  w.panel = w.tile / p.m_tiles;
  w.m0 = (w.tile - w.panel * p.m_tiles) * p.tok;
  if (PAIR) w.panel = 2 * w.panel + rank;
  const int rest = p.nbs - kPanelTiles * w.panel;
  w.R = rest < kPanelTiles ? (rest > 0 ? rest : 0) : kPanelTiles;  // 0: the odd panel out of a pair
  w.g0 = SPLIT ? (int)((long long)p.ng * ks / ksplit) : 0;
  w.g1 = SPLIT ? (int)((long long)p.ng * (ks + 1) / ksplit) : p.ng;
  return w;
}

// ADD: the fused residual add (TcParams::add is set); a separate instantiation so that the plain
// kernel keeps its registers.
// PAIR: two CTAs of a cluster (an SM pair) share a work item of 256 weight columns x tok tokens.
// Each CTA dequantizes its own panel into its own tensor memory and loads HALF of the token box;
// CTA 0 issues tcgen05.mma.cta_group::2 (M = 256: 128 accumulator lanes in either CTA, the token
// operand read from both CTAs' shared memory).  Per SM the token bytes halve, so twice as many
// stages fit the same ring and the L2 serves half the traffic.  The stage barriers that the MMA
// warp waits on live in CTA 0 (CTA 1 signals them through the cluster window); the release
// barriers are signalled in both CTAs by a multicast commit.  No TMA multicast is used.
// EPI: 0 plain store, 1 = ADD, 2 = SwiGLU: y[M, N / 2] with y[m, 8 j + c] = silu(Y[m, 16 j + c]) * Y[m, 16 j + 8 + c]
// for c < 8 (gate and up columns interleaved in blocks of eight), in fp32, rounded once.
// BIG: a pipeline round covers a whole 128-k group (two token boxes, two operand slots, eight MMAs
// per wait and commit).  Token tiles of at most 128 tokens use it: their rounds are so short that
// the single-thread roles (one wait, one commit and one pass through the loop per round) set the
// pace, and a round twice as long halves that cost per weight.
// G: quantization group size (128, 64 or 32): a tile row of 128 k carries 128 / G scale words per
// column, and the dequantizers change theirs every G k.
// BITS: 4 (E0M4) or 8 (E0M8: one byte per code, tiles of 2048 bytes, a packed slot of 16 KB; a
// dequantizer moves two neighbouring bytes into the halves of a register with one byte permute
// that also supplies the exponent byte of the binade [8, 16), where a code step is 2^-7).
template <bool SPLIT, int EPI, bool PAIR, bool BIG, int G, int BITS = 4>
__global__ void __launch_bounds__(kThreadsTc, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap x_map, const TcParams p) {
  constexpr bool ADD = EPI == 1;
  constexpr bool GLU = EPI == 2;
  static_assert(!(PAIR && SPLIT), "pairs do not split K");
  static_assert(!(PAIR && BIG), "pairs work in 64-k rounds");
  constexpr int HALVES = BIG ? 2 : 1;  // 64-k halves per round
  constexpr int kSubs = kGroup / G;    // scale words per column and tile row
  static_assert(BITS == 4 || ((BITS == 8 || BITS == 3 || BITS == 5) && G == kGroup), "other widths come with groups of 128");
  constexpr int kTileB = 256 * BITS;                // bytes of a packed tile (16 columns x 128 k)
  constexpr int kCodeBytes = kPanelTiles * kTileB;  // codes of a slot; the scale words follow them
  constexpr int kSlot = tc_slot_bytes(BITS, G);
  const int S = p.sx;
  const int rank = PAIR ? (int)(blockIdx.x & 1u) : 0;              // CTA rank in the cluster of two
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;  // index of the CTA (pair) among its peers
  const int units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr uint32_t kLeaderMask = PAIR ? 0xFEFFFFFFu : 0xFFFFFFFFu;  // clears the CTA-rank bit of a cluster address
  const int box_tok = PAIR ? p.tok / 2 : p.tok;                    // token rows this CTA loads per stage
  const uint32_t x_half_bytes = (uint32_t)box_tok * kStageK * 2;  // one token box: box_tok rows of 64 k
  const uint32_t x_stage_bytes = HALVES * x_half_bytes;
  constexpr int PM = kMaxPackedSlots;
  const int P = p.pslots;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t pk0 = smem0 + (uint32_t)S * x_stage_bytes;  // the packed ring follows the token boxes
  const uint32_t bar0 = smem0 + kBarOffset;
  constexpr int SA = kAStages / HALVES;         // rounds in flight: each takes HALVES operand slots
  constexpr int kRoundCols = HALVES * kAStageCols;
  // Stage `it` (counted over the whole launch) uses barrier pair it % SA, weight slot it % SA of
  // tensor memory and token box it % S of shared memory.
  const uint32_t ready = bar0;                  // [SA] token box landed and weights dequantized
  const uint32_t consumed = bar0 + 8 * SA;      // [SA] the tensor core is done with the stage
  const uint32_t full_p = consumed + 8 * SA;    // [P] packed chunk has landed
  const uint32_t empty_p = full_p + 8 * PM;     // [P] dequantizers are done with the chunk
  const uint32_t acc_full = empty_p + 8 * PM;   // the tile's accumulator is complete
  const uint32_t acc_empty = acc_full + 8;      // the epilogue has drained it
  const uint32_t tmem_slot = acc_empty + 8;
  const uint32_t last_flag = tmem_slot + 4;     // split-K: this CTA arrived last at its tile

  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform for the compiler too
  const int lane = tid & 31;
  const int ng = p.ng;
  const int m_tiles = p.m_tiles;
  const int panels = (p.nbs + kPanelTiles - 1) / kPanelTiles;
  const int total_items = m_tiles * (PAIR ? (panels + 1) / 2 : panels) * (SPLIT ? p.ksplit : 1);

  if (tid == 0) {
    for (int s = 0; s < SA; ++s) {
      ptx::mbar_init(ready + 8 * s, PAIR ? 9 : 5);  // four dequantizer warps (per CTA) + the token producer
      ptx::mbar_init(consumed + 8 * s, 1);
    }
    for (int s = 0; s < P; ++s) {
      ptx::mbar_init(full_p + 8 * s, 1);
      ptx::mbar_init(empty_p + 8 * s, BIG ? 4 : 8);  // the 4 warps of either half's stage read every chunk
    }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, (PAIR ? 2 : 1) * kEpilogueWarpsTc);
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
  // Programmatic dependent launch: the next kernel of the stream may start its own set-up and
  // weight prefetch now.  Here only the weights (never written by a kernel of this library's
  // matmul path) are touched before griddepcontrol.wait: the token producer waits before its first
  // read of x, the epilogue warps before their first write to y or to the split-K scratch.
  ptx::pdl_launch_dependents();

  bool ok = true;
  if (warp == 0) {
    // ------------------------------------------------- producer of packed codes and scale words
    if (lane == 0 && !p.skip_copies) {
      int ps = 0, pphase = 0, first = 1;
      for (int item = unit; item < total_items && ok; item += units) {
        const TcItem wi = tc_item<SPLIT, PAIR>(p, item, rank);
        const int R = wi.R;
        const size_t tile_base = (size_t)wi.panel * kPanelTiles * ng;
        for (int g = wi.g0; g < wi.g1; ++g) {
          if (!first && !ptx::mbar_wait_bounded(empty_p + 8 * ps, pphase ^ 1, p.wait_limit)) { ok = false; break; }
          const size_t tile0 = tile_base + (size_t)g * R;
          const uint32_t pk = pk0 + ps * kSlot;
          if (R > 0) {
            ptx::mbar_arrive_expect_tx(full_p + 8 * ps, R * (kTileB + 64 * kSubs));
            ptx::bulk_g2s(pk, p.packed + tile0 * kTileB, R * kTileB, full_p + 8 * ps);
            ptx::bulk_g2s(pk + kCodeBytes, p.scales + tile0 * (64 * kSubs), R * 64 * kSubs, full_p + 8 * ps);
          } else {
            ptx::mbar_arrive(full_p + 8 * ps);  // the odd panel out of a pair: nothing to fetch, zeros to feed
          }
          if (++ps == P) { ps = 0; pphase ^= 1; first = 0; }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------- producer of the token boxes
    if (lane == 0 && !p.skip_copies) {
      ptx::pdl_wait();
      int s = 0, it = 0;
      for (int item = unit; item < total_items && ok; item += units) {
        const TcItem wi = tc_item<SPLIT, PAIR>(p, item, rank);
        const int m0 = wi.m0;
        for (int kh = 2 * wi.g0; kh < 2 * wi.g1; kh += HALVES, ++it) {
          // the box was last used by stage it - S
          const int prev = it - S;
          if (prev >= 0 && !ptx::mbar_wait_bounded(consumed + 8 * (prev & (SA - 1)), (prev / SA) & 1, p.wait_limit)) {
            ok = false;
            break;
          }
          const uint32_t bar = (ready + 8 * (it & (SA - 1))) & kLeaderMask;
          if constexpr (PAIR) {
            // CTA 0 announces the bytes of both halves; either CTA's copy completes on CTA 0's barrier
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar, 2 * x_stage_bytes);
            tma_load_2d_pair(smem0 + s * x_stage_bytes, &x_map, kh * kStageK, m0 + rank * box_tok, bar);
          } else {
            ptx::mbar_arrive_expect_tx(bar, x_stage_bytes);
            tma_load_2d(smem0 + s * x_stage_bytes, &x_map, kh * kStageK, m0, bar);
            if constexpr (BIG) tma_load_2d(smem0 + s * x_stage_bytes + x_half_bytes, &x_map, (kh + 1) * kStageK, m0, bar);
          }
          if (++s == S) s = 0;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------- MMA issuer
    // The whole warp walks the loop so that every operand of the MMA is warp-uniform (the
    // instruction takes them from uniform registers); one elected lane issues and commits.
    uint32_t leader;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
    const uint32_t t_base = __shfl_sync(0xffffffffu, tmem_base, 0);
    // fp32 accumulate, fp16 operands, K-major; M = 128 weight columns, N = tokens of a tile
    const uint32_t idesc = (1u << 4) | ((uint32_t)(p.tok >> 3) << 17) | (((PAIR ? 256u : 128u) >> 4) << 24);
    int s = 0, sa = 0, aphase = 0, lt = 0;
    if (PAIR && rank != 0) lt = total_items;  // only CTA 0 of a pair issues
    for (int item = PAIR && rank != 0 ? total_items : unit; item < total_items && ok; item += units, ++lt) {
      if (lt > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait_bounded(acc_empty, (lt - 1) & 1, p.wait_limit))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const TcItem wi = tc_item<SPLIT, PAIR>(p, item, rank);
      const int stages = (2 / HALVES) * (wi.g1 - wi.g0);
      for (int kh = 0; kh < stages; ++kh) {
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(ready + 8 * sa, aphase, p.wait_limit))) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t x_st = smem0 + s * x_stage_bytes;
        const uint32_t a_t = t_base + kAccCols + sa * kRoundCols;
        const uint64_t b_desc = umma_desc_sw128(x_st);
        const uint64_t b_desc2 = BIG ? umma_desc_sw128(x_st + x_half_bytes) : b_desc;  // the round's second token box
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < HALVES * kStageK / 16; ++kk)  // 16 k = 8 operand columns = 32 bytes of a token row
            if constexpr (PAIR)
              umma_f16_ts_pair(t_base, a_t + kk * 8, b_desc + (uint64_t)(kk * 2), idesc, (kh > 0 || kk > 0) ? 1u : 0u);
            else
              umma_f16_ts(t_base, a_t + kk * 8, (kk < 4 ? b_desc : b_desc2) + (uint64_t)((kk & 3) * 2), idesc,
                          (kh > 0 || kk > 0) ? 1u : 0u);
          if constexpr (PAIR) umma_commit_pair(consumed + 8 * sa); else umma_commit(consumed + 8 * sa);
        }
        if (++s == S) s = 0;
        if (++sa == SA) { sa = 0; aphase ^= 1; }
      }
      if (ok && leader) {
        if constexpr (PAIR) umma_commit_pair(acc_full); else umma_commit(acc_full);
      }
    }
  } else if (warp < kFirstDequantWarp + kDequantWarps) {
    // ------------------------------------------------------------------------- dequantizers
    const int quad = warp & 3;                          // tensor-memory lane quadrant of this warp
    const int jg = (warp - kFirstDequantWarp) >> 2;     // this warp group takes stages jg, jg + 4, ...
    const int n = quad * 32 + lane;                     // weight column of the panel = operand row
    const int t_tile = n >> 4;
    const uint32_t mask_lo = reg_const(kMaskLo), exp_lo = reg_const(kExpLo);
    const uint32_t mask_hi = reg_const(kMaskHi), exp_hi = reg_const(kExpHi);
    int it = 0;                  // running stage counter over all items
    int ps = 0, pphase = 0;      // packed ring position of the current group
    for (int item = unit; item < total_items && ok; item += units) {
      const TcItem wi = tc_item<SPLIT, PAIR>(p, item, rank);
      const int R = wi.R;
      for (int g = wi.g0; g < wi.g1 && ok; ++g) {
        auto expand_half = [&](uint32_t pk, int h, uint32_t taddr) {
          expand_half_to_tmem<G, BITS>(pk, h, taddr, t_tile, R, n, mask_lo, exp_lo, mask_hi, exp_hi);
        };
        for (int h = 0; h < 2; h += HALVES, ++it) {
          if ((it & 3) != jg) continue;
          const int s = it & (SA - 1), sn = it / SA;
          // The tensor core must be done with the previous contents of this operand slot.  This wait
          // comes first: a packed slot's barrier is waited on by a different warp group every time
          // round the ring, with nothing but a phase parity to tell the rounds apart, so a group
          // must not look at it a whole phase early (a parity wait on a phase that has not begun
          // passes at once).  The MMAs run in order, so once the round that last used this operand
          // slot, four rounds of 128 k ago, has been consumed, the codes of every round up to that
          // one have landed; with at least four packed slots that includes the previous round of
          // the packed slot waited on next.
          if (sn > 0 && !ptx::mbar_wait_bounded(consumed + 8 * s, (sn - 1) & 1, p.wait_limit)) { ok = false; break; }
          if (!ptx::mbar_wait_bounded(full_p + 8 * ps, pphase, p.wait_limit)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t pk = pk0 + ps * kSlot;
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + kAccCols + s * kRoundCols;
          expand_half(pk, h, taddr);
          if constexpr (BIG) expand_half(pk, 1, taddr + kAStageCols);
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster((ready + 8 * s) & kLeaderMask); else ptx::mbar_arrive(ready + 8 * s);
            ptx::mbar_arrive(empty_p + 8 * ps);
          }
        }
        if (++ps == P) { ps = 0; pphase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------------- epilogue
    const int quad = warp & 3;          // the tensor-memory lane quadrant this warp may read
    const int et = tid - (kFirstDequantWarp + kDequantWarps) * 32;  // 0..255 over the epilogue warps
    const int turn = (et >> 5) >> 2;    // which of the quadrant's two warps: it takes blocks turn, turn + 2, ...
    ptx::pdl_wait();
    int lt = 0;
    for (int item = unit; item < total_items && ok; item += units, ++lt) {
      const TcItem wi = tc_item<SPLIT, PAIR>(p, item, rank);
      const int panel = wi.panel, m0 = wi.m0;
      const int cols = wi.R * kTileN;
      const int rows_here = p.M - m0 < p.tok ? p.M - m0 : p.tok;
      const int chunk = lane & 3;                               // which 8 columns of the warp's 32
      const bool chunk_ok = quad * 32 + chunk * 8 < cols;       // cols is a multiple of 16
      // The optional addend: a lane's four 16-byte vectors of a block of 32 tokens (the rows it
      // stores).  They are fetched one block ahead, the first ones before the accumulator is even
      // complete, so that their latency never holds the accumulator.
      const __half* add_chunk =
          (!SPLIT && ADD) ? p.add + (size_t)m0 * p.add_stride + (size_t)panel * 128 + quad * 32 + chunk * 8 : nullptr;
      auto load_add = [&](uint4 (&a)[4], int mb) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int row = mb + (u >> 1) * 16 + (lane >> 2) + 8 * (u & 1);
          a[u] = make_uint4(0u, 0u, 0u, 0u);
          if (chunk_ok && row < rows_here) a[u] = *reinterpret_cast<const uint4*>(add_chunk + (size_t)row * p.add_stride);
        }
      };
      uint4 a_cur[4], a_nxt[4];
      if constexpr (!SPLIT && ADD) load_add(a_cur, 32 * turn);
      if (!ptx::mbar_wait_bounded(acc_full, lt & 1, p.wait_limit)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t t_acc = tmem_base + ((uint32_t)(quad * 32) << 16);
      // Staging tile of this warp: [token 0..31][column 0..31] fp16, so that the global stores are
      // 16 bytes per thread (eight neighbouring columns of one token).
      const uint32_t stg = smem0 + kOutStageOffsetTc + (uint32_t)(et >> 5) * kOutStageBytes;
      __half* y_chunk = p.y + (size_t)panel * 128 + quad * 32 + chunk * 8;
      // r[e] = this thread's output column at token mb + e: round, transpose through the staging
      // tile and store rows mb .. mb + 31 of the warp's 32 columns.
      auto store_block = [&](const uint32_t (&r)[32], int mb, const uint4 (&add)[4]) {
        if constexpr (GLU) {
          // gate column c and up column c + 8 of a 16-column block sit 8 lanes apart.  The two lanes
          // share the work: of every two tokens the gate lane forms the output of the first (it
          // receives the up value), the up lane that of the second (it receives the gate value).
          // The warp's 16 outputs of a token are 32 bytes of the staging tile.
          __syncwarp();
          const bool up_lane = (lane & 8) != 0;
          const uint32_t col2 = ((lane >> 4) * 8 + (lane & 7)) * 2;
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float mine = __uint_as_float(up_lane ? r[e + 1] : r[e]);     // what this lane keeps
            const float give = __uint_as_float(up_lane ? r[e] : r[e + 1]);     // what the partner needs
            const float got = __shfl_xor_sync(0xffffffffu, give, 8);
            const float g = up_lane ? got : mine, u = up_lane ? mine : got;
            const float o = g * __frcp_rn(1.0f + __expf(-g)) * u;
            const unsigned short hv = __half_as_ushort(__float2half_rn(o));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(stg + (e + (up_lane ? 1 : 0)) * 32 + col2), "h"(hv) : "memory");
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int tok = (lane >> 1) + 16 * j, ch = lane & 1;
            const uint4 v = ptx::lds128(stg + tok * 32 + ch * 16);
            if (quad * 32 + ch * 16 < cols && mb + tok < rows_here)
              *reinterpret_cast<uint4*>(p.y + (size_t)(m0 + mb + tok) * (p.N >> 1) + (size_t)panel * 64 + quad * 16 + ch * 8) = v;
          }
        } else if constexpr (!ADD) {
          __syncwarp();  // the previous block's staging reads are done
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const unsigned short hv = __half_as_ushort(__float2half_rn(__uint_as_float(r[e])));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(stg + e * 64 + lane * 2), "h"(hv) : "memory");
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int tok = (lane >> 2) + 8 * j;
            const int m = m0 + mb + tok;
            const uint4 v = ptx::lds128(stg + tok * 64 + chunk * 16);
            // a block of 32 may reach past the tile (tok is a multiple of 16) or past M
            if (chunk_ok && mb + tok < rows_here) *reinterpret_cast<uint4*>(y_chunk + (size_t)m * p.N) = v;
          }
        } else {
          // With an addend the sums stay fp32 through the staging tile (16 tokens at a time, the
          // tile is [16][32] floats then), meet the addend as 16-byte vectors and are rounded once.
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            __syncwarp();
#pragma unroll
            for (int e = 0; e < 16; ++e)
              asm volatile("st.shared.b32 [%0], %1;" ::"r"(stg + e * 128 + lane * 4), "r"(r[half * 16 + e]) : "memory");
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const int tok = (lane >> 2) + 8 * j;
              const int row = mb + half * 16 + tok;
              const float4 lo = ptx::lds128f(stg + tok * 128 + chunk * 32);
              const float4 hi = ptx::lds128f(stg + tok * 128 + chunk * 32 + 16);
              if (chunk_ok && row < rows_here) {
                const size_t at = (size_t)(m0 + row) * p.N;
                const uint4 a = add[half * 2 + j];
                const float2 a0 = __half22float2(*reinterpret_cast<const __half2*>(&a.x));
                const float2 a1 = __half22float2(*reinterpret_cast<const __half2*>(&a.y));
                const float2 a2 = __half22float2(*reinterpret_cast<const __half2*>(&a.z));
                const float2 a3 = __half22float2(*reinterpret_cast<const __half2*>(&a.w));
                const __half2 o0 = __floats2half2_rn(lo.x + a0.x, lo.y + a0.y), o1 = __floats2half2_rn(lo.z + a1.x, lo.w + a1.y);
                const __half2 o2 = __floats2half2_rn(hi.x + a2.x, hi.y + a2.y), o3 = __floats2half2_rn(hi.z + a3.x, hi.w + a3.y);
                uint4 v;
                v.x = *reinterpret_cast<const uint32_t*>(&o0);
                v.y = *reinterpret_cast<const uint32_t*>(&o1);
                v.z = *reinterpret_cast<const uint32_t*>(&o2);
                v.w = *reinterpret_cast<const uint32_t*>(&o3);
                *reinterpret_cast<uint4*>(y_chunk + at) = v;
              }
            }
          }
        }
      };
      // Split-K scratch of the tile: [tok tokens][128 columns] fp32; a warp's 32 lanes add into 128
      // consecutive bytes, which the L2 takes as one request.
      const int nl = quad * 32 + lane;
      float* tile_ws = SPLIT ? p.ws + (size_t)wi.tile * p.tok * 128 : nullptr;
      // this warp's blocks of 32 tokens: turn, turn + 2, ... (the quadrant's other warp takes the rest);
      // a warp without a block hands its share of the accumulator back at once
      if (32 * turn >= rows_here) {
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          if constexpr (PAIR) mbar_arrive_cluster(acc_empty & kLeaderMask); else ptx::mbar_arrive(acc_empty);
        }
      }
#pragma unroll 1
      for (int mb = 32 * turn; mb < rows_here; mb += 64) {
        uint32_t r[32];
        tmem_ld_32x32(t_acc + mb, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (mb + 64 >= rows_here) {
          // this warp's last block is in registers: hand its share of the accumulator back before the stores
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(acc_empty & kLeaderMask); else ptx::mbar_arrive(acc_empty);
          }
        }
        if constexpr (!SPLIT) {
          if constexpr (ADD) {
            if (mb + 64 < rows_here) load_add(a_nxt, mb + 64);
          }
          store_block(r, mb, a_cur);
          if constexpr (ADD) {
#pragma unroll
            for (int u = 0; u < 4; ++u) a_cur[u] = a_nxt[u];
          }
        } else if (nl < cols) {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (mb + e < rows_here) atomicAdd(tile_ws + (mb + e) * 128 + nl, __uint_as_float(r[e]));
        }
      }
      if constexpr (SPLIT) {
        // The CTA that arrives last at the tile converts the sums and leaves the scratch zero.
        __threadfence();
        ptx::named_bar_sync(2, kEpilogueWarpsTc * 32);
        if (et == 0) {
          const unsigned prev = atomicAdd(p.cnt + wi.tile, 1u);
          asm volatile("st.shared.u32 [%0], %1;" ::"r"(last_flag), "r"(prev == (unsigned)p.ksplit - 1 ? 1u : 0u)
                       : "memory");
        }
        ptx::named_bar_sync(2, kEpilogueWarpsTc * 32);
        uint32_t last;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(last) : "r"(last_flag) : "memory");
        if (last) {
          __threadfence();
          if constexpr (GLU) {
            // a thread takes four gate columns of a row and the four up columns 8 further on
            float4* src = reinterpret_cast<float4*>(tile_ws);
            const int units = rows_here * 16;
#pragma unroll 1
            for (int unit = et; unit < units; unit += kEpilogueWarpsTc * 32) {
              const int row = unit >> 4, b = (unit >> 1) & 7, h = unit & 1;
              const int q4 = row * 32 + 4 * b + h;          // float4 index of the gate quad
              const float4 g = __ldcg(src + q4), u = __ldcg(src + q4 + 2);
              __stcg(src + q4, make_float4(0.f, 0.f, 0.f, 0.f));
              __stcg(src + q4 + 2, make_float4(0.f, 0.f, 0.f, 0.f));
              if (16 * b < cols) {
                const __half2 lo = __floats2half2_rn(g.x * __frcp_rn(1.0f + __expf(-g.x)) * u.x, g.y * __frcp_rn(1.0f + __expf(-g.y)) * u.y);
                const __half2 hi = __floats2half2_rn(g.z * __frcp_rn(1.0f + __expf(-g.z)) * u.z, g.w * __frcp_rn(1.0f + __expf(-g.w)) * u.w);
                uint2 out;
                out.x = *reinterpret_cast<const uint32_t*>(&lo);
                out.y = *reinterpret_cast<const uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(p.y + (size_t)(m0 + row) * (p.N >> 1) + (size_t)panel * 64 + 8 * b + 4 * h) = out;
              }
            }
          } else {
          // linear sweep over [rows_here][128] floats: a thread takes 4 columns of a row at a time
            float4* src = reinterpret_cast<float4*>(tile_ws);
            const int n4 = rows_here * 32;
  #pragma unroll 1
            for (int i0 = 0; i0 < n4; i0 += 4 * kEpilogueWarpsTc * 32) {
              float4 v[4];
  #pragma unroll
              for (int u = 0; u < 4; ++u) {
                const int idx = i0 + u * kEpilogueWarpsTc * 32 + et;
                v[u] = idx < n4 ? __ldcg(src + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
  #pragma unroll
              for (int u = 0; u < 4; ++u) {
                const int idx = i0 + u * kEpilogueWarpsTc * 32 + et;
                if (idx < n4) {
                  const int m = m0 + (idx >> 5), c4 = (idx & 31) * 4;
                  __stcg(src + idx, make_float4(0.0f, 0.0f, 0.0f, 0.0f));
                  if (c4 < cols) {
                    if constexpr (ADD) {
                      const uint2 a = *reinterpret_cast<const uint2*>(p.add + (size_t)m * p.add_stride + (size_t)panel * 128 + c4);
                      const float2 a01 = __half22float2(*reinterpret_cast<const __half2*>(&a.x));
                      const float2 a23 = __half22float2(*reinterpret_cast<const __half2*>(&a.y));
                      v[u].x += a01.x;
                      v[u].y += a01.y;
                      v[u].z += a23.x;
                      v[u].w += a23.y;
                    }
                    const __half2 lo = __floats2half2_rn(v[u].x, v[u].y), hi = __floats2half2_rn(v[u].z, v[u].w);
                    uint2 out;
                    out.x = *reinterpret_cast<const uint32_t*>(&lo);
                    out.y = *reinterpret_cast<const uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>(p.y + (size_t)m * p.N + (size_t)panel * 128 + c4) = out;
                  }
                }
              }
            }
          }
          if (et == 0) p.cnt[wi.tile] = 0;
        }
        ptx::named_bar_sync(2, kEpilogueWarpsTc * 32);
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

constexpr int kPolicySMs = 148;  // SM count the split-K policy (and so the scratch size) assumes

struct TcPlan {
  int tok, m_tiles, tiles, ksplit;
  bool pair;  // two CTAs per work item (cta_group::2); tiles then counts panel pairs x token tiles
  bool big;   // pipeline rounds of a whole 128-k group (token tiles of at most 128 tokens)
};

// Equal token tiles, rounded up to the MMA's granularity of 16: as few as 256 tokens each allow,
// or a multiple of that when the fewest leave SMs idle.  When the output tiles would still leave
// SMs idle or fill the last wave badly, several CTAs share a tile along K.  The cut of M and the
// number of k slices minimise a time model in microseconds, fitted to
// measurements on a B200: waves of CTAs x (stages of a slice x time per stage + a fixed cost per
// work item for pipeline fill and drain), plus, when tiles are shared, the last CTA's sweep over
// its tile's scratch and the fp32 additions into the scratch, which the L2 retires at about 0.3
// per picosecond over the whole GPU.
TcPlan tc_plan(int64_t M, int64_t K, int64_t N, int bits = 4) {
  TcPlan pl;
  const int64_t want = (M + kTokTile - 1) / kTokTile;
  const int nbs = (int)(N / kTileN);
  const int panels = (nbs + kPanelTiles - 1) / kPanelTiles;
  const int ng = (int)(K / kGroup);
  const double t_item = 3.5;
  // tl_e0m4_tuning_set("tc_mtiles", 1 / 2 / 4 / 8) fixes the multiple of the fewest token tiles.
  const int64_t mt_set = tune(kTuneTcMtiles);
  const int forced_mult = (mt_set == 1 || mt_set == 2 || mt_set == 4 || mt_set == 8) ? (int)mt_set : 0;
  int best = 1;
  double best_cost = 1e30;
  pl.tok = 0;
  // Token tiles: as few as 256 tokens each allow, or 2, 4, 8 times as many smaller ones when the
  // fewest would leave SMs idle (every CTA of a panel then dequantizes the panel again, on an SM
  // that had nothing to do, and the weights come from L2).
  for (int mult = 1; mult <= 8; mult *= 2) {
    if (forced_mult ? mult != forced_mult : (mult > 1 && panels * want * (mult / 2) >= kPolicySMs)) continue;
    const int64_t cut = want * mult;
    const int tok = (int)(((M + cut - 1) / cut + 15) / 16 * 16);
    if (mult > 1 && tok < 32) break;
    const int m_tiles = (int)((M + tok - 1) / tok);
    const int tiles = panels * m_tiles;
    // time per 64 k of a tile: rounds of a whole group (tiles of at most 128 tokens) cost 0.24 us per
    // 128 k up to 64 tokens and 0.41 us at 128 when most SMs are busy (0.33 us when few are);
    // rounds of 64 k cost 0.22 us each up to 150 tokens
    double t_stage = tok <= 128 ? (tok * 0.0016 > 0.12 ? tok * 0.0016 : 0.12)
                                : (tok * 0.00146 > 0.22 ? tok * 0.00146 : 0.22);
    // 8-bit codes: a stage brings 8 KB per SM, which HBM delivers in 0.2 us when every SM asks
    if (bits == 8 && t_stage < 0.2) t_stage = 0.2;
    for (int ks = 1; ks <= 8 && (ks == 1 || ks * 4 <= ng); ++ks) {
      const long long waves = ((long long)tiles * ks + kPolicySMs - 1) / kPolicySMs;
      double cost = (double)waves * (2.0 * ng / ks * t_stage + t_item);
      if (ks > 1) cost += 1.0 + 0.03 * tok + (double)ks * tiles * tok * 128 / 3.0e5;
      if (cost < best_cost * 0.97) {  // a further slice or cut has to pay for itself
        best_cost = cost;
        best = ks;
        pl.tok = tok;
        pl.m_tiles = m_tiles;
        pl.tiles = tiles;
      }
    }
  }
  const bool fewest_tiles = pl.tok == (int)(((M + want - 1) / want + 15) / 16 * 16);  // M was not cut further
  pl.ksplit = best;
  pl.pair = false;
  // tl_e0m4_tuning_set("ksplit", n) forces n slices where the shape allows them.
  {
    const int64_t f = tune(kTuneKsplit);
    if (f >= 1 && f <= 8 && (f == 1 || f * 4 <= ng)) pl.ksplit = (int)f;
  }
  // Pairs: when nothing is split and there is enough work for every SM pair.  The token tile is
  // then a multiple of 32 (the two-CTA MMA's granularity).
  // tl_e0m4_tuning_set("tc_pair", 0 / 1) forces the choice where the shape allows it.
  const int pair_tok = (int)(((M + want - 1) / want + 31) / 32 * 32);
  const int pair_tiles = ((panels + 1) / 2) * (int)((M + pair_tok - 1) / pair_tok);
  bool pair = pl.ksplit == 1 && fewest_tiles && panels >= 2 && pair_tok <= kTokTile && M > 128 &&
              pair_tiles >= kPolicySMs / 2;
  if (tune(kTuneTcPair) == 0) pair = false;
  if (tune(kTuneTcPair) == 1) pair = pl.ksplit == 1 && fewest_tiles && panels >= 2 && pair_tok <= kTokTile;
  if (pair) {
    pl.pair = true;
    pl.tok = pair_tok;
    pl.m_tiles = (int)((M + pair_tok - 1) / pair_tok);
    pl.tiles = pair_tiles;
  }
  pl.big = !pl.pair && pl.tok <= 128;
  if (tune(kTuneTcBig) == 0) pl.big = false;  // forces rounds of 64 k
  return pl;
}

template <bool SPLIT, int EPI, bool PAIR, bool BIG, int G, int BITS = 4>
cudaError_t launch_tc(const CUtensorMap& map, const TcParams& p, int items, cudaStream_t stream) {
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<SPLIT, EPI, PAIR, BIG, G, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemTotal);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  int sms = 0;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (sms <= 0) sms = kPolicySMs;
  int grid = items < sms ? items : sms;  // persistent: one CTA per SM walks the items
  if (PAIR) {
    const int pairs = sms / 2;
    grid = 2 * (items < pairs ? items : pairs);  // `items` counts work items of a pair
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreadsTc);
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
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<SPLIT, EPI, PAIR, BIG, G, BITS>, map, p);
}

}  // namespace

size_t gemm_tc_workspace_bytes(int64_t M, int64_t K, int64_t N, int bits) {
  const TcPlan pl = tc_plan(M, K, N, bits);
  if (pl.ksplit == 1) return 0;
  return ((size_t)pl.tiles * pl.tok * 128 * sizeof(float) + (size_t)pl.tiles * sizeof(unsigned int) + 255) &
         ~(size_t)255;
}

cudaError_t launch_gemm_tc(const __half* x, const uint32_t* packed, const uint32_t* scales, __half* y,
                           int64_t M, int64_t K, int64_t N, void* workspace, unsigned int* status,
                           cudaStream_t stream, const __half* add, bool swiglu, int group, int64_t add_stride,
                           int bits) {
  const TcPlan pl = tc_plan(M, K, N, bits);
  CUtensorMap map;
  const int box_tok = pl.pair ? pl.tok / 2 : pl.tok;  // token rows of one CTA's box
  if (!x_tensor_map(x, M, K, box_tok, &map)) return cudaErrorUnknown;
  TcParams p;
  p.tok = pl.tok;
  p.m_tiles = pl.m_tiles;
  const int round_bytes = box_tok * kStageK * 2 * (pl.big ? 2 : 1);  // token bytes of one pipeline round
  const int max_sx = pl.big ? kAStages / 2 : kMaxXStages;              // both rings share the release barriers
  p.sx = kXRingBytes / round_bytes;
  if (p.sx > max_sx) p.sx = max_sx;
  if (bits == 8 && p.sx * round_bytes > 4 * 32768) --p.sx;  // the 16 KB slots need the room of a token box
  p.pslots = (kOutStageOffsetTc - p.sx * round_bytes) / tc_slot_bytes(bits, group);
  if (p.pslots > kMaxPackedSlots) p.pslots = kMaxPackedSlots;
  if (p.pslots < 4) return cudaErrorInvalidConfiguration;  // the dequantizers' wait order relies on four slots
  p.ksplit = pl.ksplit;
  p.ws = static_cast<float*>(workspace);
  p.cnt = reinterpret_cast<unsigned int*>(static_cast<float*>(workspace) + (size_t)pl.tiles * pl.tok * 128);
  p.packed = reinterpret_cast<const uint8_t*>(packed);
  p.scales = reinterpret_cast<const uint8_t*>(scales);
  p.y = y;
  p.add = add;
  p.add_stride = add_stride >= 0 ? add_stride : N;
  p.status = status;
  p.wait_limit = wait_limit_cycles();
  p.skip_copies = tune(kTuneSkipCopies) == 1;
  p.M = (int)M;
  p.K = (int)K;
  p.N = (int)N;
  p.ng = (int)(K / kGroup);
  p.nbs = (int)(N / kTileN);
  cudaError_t e;
  const int items = pl.tiles * pl.ksplit;
  auto launch_group = [&](auto epi, auto grp, auto width) {
    constexpr int EPI = decltype(epi)::value;
    constexpr int G = decltype(grp)::value;
    constexpr int BITS = decltype(width)::value;
    if (pl.pair) return launch_tc<false, EPI, true, false, G, BITS>(map, p, pl.tiles, stream);
    if (pl.big)
      return pl.ksplit > 1 ? launch_tc<true, EPI, false, true, G, BITS>(map, p, items, stream)
                           : launch_tc<false, EPI, false, true, G, BITS>(map, p, items, stream);
    return pl.ksplit > 1 ? launch_tc<true, EPI, false, false, G, BITS>(map, p, items, stream)
                         : launch_tc<false, EPI, false, false, G, BITS>(map, p, items, stream);
  };
  auto launch_epi = [&](auto epi) {
    constexpr std::integral_constant<int, 4> four{};
    if (bits == 8) return launch_group(epi, std::integral_constant<int, kGroup>{}, std::integral_constant<int, 8>{});
    if constexpr (decltype(epi)::value == 0) {  // 3-bit and 5-bit codes: the plain product only
      if (bits == 3) return launch_group(epi, std::integral_constant<int, kGroup>{}, std::integral_constant<int, 3>{});
      if (bits == 5) return launch_group(epi, std::integral_constant<int, kGroup>{}, std::integral_constant<int, 5>{});
    }
    if (bits != 4) return cudaErrorInvalidValue;
    if (group == 32) return launch_group(epi, std::integral_constant<int, 32>{}, four);
    if (group == 64) return launch_group(epi, std::integral_constant<int, 64>{}, four);
    return launch_group(epi, std::integral_constant<int, 128>{}, four);
  };
  if (bits != 4 && group != kGroup) return cudaErrorInvalidValue;
  if (add) e = launch_epi(std::integral_constant<int, 1>{});
  else if (swiglu) e = launch_epi(std::integral_constant<int, 2>{});
  else e = launch_epi(std::integral_constant<int, 0>{});
  count_launch();
  return e;
}

}  // namespace tl
