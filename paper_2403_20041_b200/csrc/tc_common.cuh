// Constants and device helpers shared by the tensor-core kernels (the single-problem kernel and
// the batch kernel): shared-memory and tensor-memory maps, warp roles, the tensor-memory store and
// the MMA whose A operand is read from tensor memory.
#pragma once

#include "common.cuh"
#include "ptx.cuh"
#include "umma.cuh"

namespace tl {

constexpr int kTokTile = 256;             // most tokens per CTA tile; a launch uses a multiple of 16 up to this
constexpr int kStageK = 64;               // k per pipeline stage: half a quantization group
constexpr int kXRingBytes = 5 * 32768;    // shared memory of the token ring: 5 boxes of 256 tokens, more of smaller ones
constexpr int kMaxXStages = 8;            // not more than kAStages: both rings share the release barriers
constexpr int kAStages = 8;               // dequantized weight tiles in tensor memory
constexpr int kPackedSlots = 6;           // with token boxes of 256 tokens; smaller boxes leave room for more
constexpr int kMaxPackedSlots = 24;
// a slot of the packed ring: 8 KB codes + the scale words of 128 k (512 B per group row of the
// tile), padded to a multiple of 1024
__host__ __device__ constexpr int packed_slot_bytes(int group) { return 8192 + (512 * (kGroup / group) + 1023) / 1024 * 1024; }
// the same for every code width: 8-bit codes take 16 KB per 128 k of a panel, 3-bit and 5-bit
// codes 6 KB and 10 KB (groups of 128 only), each followed by 1 KB for the scale words
__host__ __device__ constexpr int tc_slot_bytes(int bits, int group) {
  return bits == 4 ? packed_slot_bytes(group) : kPanelTiles * 256 * bits + 1024;
}
constexpr int kPackedSlotBytes = packed_slot_bytes(kGroup);
constexpr int kPackedOffset = kXRingBytes;
constexpr int kOutStageOffset = kPackedOffset + kPackedSlots * kPackedSlotBytes;
constexpr int kOutStageBytes = 32 * 64;   // per epilogue warp: 32 tokens x 32 columns fp16
constexpr int kBarOffset = kOutStageOffset + 4 * kOutStageBytes;
constexpr int kSmemTotal = kBarOffset + 1024 + 1024;
constexpr int kFirstDequantWarp = 3;
constexpr int kDequantWarps = 16;         // 4 groups of 4 warps; a group covers the 128 lanes of a stage
constexpr int kEpilogueWarps = 4;         // list kernels: one warp per tensor-memory lane quadrant
// The single-problem kernel drains its accumulator with TWO warps per lane quadrant, which take the
// blocks of 32 tokens in turn: the accumulator goes back to the tensor core in half the time.  Its
// eight staging tiles take the last packed slot's room.
constexpr int kEpilogueWarpsTc = 8;
constexpr int kOutStageOffsetTc = kOutStageOffset - (kEpilogueWarpsTc - kEpilogueWarps) * kOutStageBytes;
constexpr int kThreadsTc = (kFirstDequantWarp + kDequantWarps + kEpilogueWarpsTc) * 32;
constexpr int kAccCols = kTokTile;        // tensor-memory columns of the accumulator
constexpr int kAStageCols = kStageK / 2;  // 32 columns: 64 fp16 per lane
constexpr int kTmemCols = 512;            // 256 accumulator + 8 x 32 operand columns
static_assert(kAccCols + kAStages * kAStageCols <= kTmemCols, "tensor memory budget");
static_assert(kSmemTotal <= 232448, "shared memory budget");

__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
      "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
      "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

// The dequantizer of the tensor-core kernels: 64 k of one weight column (thread = column n of the
// panel, `h` = which half of the 128-k round) are expanded from the packed slot at shared address
// `pk`, dequantized exactly as the standalone dequantizer does, (w1 - b) * d with the bias seen
// from the binade the code was completed in, and written as one operand row of 32 tensor-memory
// columns at `taddr`.  Columns of a ragged panel beyond its last tile (t_tile >= R) are fed zeros.
// 4-bit tiles: a column's 64 bytes are consecutive; 8-bit tiles: chunks of 16 rows, 16 bytes per
// column, and one byte permute puts two codes into the halves of a register together with the
// exponent byte of the binade [8, 16).  3-bit and 5-bit tiles: a column's 128 codes are one little-endian
// bit string of 16 * bits bytes; the codes are cut out of it with funnel shifts and completed in the
// binade [2, 4) itself (shift 10 - bits), as the formula of Section 2.3 has it.
template <int G, int BITS>
__device__ __forceinline__ void expand_half_to_tmem(uint32_t pk, int h, uint32_t taddr, int t_tile, int R, int n,
                                                    uint32_t mask_lo, uint32_t exp_lo, uint32_t mask_hi,
                                                    uint32_t exp_hi) {
  constexpr int kSubs = kGroup / G;                       // scale words per column and tile row
  constexpr int kTileB = 256 * BITS;                      // bytes of a packed tile (16 columns x 128 k)
  constexpr int kCodeBytes = kPanelTiles * kTileB;        // codes of a slot; the scale words follow them
  const uint32_t pk_off = t_tile * kTileB + (n & 15) * (BITS == 8 ? 16 : 16 * BITS);
  const __half2 off_lo = __float2half2_rn(126.0f), off_hi = __float2half2_rn(6.0f);
  uint32_t out[32];
  if (t_tile < R) {
    __half2 d2, b2, b_lo, b_hi;
    auto load_scale = [&](int sub) {  // the scale word of group row `sub` of the tile
      const uint32_t sc = ptx::lds32(pk + kCodeBytes + ((t_tile * kSubs + sub) * 16 + (n & 15)) * 4);
      const __half2 db = *reinterpret_cast<const __half2*>(&sc);  // {d, b}
      b2 = __high2half2(db);
      d2 = __low2half2(db);
      b_lo = __hadd2(b2, off_lo);  // bias seen from the [128, 256) binade (exact)
      b_hi = __hadd2(b2, off_hi);  // bias seen from the [8, 16) binade (exact)
    };
    load_scale(h * 64 / G);
    if constexpr (BITS == 8) {
      // 64 codes = four 16-byte chunks; a register of four codes gives two operand words
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const uint4 wv = ptx::lds128(pk + pk_off + (h * 4 + v) * 256);
        const uint32_t words[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t e01 = __byte_perm(words[j], 0x48484848u, 0x4140u);  // {8 + q0 / 128, 8 + q1 / 128}
          uint32_t e23 = __byte_perm(words[j], 0x48484848u, 0x4342u);
          const __half2 r01 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e01), b_hi), d2);
          const __half2 r23 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e23), b_hi), d2);
          out[8 * v + 2 * j + 0] = *reinterpret_cast<const uint32_t*>(&r01);
          out[8 * v + 2 * j + 1] = *reinterpret_cast<const uint32_t*>(&r23);
        }
      }
    } else if constexpr (BITS == 3 || BITS == 5) {
      constexpr int kW = 64 * BITS / 32;  // words of this half of the column's bit string
      uint32_t wds[kW + 1];
#pragma unroll
      for (int i = 0; i < kW; ++i) wds[i] = ptx::lds32(pk + pk_off + h * (8 * BITS) + 4 * i);
      wds[kW] = 0u;
#pragma unroll
      for (int c = 0; c < 64; c += 2) {
        const int at0 = c * BITS, at1 = at0 + BITS;
        const uint32_t q0 = __funnelshift_r(wds[at0 >> 5], wds[(at0 >> 5) + 1], at0 & 31) & ((1u << BITS) - 1u);
        const uint32_t q1 = __funnelshift_r(wds[at1 >> 5], wds[(at1 >> 5) + 1], at1 & 31) & ((1u << BITS) - 1u);
        uint32_t e = 0x40004000u | (q0 << (10 - BITS)) | (q1 << (26 - BITS));  // {2 + q0 / 2^(bits-1), 2 + q1 / ...}
        const __half2 r = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e), b2), d2);
        out[c >> 1] = *reinterpret_cast<const uint32_t*>(&r);
      }
    } else {
      const uint4 wa = ptx::lds128(pk + pk_off + h * 32);
      const uint4 wb = ptx::lds128(pk + pk_off + h * 32 + 16);
      const uint32_t words[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        if (G == 32 && v == 4) load_scale(2 * h + 1);
        const uint32_t w = words[v], w2 = w >> 8;
        uint32_t e01 = and_or(w, mask_lo, exp_lo), e23 = and_or(w, mask_hi, exp_hi);
        uint32_t e45 = and_or(w2, mask_lo, exp_lo), e67 = and_or(w2, mask_hi, exp_hi);
        const __half2 r01 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e01), b_lo), d2);
        const __half2 r23 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e23), b_hi), d2);
        const __half2 r45 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e45), b_lo), d2);
        const __half2 r67 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&e67), b_hi), d2);
        out[4 * v + 0] = *reinterpret_cast<const uint32_t*>(&r01);
        out[4 * v + 1] = *reinterpret_cast<const uint32_t*>(&r23);
        out[4 * v + 2] = *reinterpret_cast<const uint32_t*>(&r45);
        out[4 * v + 3] = *reinterpret_cast<const uint32_t*>(&r67);
      }
    }
  } else {
#pragma unroll
    for (int v = 0; v < 32; ++v) out[v] = 0u;
  }
  // one row of the operand: lane = weight column, 32 columns = 64 consecutive k
  tmem_st_32x32(taddr, out);
}

// D[tmem] (+)= A[tmem] * B[smem]: A is read from tensor memory (row = lane, two fp16 per column).
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The forms of a pair of CTAs (cta_group::2): the MMA spans both CTAs' tensor memory and reads the
// token operand from both CTAs' shared memory; the commit signals the barrier at the same offset
// in both CTAs; the tensor copy writes this CTA's shared memory and completes on a barrier given
// as a cluster address (CTA 0's); the arrive takes a cluster address as well.
__device__ __forceinline__ void umma_f16_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((unsigned short)3)
      : "memory");
}

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

}  // namespace tl
