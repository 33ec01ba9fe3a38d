// Decode-stage E0M4 matmul: y[M, N] = x[M, K] . W for a handful of tokens (Section 2.2: the
// vector-matrix implementation; its speed is set by how fast the packed weights stream in).
//
// Shape of the kernel
//   * The packed stream is a sequence of chunks: chunk (panel p, group g) holds the tiles of up
//     to 8 neighbouring column blocks (128 columns) for one 128-k group, 8 KB of codes plus
//     512 B of scale words, contiguous in memory; consecutive g follow each other.  The chunk
//     sequence is cut into equal contiguous ranges, one per CTA (at most two CTAs per SM),
//     either on panel boundaries or, when that would leave SMs idle, anywhere ("stream-K").
//   * A stage of the shared-memory ring holds up to kStageGroups consecutive chunks of one
//     panel.  Warp 8 is the producer: one thread fills the ring with bulk asynchronous copies
//     (TMA) that complete on mbarriers: codes, scale words and the matching slice of every
//     activation row.  Warp 9 adds up each activation row per group (sum_k x, and the total of
//     the binade offsets) as soon as the slice has landed, with one tensor-core product per 32 k
//     against a constant operand (stage_row_sums), and only then hands the stage to the
//     consumers: its time per stage is latency on the ring's critical path.
//   * Warps 0-7 are consumers; warp r owns column block r of the panel and keeps its fp32
//     accumulators in registers over all groups.  Per tile a lane reads 2 x 16 bytes of
//     codes, rebuilds the fp16 numbers 2 + code/8 with the shift/mask/OR of Section 2.3 and
//     feeds them, as the 16-row operand, to mma.sync.m16n8k16 with the tokens as the 8-wide
//     operand (fp32 accumulation).  Scale and bias are applied once per group and column on
//     the fp32 sums:  y += d * (sum_k x*w1 - b * sum_k x)  (plus the binade offsets, see below).
//   * A panel that the CTA covered completely is stored straight from registers; otherwise
//     the sums go to an fp32 scratch with atomics and the CTA that completes the panel (a
//     per-panel chunk counter tells) converts it to fp16 and zeroes the scratch again.
//   * The same kernel serves a batch of independent problems that share M: their chunk
//     sequences are concatenated and cut into one range per CTA, so a whole stack of layers
//     streams through one persistent launch without a bubble between matrices.
//   * Programmatic dependent launch: the kernel lets its successor start at once, and itself
//     prefetches weights (which no predecessor writes) before it waits for its predecessor;
//     activations, outputs and scratch are touched only after that wait.
#include <atomic>
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"
#include "tuning.h"

namespace tl {
namespace {

constexpr int kConsumerWarps = kPanelTiles;          // one warp per column block of a panel
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 64;      // + producer warp + row-sum warp
constexpr int kStageGroups = 4;                      // chunks (k groups) per ring stage
constexpr int kTileBytes = 1024;                     // packed codes of one tile
// scale words of one tile: 16 per group of its 128 rows (one group, or two or four smaller ones)
__host__ __device__ constexpr int tile_scale_bytes(int group) { return 64 * (kGroup / group); }
constexpr int kScaleOffset = kStageGroups * kPanelTiles * kTileBytes;                  // 32768
// the activation rows follow the scale words: at 34816 with groups of 128
__host__ __device__ constexpr int x_offset(int group) { return kScaleOffset + kStageGroups * kPanelTiles * tile_scale_bytes(group); }
// One token's slice of a stage, padded by 32 bytes: together with the rotated chunk order of the
// consumers (see ROT below) the eight lanes of a quarter warp (two tokens x four k slices) read
// 32 different banks.
constexpr int kXRowBytes = kStageGroups * 256 + 32;
constexpr int kWsPad = 16;                           // scratch floats per output column
constexpr int kMaxStages = 4;
// the 64 zero bytes that stand in for missing token rows follow the barriers and two flag words and
// are read with 16-byte loads
static_assert((3 * kMaxStages * 8 + 16) % 16 == 0, "an odd number of ring stages would misalign the zero block");

// Panels whose k groups are shared by the s = 2, 4 or 8 CTAs of (a part of) a cluster meet in
// shared memory instead of the global scratch: every CTA sends the partial sums of tile t to the
// CTA with rank t % s of its group, which adds the s contributions of its 8 / s tiles and stores
// them.  The receiving buffer: [sender x tile: 8][16 columns][8 MT tokens] fp32, and one barrier.
__host__ __device__ constexpr int red_bytes(int mt) { return kPanelTiles * kTileN * 8 * mt * 4; }  // 8 tokens per block of tokens
constexpr int kRedOffset = (3 * kMaxStages + 48) * 8;  // from the barriers: past flags, zero block and row factors
constexpr int kSmemTail = 3 * kMaxStages * 8 + 16 + 64;             // barriers, flags, zero block
// ... row factors, exchange barrier and buffer
__host__ __device__ constexpr int smem_tail_cluster(int mt) { return kRedOffset + 16 + red_bytes(mt); }

constexpr int kSlotFloats = kPanelTiles * kTileN * kWsPad;  // fp32 partial sums of one panel
constexpr int kSlotBytes = kSlotFloats * 4 + 128;           // + the panel's chunk counter
constexpr int kMaxSlots = 320;                              // >= number of CTAs of a launch

struct Prob {
  const __half* x;
  const uint8_t* packed;
  const uint8_t* scales;
  __half* y;
  int K, N, ng;
  int nbs;          // N / 16
  int panels;       // ceil(nbs / 8)
  int chunk_begin;  // first chunk of this problem in the concatenated sequence
};

template <int NB>
struct DecodeParams {
  static constexpr bool kChain = false;
  static constexpr bool kCluster = NB == 1;  // lone problems may be launched as clusters (see red_bytes)
  uint8_t* ws;            // kMaxSlots slots of {fp32 [128][16] partial sums, chunk counter}, zero between calls
  unsigned int* status;   // device status word (0 = fine)
  int M;
  int count;              // problems in this launch (<= NB)
  int total_chunks;
  int unit;               // split granularity in chunks (1, or ng of a lone problem); -s: s CTAs per panel
  int stages;
  int stage_bytes;
  int xsum_offset;        // offset of the kStageGroups x 16 x 2 activation-row sums inside a stage
  Prob prob[NB];
  const __half* add;      // single-problem launches only: optional fp16 [M, N] added to the product
                          // before the one rounding (may be y); NULL otherwise
  long long add_stride;   // elements between the addend's token rows: N, or 0 for a bias row shared by all tokens
  long long wait_limit;   // SM cycles after which a bounded wait gives up
  int skip_copies;        // diagnostics: the producer issues nothing, so every wait runs out
  int cluster;            // CTAs per thread-block cluster of this launch (1 = no clusters)
};

// ---- a chain of steps that may depend on one another (tl_e0m4_matmul_chain)
// The steps are grouped into phases: a phase is a run of steps that do not read what another step
// of the same phase writes, and every phase after the first begins only when ALL earlier steps are
// complete.  Within a phase the chunk sequences of its steps are concatenated and cut over ALL CTAs
// of the launch, exactly as a list of independent problems is; the CTAs walk the phases in order.
// What crosses a phase boundary without waiting is the weight stream: a CTA's producer fills its
// ring with the next phase's codes while the last CTAs are still finishing the current one.
struct ChainProb {
  const __half* x;
  const uint8_t* packed;
  const uint8_t* scales;
  __half* y;
  const __half* add;      // epi 1: fp16 addend, matrix (add_stride = N) or bias row (add_stride = 0)
  long long add_stride;
  int K, N, ng, nbs, panels;
  int chunk_begin;        // first chunk of this step in its PHASE's concatenated sequence
  int epi;                // 0 plain store, 1 addend, 2 SwiGLU over column blocks of 8
  int phase;
  float rms_eps;          // >= 0: every output row is multiplied by rsqrt(mean_k x[m, k]^2 + eps); < 0: no factor
};

struct ChainPhase {
  int first, last;        // steps [first, last) of the launch
  int chunks;             // chunks of the phase
  int unit;               // as DecodeParams::unit, for this phase
  unsigned int wait_target;  // 8 x the panels of all earlier phases: the phase's activations exist once that much is final
};

constexpr int kMaxChain = 128;       // steps per launch (their descriptors travel as kernel parameters)
constexpr int kChainRmsSlots = 8;    // row factors are kept for this many steps (a ring: consumers lag the row-sum warp by less)

struct ChainParams {
  static constexpr bool kChain = true;
  static constexpr bool kCluster = true;
  uint8_t* ws;            // the scratch slots of DecodeParams::ws
  unsigned int* status;
  unsigned int* sync;     // [0] eighths of panels made final so far in this launch, [1] CTAs that have finished; zero between launches
  int M;
  int count;
  int phases;
  int stages;
  int stage_bytes;
  int xsum_offset;
  long long wait_limit;
  int skip_copies;
  int cluster;            // CTAs per thread-block cluster of this launch (1 = no clusters)
  ChainProb prob[kMaxChain];
  ChainPhase phase[kMaxChain];
};

// This CTA's contiguous range [c0, c1) of a sequence of `total` chunks.  unit > 0: equal ranges in
// multiples of `unit` chunks; unit < 0: -unit CTAs per panel of a lone problem with `ng` groups and
// `panels` panels, CTA i of a panel taking groups [ng i / s, ng (i + 1) / s).
__device__ __forceinline__ void cta_range(int total, int unit, int ng, int panels, int& c0, int& c1) {
  if (unit < 0) {
    const int s = -unit;
    const int panel = blockIdx.x / s, i = blockIdx.x - panel * s;
    if (panel >= panels) {
      c0 = c1 = 0;
      return;
    }
    c0 = panel * ng + ng * i / s;
    c1 = panel * ng + ng * (i + 1) / s;
  } else {
    const unsigned int units = (unsigned int)(total / unit), b = blockIdx.x, n = gridDim.x;
    if (units < 0xFFFFFFFFu / (n + 1)) {  // the products fit 32 bits: a 64-bit division costs hundreds of cycles
      c0 = (int)(units * b / n) * unit;
      c1 = (int)(units * (b + 1) / n) * unit;
    } else {
      c0 = (int)((unsigned long long)units * b / n) * unit;
      c1 = (int)((unsigned long long)units * (b + 1) / n) * unit;
    }
  }
}

// silu(g) * u in fp32 (Section 2.2's element-wise fusion for gated MLPs)
__device__ __forceinline__ float swiglu(float g, float u) { return g / (1.0f + __expf(-g)) * u; }

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// First product of a chain: the accumulator input is {e, o, e, o} (the seeds of the even and the
// odd token column of this lane), passed as operands so that no register has to be copied.
__device__ __forceinline__ void mma16816_init(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1, float e, float o) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%10,%11,%10,%11};\n"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(e), "f"(o));
}

// (a & b) | c in one LOP3; b and c are passed in registers so that both stay operands of the
// single instruction.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Loads a 32-bit constant through an opaque move so that the compiler keeps it in a register
// instead of folding it into each use as a second immediate.
__device__ __forceinline__ uint32_t reg_const(uint32_t v) {
  uint32_t r;
  asm volatile("mov.b32 %0, %1;" : "=r"(r) : "r"(v));
  return r;
}

// Section 2.3 allows any binade: a nibble that already sits on fraction bits 3..0 of a half is
// completed by the exponent of [128, 256) (ulp 1/8, value 128 + code/8), one on bits 7..4 by the
// exponent of [8, 16) (value 8 + code/8).  So only one shift per packed word is needed; the
// constant offsets (126 resp. 6 above 2 + code/8) are removed together with the bias, using the
// activation sums over the k that carry each offset.
constexpr uint32_t kMaskLo = 0x000F000Fu, kExpLo = 0x58005800u;  // 128 + code/8
constexpr uint32_t kMaskHi = 0x00F000F0u, kExpHi = 0x48004800u;  // 8 + code/8
constexpr float kOffLo = 126.0f, kOffHi = 6.0f;

// Row sums of one ring stage on the tensor core (the row-sum warp).  Both numbers the consumers
// need per token and group come out of one product with the activations as the 16-row operand:
// against a column of ones the plain sum (it multiplies the bias), against a column of -126 / -6
// minus the total of the constant offsets (it seeds the consumers' accumulator).  A lane's 16
// bytes are eight consecutive k: the halves 0,1 and 4,5 (k % 4 < 2, offset 126) become the first
// eight k of a product, the halves 2,3 and 6,7 (offset 6) its last eight; the order of k inside
// a sum does not matter.
// The 16 rows are filled whatever the token count T (2, 4, 8 or 16 tokens per row set): row r is
// token r % T, and r / T counts through the groups of the stage; with two tokens the eight rows
// left over take the second half of each group's k, and a lane adds the two halves up.  All
// chains run without a branch; a group the stage does not have reads stale bytes of the stage's
// own activation rows and is not stored.  b_first / b_last: the constant operand of this lane.
template <int T>
__device__ __forceinline__ void stage_row_sums(uint32_t x_rows, float* xsum, int M, int groups, int lane,
                                               uint32_t b_first, uint32_t b_last) {
  constexpr int kSets = T * kStageGroups > 16 ? T * kStageGroups / 16 : 1;  // products side by side: 1, 1, 2, 4
  constexpr int kGroupsPerSet = kStageGroups / kSets;
  constexpr bool kHalves = T * kStageGroups < 16;  // T = 2: rows 8..15 are the second half of k
  constexpr int kChunks = kHalves ? 2 : 4;         // 64-byte pieces of k per row
  const int gid = lane >> 2, t = lane & 3;
  // rows gid and gid + 8: token, group inside the set, half of k
  const int m_lo = gid % T, i_lo = gid / T, m_hi = (gid + 8) % T, i_hi = (gid + 8) / T;
  const int g_lo = i_lo % kGroupsPerSet, g_hi = i_hi % kGroupsPerSet;
  const bool has_lo = m_lo < M, has_hi = m_hi < M;
  const uint32_t at_lo = x_rows + m_lo * kXRowBytes + g_lo * 256 + (i_lo / kGroupsPerSet) * 128 + t * 16;
  const uint32_t at_hi = x_rows + m_hi * kXRowBytes + g_hi * 256 + (i_hi / kGroupsPerSet) * 128 + t * 16;
  float c[kSets][2][4];
#pragma unroll
  for (int rs = 0; rs < kSets; ++rs) {
#pragma unroll
    for (int i = 0; i < 4; ++i) c[rs][0][i] = c[rs][1][i] = 0.0f;
#pragma unroll
    for (int j = 0; j < kChunks; ++j) {
      const uint32_t off = rs * kGroupsPerSet * 256 + j * 64;
      const uint4 lo = has_lo ? ptx::lds128(at_lo + off) : make_uint4(0u, 0u, 0u, 0u);
      const uint4 hi = has_hi ? ptx::lds128(at_hi + off) : make_uint4(0u, 0u, 0u, 0u);
      mma16816(c[rs][0], lo.x, hi.x, lo.y, hi.y, b_first, b_last);
      mma16816(c[rs][1], lo.z, hi.z, lo.w, hi.w, b_first, b_last);
    }
  }
  if (t == 0) {
#pragma unroll
    for (int rs = 0; rs < kSets; ++rs) {
      float2 lo = make_float2(c[rs][0][0] + c[rs][1][0], c[rs][0][1] + c[rs][1][1]);
      const float2 hi = make_float2(c[rs][0][2] + c[rs][1][2], c[rs][0][3] + c[rs][1][3]);
      if (kHalves) lo = make_float2(lo.x + hi.x, lo.y + hi.y);
      const int gl = rs * kGroupsPerSet + g_lo, gh = rs * kGroupsPerSet + g_hi;
      if (gl < groups && has_lo) *reinterpret_cast<float2*>(xsum + (gl * 16 + m_lo) * 2) = lo;
      if (!kHalves && gh < groups && has_hi) *reinterpret_cast<float2*>(xsum + (gh * 16 + m_hi) * 2) = hi;
    }
  }
}

// Walks the CTA's chunk range stage by stage, across problems: a stage never crosses a panel end.
// For a chain the walk goes on through the phases: when the CTA's range of one phase is used up it
// moves to the CTA's range of the next phase in which it has any chunks.
template <class PT>
struct StageWalk {
  const PT& p;
  int j, panel, g, left, ng, panels;
  int ph;  // chain: the phase being walked
  __device__ void seek(int c0, int n_chunks, int lo, int hi) {
    // the problem whose chunks contain c0: the last one of [lo, hi] that begins at or before it
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (p.prob[mid].chunk_begin <= c0) lo = mid; else hi = mid - 1;
    }
    j = lo;
    ng = p.prob[j].ng;
    panels = p.prob[j].panels;
    const int off = c0 - p.prob[j].chunk_begin;
    panel = off / ng;
    g = off - panel * ng;
    left = n_chunks;
  }
  __device__ void next_phase() {
    if constexpr (PT::kChain) {
      left = 0;
      while (++ph < p.phases) {
        const ChainPhase& f = p.phase[ph];
        int c0, c1;
        cta_range(f.chunks, f.unit, p.prob[f.first].ng, p.prob[f.first].panels, c0, c1);
        if (c1 > c0) {
          seek(c0, c1 - c0, f.first, f.last - 1);
          return;
        }
      }
    }
  }
  // a list of independent problems: the range [c0, c0 + n_chunks) of the one sequence
  __device__ StageWalk(const PT& p_, int c0, int n_chunks) : p(p_), ph(0) { seek(c0, n_chunks, 0, p.count - 1); }
  // a chain: from the first phase on
  __device__ explicit StageWalk(const PT& p_) : p(p_), j(0), panel(0), g(0), left(0), ng(1), panels(1), ph(-1) { next_phase(); }
  __device__ bool done() const { return left <= 0; }
  __device__ int groups() const {
    int n = ng - g;
    n = n < kStageGroups ? n : kStageGroups;
    return n < left ? n : left;
  }
  __device__ void next() {
    const int n = groups();
    g += n;
    left -= n;
    if (g == ng) {
      g = 0;
      if (++panel == panels && left > 0) {
        panel = 0;
        ++j;
        ng = p.prob[j].ng;
        panels = p.prob[j].panels;
      }
    }
    if (PT::kChain && left <= 0) next_phase();
  }
};

// MT = number of 8-token blocks (1: M <= 8, 2: M <= 16).
// ROT: lanes that own k slices 2 and 3 of a group take the four 16-byte chunks of their slice (and
// the four packed words that go with them) in the order 1,2,3,0.  The contraction does not care
// about the order, and it makes the activation loads of several tokens free of bank conflicts;
// it costs eight selects per tile, so launches of fewer than five tokens do without it.
// ADD: the fused residual add of single-problem launches (DecodeParams::add); its own instantiation,
// because this kernel's speed depends on the exact code the plain one compiles to.
// EPI: 0 plain store, 1 = ADD, 2 = SwiGLU over column blocks of 8 (see the epilogue).
// G: quantization group size.  With 128 the scale and the bias are factored out of the tensor-core
// sums (one fused multiply-add per group and output).  Groups of 64 or 32 rows do not line up
// with the k a tensor-core step covers (it takes 8 k from each 32-wide slice of the tile row), so
// there every lane dequantizes its own slice — which lies in ONE group — to fp16 in registers,
// (w1 - b) * d exactly as the standalone dequantizer does, and the sums need no correction.
// PT: DecodeParams<NB> (a list of independent problems) or ChainParams (steps in phases, see above).
template <int MT, class PT, bool ROT, int EPI, int G>
__global__ void __launch_bounds__(kThreads, 2)
gemv_decode_kernel(const __grid_constant__ PT p) {
  constexpr bool CHAIN = PT::kChain;
  constexpr int kTileScaleBytes = tile_scale_bytes(G);
  constexpr int kXOffset = x_offset(G);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) &
                                             ~static_cast<uintptr_t>(127));
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + (size_t)p.stages * p.stage_bytes);
  volatile int* flags = reinterpret_cast<volatile int*>(bars + 3 * kMaxStages);
  const uint32_t zero_block = ptx::smem_u32(bars + 3 * kMaxStages + 2);  // 64 zero bytes
  // chain: row factors of the last kChainRmsSlots steps, [slot][8 tokens], and the step each slot holds
  float* rms_val = reinterpret_cast<float*>(bars + 3 * kMaxStages + 10);
  volatile int* rms_step = reinterpret_cast<volatile int*>(rms_val + kChainRmsSlots * 8);
  const uint32_t red_bar = ptx::smem_u32(bars) + kRedOffset;   // cluster launches: the exchange barrier ...
  const uint32_t red_buf = red_bar + 16;                       // ... and the buffer the group's CTAs write into

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const uint32_t full0 = ptx::smem_u32(bars);                   // codes + scales + row sums ready
  const uint32_t empty0 = ptx::smem_u32(bars + kMaxStages);     // consumers are done with a stage
  const uint32_t xbar0 = ptx::smem_u32(bars + 2 * kMaxStages);  // activation slice has landed
  const int S = p.stages;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      ptx::mbar_init(full0 + 8 * s, 2);
      ptx::mbar_init(empty0 + 8 * s, kConsumerWarps);
      ptx::mbar_init(xbar0 + 8 * s, 1);
    }
    flags[0] = 0;
    if constexpr (PT::kCluster) {
      if (p.cluster > 1) ptx::mbar_init(red_bar, 1);
    }
    ptx::fence_mbar_init();
  }
  if (tid < 16) reinterpret_cast<uint32_t*>(bars + 3 * kMaxStages + 2)[tid] = 0u;
  if (CHAIN && tid < kChainRmsSlots) rms_step[tid] = -1;
  __syncthreads();
  // Every CTA's exchange barrier has to exist before a neighbour arrives on it.  All threads arrive
  // at the cluster barrier here and wait for it where they would be idle anyway (cluster_ready):
  // the producer after it has requested its first stages, everybody else at once.
  [[maybe_unused]] const bool clustered = PT::kCluster && p.cluster > 1;
  if constexpr (PT::kCluster) {
    if (clustered) ptx::cluster_arrive_release();
  }
  auto cluster_ready = [&]() {
    if constexpr (PT::kCluster) {
      if (clustered) ptx::cluster_wait_acquire();
    }
  };
  ptx::pdl_launch_dependents();

  // this CTA's contiguous range of chunks (a chain has one per phase: see StageWalk)
  int c0 = 0, c1 = 0;
  if constexpr (!CHAIN) {
    cta_range(p.total_chunks, p.unit, p.prob[0].ng, p.prob[0].panels, c0, c1);
    if (c1 <= c0) {
      cluster_ready();
      return;
    }
  }
  const int n_chunks = c1 - c0;
  const int M = p.M;
  // one walk per warp role; all roles of a CTA walk the same stages in the same order
  auto make_walk = [&]() {
    if constexpr (CHAIN) return StageWalk<PT>(p); else return StageWalk<PT>(p, c0, n_chunks);
  };

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------------- producer
    if (lane != 0 || p.skip_copies) {
      cluster_ready();
      return;
    }
    const uint32_t ring_s = ptx::smem_u32(ring);
    auto issue_w = [&](const StageWalk<PT>& w, int s) {
      const auto& q = p.prob[w.j];
      const int rest = q.nbs - kPanelTiles * w.panel;
      const int R = rest < kPanelTiles ? rest : kPanelTiles;
      const int tiles = w.groups() * R;
      const size_t tile0 = (size_t)w.panel * kPanelTiles * w.ng + (size_t)w.g * R;
      const uint32_t st = ring_s + s * p.stage_bytes;
      const uint32_t bar = full0 + 8 * s;
      ptx::mbar_arrive_expect_tx(bar, tiles * (kTileBytes + kTileScaleBytes));
      ptx::bulk_g2s(st, q.packed + tile0 * kTileBytes, tiles * kTileBytes, bar);
      ptx::bulk_g2s(st + kScaleOffset, q.scales + tile0 * kTileScaleBytes, tiles * kTileScaleBytes, bar);
    };
    auto issue_x = [&](const StageWalk<PT>& w, int s) {
      const auto& q = p.prob[w.j];
      const uint32_t st = ring_s + s * p.stage_bytes + kXOffset;
      const uint32_t bar = xbar0 + 8 * s;
      const uint32_t bytes = w.groups() * 256;
      ptx::mbar_arrive_expect_tx(bar, M * bytes);
      for (int m = 0; m < M; ++m)
        ptx::bulk_g2s(st + m * kXRowBytes, q.x + (size_t)m * q.K + (size_t)w.g * kGroup, bytes, bar);
    };

    if constexpr (CHAIN) {
      // One thread, two cursors over the same walk.  The weight cursor runs ahead: it refills a stage
      // as soon as the consumers release it, whatever phase the stage belongs to, so the codes of
      // the next phase stream in while the current one is being finished.  The activation cursor
      // follows: the slice of a stage is requested once its stage holds the weights AND every
      // earlier phase is complete (the counter of final panels has reached the phase's target),
      // because the slice is some earlier step's output.  Neither cursor blocks the other: both
      // conditions are probed without waiting.
      cluster_ready();
      StageWalk<PT> w = make_walk();
      StageWalk<PT> wx = w;
      int iw = 0, ix = 0;            // stages whose weights / activations have been requested
      int sw = 0, pw = 0, sx = 0;    // ring positions; pw: parity of the release the weight cursor needs next
      unsigned int seen = 0;         // final panels observed so far
      bool synced = false;           // pdl_wait done (before the first activation request)
      long long t0 = clock64();
      while (!wx.done()) {
        bool progress = false;
        if (!w.done() && (iw < S || ptx::mbar_test_wait(empty0 + 8 * sw, pw))) {
          issue_w(w, sw);
          w.next();
          ++iw;
          if (++sw == S) {
            sw = 0;
            if (iw > S) pw ^= 1;
          }
          progress = true;
        }
        if (ix < iw) {
          if (!synced) {
            ptx::pdl_wait();
            synced = true;
          }
          const unsigned int target = p.phase[wx.ph].wait_target;
          if (seen < target) {
            seen = ptx::ld_acquire_gpu(p.sync);
            if (seen >= target) ptx::fence_proxy_async_all();
          }
          if (seen >= target) {
            issue_x(wx, sx);
            wx.next();
            ++ix;
            if (++sx == S) sx = 0;
            progress = true;
          }
        }
        if (progress) {
          t0 = clock64();
        } else if (clock64() - t0 > p.wait_limit) {
          atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
          return;
        }
      }
      return;
    }
    // weights and scales of the first stages do not depend on the previous kernel
    StageWalk<PT> w = make_walk();
    StageWalk<PT> wx = w;
    int issued = 0;
    for (; issued < S && !w.done(); ++issued) {
      issue_w(w, issued);
      w.next();
    }
    cluster_ready();
    ptx::pdl_wait();
    for (int i = 0; i < issued; ++i) {
      issue_x(wx, i);
      wx.next();
    }
    // steady state: refill a stage as soon as the consumers have released it
    int s = 0, phase = 0;
    while (!w.done()) {
      if (!ptx::mbar_wait_bounded(empty0 + 8 * s, phase, p.wait_limit)) {
        atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
        return;
      }
      issue_w(w, s);
      issue_x(w, s);
      w.next();
      if (++s == S) {
        s = 0;
        phase ^= 1;
      }
    }
    return;
  }

  if (warp == kConsumerWarps + 1) {
    // ------------------------------------------------- row sums of the activation slices
    cluster_ready();
    ptx::pdl_wait();
    int s = 0, phase = 0;
    // the constant operand of the row-sum products: even columns all ones, odd columns minus the
    // offset of the k's class
    const int gid = lane >> 2;
    const __half2 neg_lo = __float2half2_rn(-kOffLo), neg_hi = __float2half2_rn(-kOffHi);
    const uint32_t b_first = (gid & 1) ? *reinterpret_cast<const uint32_t*>(&neg_lo) : 0x3C003C00u;
    const uint32_t b_last = (gid & 1) ? *reinterpret_cast<const uint32_t*>(&neg_hi) : 0x3C003C00u;
    const uint32_t ring_h = ptx::smem_u32(ring);
    [[maybe_unused]] int rms_last = -1;  // chain: the step whose row factors were formed last
    for (StageWalk<PT> w = make_walk(); !w.done(); w.next()) {
      if (!ptx::mbar_wait_bounded(xbar0 + 8 * s, phase, p.wait_limit)) {
        if (lane == 0) atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
        return;
      }
      const uint32_t st = ring_h + s * p.stage_bytes;
      float* xsum = reinterpret_cast<float*>(ring + (size_t)s * p.stage_bytes + p.xsum_offset);
      if constexpr (G == kGroup) {  // smaller groups need no sums
        const uint32_t x_rows = st + kXOffset;
        const int groups = w.groups();
        if constexpr (MT == 2) {
          stage_row_sums<16>(x_rows, xsum, M, groups, lane, b_first, b_last);
        } else if (M <= 2) {
          stage_row_sums<2>(x_rows, xsum, M, groups, lane, b_first, b_last);
        } else if (M <= 4) {
          stage_row_sums<4>(x_rows, xsum, M, groups, lane, b_first, b_last);
        } else {
          stage_row_sums<8>(x_rows, xsum, M, groups, lane, b_first, b_last);
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(full0 + 8 * s);
      if (++s == S) {
        s = 0;
        phase ^= 1;
      }
      if constexpr (CHAIN) {
        // The first stage of a step with a folded rms-norm: the row factor rsqrt(mean x^2 + eps) of
        // every token, from the whole activation row in global memory (L2: the row may have been
        // written by other SMs a moment ago).  The consumers need it only when a panel ends, so it
        // is formed after the stage has been handed over.
        if (w.j != rms_last) {
          rms_last = w.j;
          const ChainProb& q = p.prob[w.j];
          if (q.rms_eps >= 0.0f) {
            (void)ptx::ld_acquire_gpu(p.sync);  // the row is final: the phase's activations were requested already
            const int slot = w.j & (kChainRmsSlots - 1);
            for (int m = 0; m < M; ++m) {
              const uint4* row = reinterpret_cast<const uint4*>(q.x + (size_t)m * q.K);
              float ss = 0.0f;
              const int vecs = q.K / 8;  // a multiple of 16
              for (int i0 = 0; i0 < vecs; i0 += 8 * 32) {
                uint4 v[8];  // eight loads in flight per lane: the row costs one or two round trips to L2
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  const int i = i0 + u * 32 + lane;
                  v[u] = i < vecs ? __ldcg(row + i) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&v[u].x));
                  const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&v[u].y));
                  const float2 f2 = __half22float2(*reinterpret_cast<const __half2*>(&v[u].z));
                  const float2 f3 = __half22float2(*reinterpret_cast<const __half2*>(&v[u].w));
                  ss += (f0.x * f0.x + f0.y * f0.y) + (f1.x * f1.x + f1.y * f1.y) + (f2.x * f2.x + f2.y * f2.y) +
                        (f3.x * f3.x + f3.y * f3.y);
                }
              }
#pragma unroll
              for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, off);
              if (lane == 0) rms_val[slot * 8 + m] = rsqrtf(ss / (float)q.K + q.rms_eps);
            }
            __syncwarp();
            if (lane == 0) {
              __threadfence_block();
              rms_step[slot] = w.j;
            }
          }
        }
      }
    }
    return;
  }

  // ---------------------------------------------------------------------- consumers
  cluster_ready();
  ptx::pdl_wait();
  const int gid = lane >> 2;  // fragment row (column of W) / token of the B fragment
  const int t = lane & 3;     // which 32-wide k slice of the group this lane owns

  float acc[MT][4];
  float acc1[G == kGroup ? 1 : MT][4];  // smaller groups: the second accumulator chain of the panel
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[mt][j] = 0.0f;
#pragma unroll
  for (int mt = 0; mt < (G == kGroup ? 1 : MT); ++mt)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc1[mt][j] = 0.0f;
  const uint32_t mask_lo = reg_const(kMaskLo), exp_lo = reg_const(kExpLo);
  const uint32_t mask_hi = reg_const(kMaskHi), exp_hi = reg_const(kExpHi);
  // Byte offsets of this lane's activation fragments and row sums inside a stage.  Lanes whose
  // token does not exist read a block of zeros instead (one address select per tile).
  int x_off[MT];
  bool has_row[MT];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int m = 8 * mt + gid;
    has_row[mt] = m < M;
    x_off[mt] = kXOffset + m * kXRowBytes + t * 64;
  }
  const int xs_off = p.xsum_offset + t * 16;
  const bool rot = ROT && t >= 2;
  int chunk_off[4];  // byte offset of the chunk this lane takes in MMA step v
#pragma unroll
  for (int v = 0; v < 4; ++v) chunk_off[v] = ((v + (rot ? 1 : 0)) & 3) * 16;
  const uint32_t ring_u32 = ptx::smem_u32(ring);

  [[maybe_unused]] auto addend = [&](const auto& q, int m, size_t n) -> float {
    if constexpr (CHAIN) return __half2float(__ldcg(q.add + (size_t)m * q.add_stride + n));  // L2: other SMs wrote it
    else return __half2float(p.add[(size_t)m * p.add_stride + n]);
  };
  [[maybe_unused]] float add_pre[MT][4];  // addend of the outputs this lane emits at the end of the current panel
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int j = 0; j < 4; ++j) add_pre[mt][j] = 0.0f;
  StageWalk<PT> w = make_walk();
  [[maybe_unused]] uint32_t red_phase = 0;  // cluster launches: parity of the next exchange
  int g_begin = w.g;
  int s = 0, phase = 0;
  while (!w.done()) {
    const auto& q = p.prob[w.j];
    const int rest = q.nbs - kPanelTiles * w.panel;
    const int R = rest < kPanelTiles ? rest : kPanelTiles;
    const int groups = w.groups();
    if (!ptx::mbar_wait_bounded(full0 + 8 * s, phase, p.wait_limit)) {
      if (lane == 0) atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
      return;  // every wait in this kernel is bounded, so the other warps leave as well
    }
    // The stage that ends the panel (or the range): the addend of the outputs this lane will emit
    // is requested now, so that its trip to L2 runs under the stage's products instead of after them.
    if constexpr (CHAIN || EPI == 1) {
      const bool ends = (w.g + groups == w.ng) || (w.left - groups <= 0);
      int epi_now = EPI;
      if constexpr (CHAIN) epi_now = q.epi;
      if (ends && epi_now == 1) {
        int tile = warp;         // the tile whose outputs this warp stores
        bool mine = warp < R;
        if constexpr (PT::kCluster) {
          const bool whole = g_begin == 0 && w.g + groups == w.ng;
          int unit;
          if constexpr (CHAIN) unit = p.phase[w.ph].unit; else unit = p.unit;
          if (!whole && unit < 0 && p.cluster > 1) {  // shared inside a cluster: see the exchange below
            const int s_grp = -unit, s_log = 31 - __clz(s_grp);
            tile = warp * s_grp + (int)(blockIdx.x & (unsigned)(s_grp - 1));
            mine = warp < (kPanelTiles >> s_log) && tile < R;
          }
        }
        if (mine) {
          const size_t n0 = (size_t)(w.panel * kPanelTiles + tile) * kTileN + gid;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int m = 8 * mt + 2 * t + (j & 1);
              if (m < M) add_pre[mt][j] = addend(q, m, n0 + (j >> 1) * 8);
            }
        }
      }
    }
    if (warp < R) {
      const uint32_t st = ring_u32 + s * p.stage_bytes;
      const uint32_t wt_base = st + warp * kTileBytes + lane * 16;
      // smaller groups: the lane's 32-wide k slice t lies in group t (G = 32) or t / 2 (G = 64) of the tile row
      const uint32_t sc_base =
          st + kScaleOffset + warp * kTileScaleBytes + (G == kGroup ? 0 : (G == 32 ? t : t >> 1)) * 64 + gid * 4;
#pragma unroll
      for (int gg = 0; gg < kStageGroups; ++gg) {
        if constexpr (G != kGroup) {
          if (gg < groups) {
            const uint4 wlo = ptx::lds128(wt_base + gg * R * kTileBytes);        // column gid
            const uint4 whi = ptx::lds128(wt_base + gg * R * kTileBytes + 512);  // column gid + 8
            const uint32_t s_lo = ptx::lds32(sc_base + gg * R * kTileScaleBytes);
            const uint32_t s_hi = ptx::lds32(sc_base + gg * R * kTileScaleBytes + 32);
            const __half2 off_lo = __float2half2_rn(kOffLo), off_hi = __float2half2_rn(kOffHi);
            const __half2 db_lo = *reinterpret_cast<const __half2*>(&s_lo);  // {d, b} of column gid
            const __half2 db_hi = *reinterpret_cast<const __half2*>(&s_hi);  // {d, b} of column gid + 8
            const __half2 dl = __low2half2(db_lo), dh = __low2half2(db_hi);
            // the bias seen from the two binades of the construction (exact sums)
            const __half2 bl_a = __hadd2(__high2half2(db_lo), off_lo), bl_b = __hadd2(__high2half2(db_lo), off_hi);
            const __half2 bh_a = __hadd2(__high2half2(db_hi), off_lo), bh_b = __hadd2(__high2half2(db_hi), off_hi);
            uint4 xv[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              const uint32_t xp = has_row[mt] ? st + x_off[mt] + gg * 256 : zero_block;
#pragma unroll
              for (int v = 0; v < 4; ++v) xv[mt][v] = ptx::lds128(xp + chunk_off[v]);
            }
            const uint32_t wl[4] = {rot ? wlo.y : wlo.x, rot ? wlo.z : wlo.y, rot ? wlo.w : wlo.z, rot ? wlo.x : wlo.w};
            const uint32_t wh[4] = {rot ? whi.y : whi.x, rot ? whi.z : whi.y, rot ? whi.w : whi.z, rot ? whi.x : whi.w};
            auto deq = [](uint32_t e, __half2 b, __half2 d) {
              const __half2 r = __hmul2(__hsub2(*reinterpret_cast<const __half2*>(&e), b), d);
              return *reinterpret_cast<const uint32_t*>(&r);
            };
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              const uint32_t wl2 = wl[v] >> 8, wh2 = wh[v] >> 8;
              const uint32_t l01 = deq(and_or(wl[v], mask_lo, exp_lo), bl_a, dl), l23 = deq(and_or(wl[v], mask_hi, exp_hi), bl_b, dl);
              const uint32_t l45 = deq(and_or(wl2, mask_lo, exp_lo), bl_a, dl), l67 = deq(and_or(wl2, mask_hi, exp_hi), bl_b, dl);
              const uint32_t h01 = deq(and_or(wh[v], mask_lo, exp_lo), bh_a, dh), h23 = deq(and_or(wh[v], mask_hi, exp_hi), bh_b, dh);
              const uint32_t h45 = deq(and_or(wh2, mask_lo, exp_lo), bh_a, dh), h67 = deq(and_or(wh2, mask_hi, exp_hi), bh_b, dh);
#pragma unroll
              for (int mt = 0; mt < MT; ++mt) {
                mma16816(acc[mt], l01, h01, l23, h23, xv[mt][v].x, xv[mt][v].y);
                mma16816(acc1[mt], l45, h45, l67, h67, xv[mt][v].z, xv[mt][v].w);
              }
            }
          }
          continue;
        }
        if (gg < groups) {
          const uint4 wlo = ptx::lds128(wt_base + gg * R * kTileBytes);        // column gid
          const uint4 whi = ptx::lds128(wt_base + gg * R * kTileBytes + 512);  // column gid + 8
          const uint32_t s_lo = ptx::lds32(sc_base + gg * R * kTileScaleBytes);
          const uint32_t s_hi = ptx::lds32(sc_base + gg * R * kTileScaleBytes + 32);

          uint4 xv[MT][4];
          float4 xs[MT];  // {sum, -offsets} of token 2t, {sum, -offsets} of token 2t+1
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const uint32_t xp = has_row[mt] ? st + x_off[mt] + gg * 256 : zero_block;
#pragma unroll
            for (int v = 0; v < 4; ++v) xv[mt][v] = ptx::lds128(xp + chunk_off[v]);
            xs[mt] = ptx::lds128f(st + xs_off + gg * 128 + mt * 64);
          }

          // two independent accumulator chains keep the tensor pipe busy; the first one starts
          // from minus the constant offsets, the second from zero
          float c[MT][2][4];
          // packed word v holds the codes of chunk v of the lane's k slice
          const uint32_t wl[4] = {rot ? wlo.y : wlo.x, rot ? wlo.z : wlo.y, rot ? wlo.w : wlo.z, rot ? wlo.x : wlo.w};
          const uint32_t wh[4] = {rot ? whi.y : whi.x, rot ? whi.z : whi.y, rot ? whi.w : whi.z, rot ? whi.x : whi.w};
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            // k 0,1 / 2,3 of the word straight from the low byte of each half; k 4,5 / 6,7 after
            // one shift by a byte
            const uint32_t wl2 = wl[v] >> 8, wh2 = wh[v] >> 8;
            const uint32_t l01 = and_or(wl[v], mask_lo, exp_lo), l23 = and_or(wl[v], mask_hi, exp_hi);
            const uint32_t l45 = and_or(wl2, mask_lo, exp_lo), l67 = and_or(wl2, mask_hi, exp_hi);
            const uint32_t h01 = and_or(wh[v], mask_lo, exp_lo), h23 = and_or(wh[v], mask_hi, exp_hi);
            const uint32_t h45 = and_or(wh2, mask_lo, exp_lo), h67 = and_or(wh2, mask_hi, exp_hi);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              if (v == 0) {
                mma16816_init(c[mt][0], l01, h01, l23, h23, xv[mt][v].x, xv[mt][v].y, xs[mt].y, xs[mt].w);
              } else {
                mma16816(c[mt][0], l01, h01, l23, h23, xv[mt][v].x, xv[mt][v].y);
              }
              mma16816(c[mt][0], l45, h45, l67, h67, xv[mt][v].z, xv[mt][v].w);
            }
          }

          const float2 db_lo = __half22float2(*reinterpret_cast<const __half2*>(&s_lo));  // {d, b}
          const float2 db_hi = __half22float2(*reinterpret_cast<const __half2*>(&s_hi));
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const float t0 = fmaf(-db_lo.y, xs[mt].x, c[mt][0][0]);
            const float t1 = fmaf(-db_lo.y, xs[mt].z, c[mt][0][1]);
            const float t2 = fmaf(-db_hi.y, xs[mt].x, c[mt][0][2]);
            const float t3 = fmaf(-db_hi.y, xs[mt].z, c[mt][0][3]);
            acc[mt][0] = fmaf(db_lo.x, t0, acc[mt][0]);
            acc[mt][1] = fmaf(db_lo.x, t1, acc[mt][1]);
            acc[mt][2] = fmaf(db_hi.x, t2, acc[mt][2]);
            acc[mt][3] = fmaf(db_hi.x, t3, acc[mt][3]);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(empty0 + 8 * s);
    if (++s == S) {
      s = 0;
      phase ^= 1;
    }
    const int panel = w.panel;
    const int ng = w.ng;
    const int g_end = w.g + groups;
    const bool range_ends = w.left - groups <= 0;  // of this phase, for a chain
    const int jq = w.j, ph = w.ph;

    if (g_end == ng || range_ends) {
      // ---- the panel ends here (or the range does): emit the 16 columns this warp owns
      const int covered = g_end - g_begin;
      if constexpr (G != kGroup) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            acc[mt][j] += acc1[mt][j];
            acc1[mt][j] = 0.0f;
          }
      }
      // What follows the sums: fixed per instantiation for a list, a property of the step in a chain.
      int epi = EPI;
      float r_even = 1.0f, r_odd = 1.0f;  // chain: row factors of tokens 2t and 2t + 1 (a folded rms-norm)
      if constexpr (CHAIN) {
        epi = q.epi;
        if (q.rms_eps >= 0.0f) {
          const int slot = jq & (kChainRmsSlots - 1);
          const long long t0 = clock64();
          while (rms_step[slot] != jq) {
            if (clock64() - t0 > p.wait_limit) {
              if (lane == 0) atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
              return;
            }
          }
          __threadfence_block();
          r_even = rms_val[slot * 8 + 2 * t];
          r_odd = rms_val[slot * 8 + 2 * t + 1];
        }
      }
      // one finished output (and, for SwiGLU, its partner 8 columns on): the epilogue and the store
      auto emit = [&](int m, size_t n, float v, float v_up, int j, int mt) {
        if (CHAIN) {
          const float r = (j & 1) ? r_odd : r_even;
          v *= r;
          v_up *= r;
        }
        if (epi == 2) {
          // columns gid (gate) and gid + 8 (up) of the tile sit in the same lane: the tile's eight
          // outputs silu(gate) * up go to columns 8 * tile + gid of y[M, N / 2]
          if (j < 2) q.y[(size_t)m * (q.N >> 1) + (n - gid) / 2 + gid] = __float2half_rn(swiglu(v, v_up));
        } else {
          if (epi == 1) v += add_pre[mt][j];
          q.y[(size_t)m * q.N + n] = __float2half_rn(v);
        }
      };
      int final_share = 0;  // chain: eighths of the panel that this CTA made final (8 = the whole panel)
      const size_t n_lo = (size_t)(panel * kPanelTiles + warp) * kTileN + gid;
      if (covered == ng) {
        if (warp < R) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int m = 8 * mt + 2 * t + (j & 1);
              if (m < M) emit(m, n_lo + (j >> 1) * 8, acc[mt][j], acc[mt][(j + 2) & 3], j, mt);
            }
          }
        }
        final_share = kPanelTiles;
      } else {
        // the panel is shared with neighbouring CTAs: its scratch slot is named after the first
        // range boundary that falls inside the panel (after the panel itself when every panel
        // has its own CTAs)
        int unit = 0, total = 0;
        if constexpr (CHAIN) {
          unit = p.phase[ph].unit;
          total = p.phase[ph].chunks;
        } else {
          unit = p.unit;
          total = p.total_chunks;
        }
        bool exchanged = false;
        if constexpr (PT::kCluster) {
          if (unit < 0 && p.cluster > 1) {
            // ---- the s CTAs that share this panel are neighbours in a cluster: exchange through shared memory
            exchanged = true;
            const int s_grp = -unit;                                           // 2, 4 or 8
            const int s_log = 31 - __clz(s_grp);
            const int my_i = (int)(blockIdx.x & (unsigned)(s_grp - 1));         // slice of the panel = rank in the group
            const uint32_t base = ptx::cluster_ctarank() - (uint32_t)my_i;     // cluster rank of the group's first CTA
            const uint32_t dst = base + (uint32_t)(warp & (s_grp - 1));        // who finishes this warp's tile
            const int per = kPanelTiles >> s_log;                              // tiles every CTA finishes
            // The receiver announces what it expects: s contributions of 16 columns x M tokens for each
            // of its tiles that exist (the byte count may be reported before or after it is announced).
            if (tid == 0) {
              int mine_tiles = 0;
              for (int u = 0; u < per; ++u) mine_tiles += (u * s_grp + my_i < R) ? 1 : 0;
              ptx::mbar_arrive_expect_tx(red_bar, (uint32_t)(mine_tiles * s_grp * kTileN * M * 4));
            }
            if (warp < R) {
              constexpr int kRedPad = 8 * MT;
              const uint32_t to = ptx::mapa(red_buf + (uint32_t)((my_i * per + (warp >> s_log)) * kTileN * kRedPad * 4), dst);
              const uint32_t to_bar = ptx::mapa(red_bar, dst);
#pragma unroll
              for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int m = 8 * mt + 2 * t + (j & 1);
                  if (m < M)
                    ptx::st_async_cluster_f32(to + (uint32_t)(((gid + (j >> 1) * 8) * kRedPad + m) * 4), acc[mt][j], to_bar);
                }
              }
            }
            // every contribution has landed once the phase completes
            if (!ptx::mbar_wait_bounded_cluster(red_bar, red_phase, p.wait_limit)) {
              if (lane == 0) atomicExch(p.status, (unsigned)TL_ERR_TIMEOUT);
              return;
            }
            red_phase ^= 1;
            const int tile = warp * s_grp + my_i;  // the tile this warp finishes, if it has one
            if (warp < per && tile < R) {
              const size_t n_out = (size_t)(panel * kPanelTiles + tile) * kTileN + gid;
              // the s contributions to this lane's four sums: all loads first, then the additions
              const uint32_t mine = red_buf + (uint32_t)(((warp * kTileN + gid) * (8 * MT) + 2 * t) * 4);
              const uint32_t src_stride = (uint32_t)(per * kTileN * 8 * MT * 4);
#pragma unroll
              for (int mt = 0; mt < MT; ++mt) {
                float2 part[kPanelTiles][2];  // [sender][column gid, column gid + 8]: tokens 2t and 2t + 1
#pragma unroll
                for (int src = 0; src < kPanelTiles; ++src) {
                  part[src][0] = part[src][1] = make_float2(0.0f, 0.0f);
                  if (src < s_grp) {
                    part[src][0] = ptx::lds64f(mine + src * src_stride + mt * 32);
                    part[src][1] = ptx::lds64f(mine + src * src_stride + mt * 32 + 8 * (8 * MT) * 4);
                  }
                }
                float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int src = 0; src < kPanelTiles; ++src) {
                  v[0] += part[src][0].x;
                  v[1] += part[src][0].y;
                  v[2] += part[src][1].x;
                  v[3] += part[src][1].y;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int m = 8 * mt + 2 * t + (j & 1);
                  if (m < M) emit(m, n_out + (j >> 1) * 8, v[j], v[(j + 2) & 3], j, mt);
                }
              }
            }
            final_share = per;
          }
        }
        int k = panel;
        if (exchanged) {
          // done above
        } else {
        if (unit > 0) {
          const long long ps = (long long)q.chunk_begin + (long long)panel * ng;
          k = (int)(ps * gridDim.x / total);
          while ((long long)total * k / gridDim.x <= ps) ++k;
        }
        float* slot = reinterpret_cast<float*>(p.ws + (size_t)k * kSlotBytes);
        unsigned int* cnt = reinterpret_cast<unsigned int*>(slot + kSlotFloats);
        const int c_lo = (warp * kTileN + gid) * kWsPad;
        if (warp < R) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int m = 8 * mt + 2 * t + (j & 1);
              if (m < M) atomicAdd(slot + c_lo + (j >> 1) * 8 * kWsPad + m, acc[mt][j]);
            }
          }
        }
        __threadfence();
        ptx::named_bar_sync(1, kConsumerThreads);
        if (tid == 0) {
          const unsigned prev = atomicAdd(cnt, (unsigned)covered);
          flags[0] = (prev + (unsigned)covered == (unsigned)ng) ? 1 : 0;
        }
        ptx::named_bar_sync(1, kConsumerThreads);
        if (flags[0]) {
          __threadfence();
          if (warp < R) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int m = 8 * mt + 2 * t + (j & 1);
                if (m < M) {
                  float* a = slot + c_lo + (j >> 1) * 8 * kWsPad + m;
                  // SwiGLU: the up half (j >= 2) is read by the iteration of its gate and cleared by its own
                  const float v = __ldcg(a);
                  const float v_up = (epi == 2 && j < 2) ? __ldcg(a + 8 * kWsPad) : 0.0f;
                  emit(m, n_lo + (j >> 1) * 8, v, v_up, j, mt);
                  __stcg(a, 0.0f);
                }
              }
            }
          }
          if (tid == 0) *cnt = 0;
          final_share = kPanelTiles;
        }
        }  // !exchanged
      }
      if constexpr (CHAIN) {
        // A panel that is final counts towards the next phase's target.  The barrier orders every
        // consumer's stores (outputs, cleared slot) before thread 0, whose addition to the counter
        // has release semantics at GPU scope, which is cumulative over what the barrier ordered.
        if (final_share > 0) {
          ptx::named_bar_sync(1, kConsumerThreads);
          if (tid == 0) ptx::red_release_gpu(p.sync, (unsigned)final_share);
        }
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[mt][j] = 0.0f;
      g_begin = (g_end == ng) ? 0 : g_end;
    }
    // (a chain's walk may have to find the CTA's range of the next phase here: after the panel has
    // been published, not before)
    w.next();
    if constexpr (CHAIN) {
      if (range_ends && !w.done()) g_begin = w.g;  // the range of the next phase may start mid-panel
    }
  }
  if constexpr (CHAIN) {
    // The last CTA to finish leaves the two counters zero for the next launch.  The fence orders this
    // CTA's additions to the panel counter before its arrival here.
    if (tid == 0) {
      __threadfence();
      const unsigned prev = atomicAdd(p.sync + 1, 1u);
      if (prev == gridDim.x - 1) {
        __threadfence();
        p.sync[0] = 0u;
        p.sync[1] = 0u;
      }
    }
  }
}

// ----------------------------------------------------------------------------- host side
__device__ unsigned int g_decode_status = 0;

unsigned int* device_status_word() {
  static unsigned int* cached[64] = {nullptr};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
  unsigned int* ptr = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_decode_status) != cudaSuccess) return nullptr;
  if (dev >= 0 && dev < 64) cached[dev] = ptr;
  return ptr;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
  int n = 0;
  cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  if (n <= 0) n = 148;
  if (dev >= 0 && dev < 64) cached[dev] = n;
  return n;
}

constexpr int kRingBudget = 110 * 1024;

template <int MT, int NB, bool ROT, int EPI, int G>
cudaError_t launch_one(const DecodeParams<NB>& p, int grid, size_t smem, cudaStream_t stream) {
  if (p.cluster > 1) smem += smem_tail_cluster(MT) - kSmemTail;  // the exchange buffer of a cluster launch
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_decode_kernel<MT, DecodeParams<NB>, ROT, EPI, G>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         // groups of 32 with more than 11 tokens need 117 KB for two stages;
                                         // cluster launches add their exchange buffer
                                         (G == kGroup ? 116 : 126) * 1024);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.cluster > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)p.cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, gemv_decode_kernel<MT, DecodeParams<NB>, ROT, EPI, G>, p);
}

// How many clusters of `size` CTAs of the lone-problem kernel can be resident at once (0 if the
// question cannot be answered).  All instantiations have the same block size and, for a given
// shared-memory size, the same footprint, so one of them answers for all; cached per device.
int lone_max_clusters(int size, size_t smem) {
  static std::atomic<int> cache[64][4];
  int dev = 0;
  cudaGetDevice(&dev);
  const int slot = size == 8 ? 3 : (size == 4 ? 2 : 1);
  if (dev >= 0 && dev < 64) {
    const int c = cache[dev][slot].load(std::memory_order_relaxed);
    if (c != 0) return c > 0 ? c : 0;
  }
  auto kernel = gemv_decode_kernel<1, DecodeParams<1>, false, 0, kGroup>;
  int clusters = 0;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 116 * 1024) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(size * 64));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess) clusters = 0;
  }
  (void)cudaGetLastError();
  if (dev >= 0 && dev < 64) cache[dev][slot].store(clusters > 0 ? clusters : -1, std::memory_order_relaxed);
  return clusters;
}

template <int NB, int G = kGroup>
cudaError_t launch_batch(const DecodeProblem* probs, int count, int M, void* workspace,
                         cudaStream_t stream) {
  const int64_t split_mode = tune(kTuneDecodeSplit);   // 1 = whole panels, 2 = stream-K ranges (tl_e0m4_tuning_set)
  const int64_t forced_slices = tune(kTuneDecodeSlices);
  const int sms = sm_count();
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  DecodeParams<NB> p;
  p.ws = static_cast<uint8_t*>(workspace);
  p.status = status;
  p.M = M;
  p.count = count;
  p.add = count == 1 ? probs[0].add : nullptr;
  p.add_stride = count == 1 && probs[0].add_stride >= 0 ? probs[0].add_stride : probs[0].N;
  p.wait_limit = wait_limit_cycles();
  p.skip_copies = tune(kTuneSkipCopies) == 1;
  p.cluster = 1;
  long long total = 0;
  for (int j = 0; j < count; ++j) {
    Prob& q = p.prob[j];
    q.x = probs[j].x;
    q.packed = reinterpret_cast<const uint8_t*>(probs[j].packed);
    q.scales = reinterpret_cast<const uint8_t*>(probs[j].scales);
    q.y = probs[j].y;
    q.K = (int)probs[j].K;
    q.N = (int)probs[j].N;
    q.ng = (int)(probs[j].K / kGroup);
    q.nbs = (int)(probs[j].N / kTileN);
    q.panels = (q.nbs + kPanelTiles - 1) / kPanelTiles;
    q.chunk_begin = (int)total;
    total += (long long)q.panels * q.ng;
    if (total > 0x7FFFFFFFLL / 512) return cudaErrorInvalidValue;
  }
  p.total_chunks = (int)total;

  // grid: one CTA per SM, fewer when there is less than one chunk per SM
  const int per_sm = tune(kTuneDecodeCtasPerSm) == 1 ? 1 : 2;
  int grid = p.total_chunks < per_sm * sms ? p.total_chunks : per_sm * sms;
  if (grid > kMaxSlots - 1) grid = kMaxSlots - 1;
  p.unit = 1;
  if (count == 1) {
    // a lone problem is split on panel boundaries when that keeps the SMs evenly loaded
    const int panels = p.prob[0].panels;
    const int per = (panels + grid - 1) / grid;
    bool aligned = panels >= grid && (double)panels / ((double)per * grid) >= 0.97;
    if (split_mode == 1) {
      aligned = true;
      if (panels < grid) grid = panels;
    }
    if (split_mode == 2) aligned = false;
    if (aligned) p.unit = p.prob[0].ng;
    // With fewer panels than CTAs every panel gets its own s CTAs, each taking one slice of the
    // panel's groups: a CTA then flushes one partial tile instead of the two of a range that
    // straddles a panel boundary, and with s = 1 none at all.  Measured at M = 1, 4, 8 on
    // fourteen layer shapes, slices are up to 1.4x faster than the stream-K ranges.
    // The CTAs of a panel meet either in the global scratch (any s) or, launched as a cluster of s = 2,
    // 4 or 8 neighbours, in one another's shared memory, which costs a fraction of the round trips
    // (only where all clusters can be resident at once: a second wave would cost more than the
    // exchange saves).  The choice minimises a small model fitted to per-launch times of sixteen
    // layer shapes: ring stages a CTA walks (about 1 us each at this size) + 2.3 us for meeting in
    // the scratch or 0.8 us for meeting in a cluster.
    int slices = 0;
    bool cluster = false;
    const int ng0 = p.prob[0].ng;
    auto stages_of = [&](int s) { return (((ng0 + s - 1) / s) + kStageGroups - 1) / kStageGroups; };
    if (panels < grid && split_mode < 0 && forced_slices < 0) {
      int nat = grid / panels < ng0 ? grid / panels : ng0;  // the most slices the grid allows
      if (nat == 2 && ng0 <= 16) nat = 1;
      slices = nat;
      double best = stages_of(nat) + (nat > 1 ? 2.3 : 0.0);
      if (nat > 1 && stages_of(1) <= best) {
        slices = 1;
        best = stages_of(1);
      }
      if (NB == 1 && tune(kTuneDecodeCluster) != 0) {
        for (int c = 8; c >= 2; c >>= 1) {
          if (c > ng0 || (long long)panels * c > grid) continue;
          // (asked for the largest shared-memory size a cluster launch uses: three stages at one token)
          if (panels > lone_max_clusters(c, 128 + 3 * 36480 + smem_tail_cluster(1))) continue;
          const double cost = stages_of(c) + 0.8;
          if (cost < best || (tune(kTuneDecodeCluster) == 1 && !cluster)) {
            best = cost;
            slices = c;
            cluster = true;
          }
        }
      }
    }
    if (forced_slices > 0 && split_mode < 0) {
      slices = (int)forced_slices;
      cluster = NB == 1 && tune(kTuneDecodeCluster) != 0 && (slices == 2 || slices == 4 || slices == 8) &&
                panels <= lone_max_clusters(slices, 128 + 3 * 36480 + smem_tail_cluster(1));
    }
    if (slices > 0 && slices <= ng0 && (long long)panels * slices <= grid) {
      if (cluster) p.cluster = slices;
      p.unit = -slices;
      grid = panels * slices;
    }
  }

  const int mt = M <= 8 ? 1 : 2;
  p.xsum_offset = x_offset(G) + M * kXRowBytes;
  p.stage_bytes = (p.xsum_offset + kStageGroups * 32 * (int)sizeof(float) + 127) & ~127;
  // (a cluster launch gives the room of its exchange buffer back, so that two CTAs still fit an SM)
  int stages = (kRingBudget - (p.cluster > 1 ? smem_tail_cluster(mt) - kSmemTail : 0)) / p.stage_bytes;
  stages = stages > kMaxStages ? kMaxStages : (stages < 2 ? 2 : stages);
  p.stages = stages;
  const size_t smem = 128 + (size_t)stages * p.stage_bytes + 3 * kMaxStages * sizeof(uint64_t) + 16 + 64;
  // measured crossover: below five tokens the selects cost more than the conflicts they avoid; a
  // list (bound by its consumers' issue slots, not by latency) gains only from seven tokens on
  const int rot_min = tune(kTuneDecodeRotMin) >= 0 ? (int)tune(kTuneDecodeRotMin) : (NB == 1 ? 5 : 7);
  cudaError_t e;
  if constexpr (NB == 1) {
    if (p.add) {
      e = mt == 2        ? launch_one<2, NB, true, 1, G>(p, grid, smem, stream)
        : M >= rot_min ? launch_one<1, NB, true, 1, G>(p, grid, smem, stream)
                       : launch_one<1, NB, false, 1, G>(p, grid, smem, stream);
      count_launch();
      return e;
    }
    if (probs[0].swiglu) {
      e = mt == 2        ? launch_one<2, NB, true, 2, G>(p, grid, smem, stream)
        : M >= rot_min ? launch_one<1, NB, true, 2, G>(p, grid, smem, stream)
                       : launch_one<1, NB, false, 2, G>(p, grid, smem, stream);
      count_launch();
      return e;
    }
  }
  e = mt == 2        ? launch_one<2, NB, true, 0, G>(p, grid, smem, stream)
    : M >= rot_min ? launch_one<1, NB, true, 0, G>(p, grid, smem, stream)
                   : launch_one<1, NB, false, 0, G>(p, grid, smem, stream);
  count_launch();
  return e;
}

}  // namespace

unsigned int* device_status_ptr() { return device_status_word(); }

size_t decode_workspace_bytes() { return (size_t)kMaxSlots * kSlotBytes; }

namespace {

template <int NB>
cudaError_t launch_batch_group(const DecodeProblem* probs, int count, int M, void* workspace, cudaStream_t stream,
                               int group) {
  if (group == 32) return launch_batch<NB, 32>(probs, count, M, workspace, stream);
  if (group == 64) return launch_batch<NB, 64>(probs, count, M, workspace, stream);
  return launch_batch<NB, kGroup>(probs, count, M, workspace, stream);
}

}  // namespace

cudaError_t launch_gemv_decode_batch(const DecodeProblem* probs, int count, int M, void* workspace,
                                     cudaStream_t stream, int group) {
  for (int j0 = 0; j0 < count; j0 += kMaxDecodeBatch) {
    const int n = count - j0 < kMaxDecodeBatch ? count - j0 : kMaxDecodeBatch;
    const cudaError_t e = n == 1 ? launch_batch_group<1>(probs + j0, 1, M, workspace, stream, group)
                                 : launch_batch_group<kMaxDecodeBatch>(probs + j0, n, M, workspace, stream, group);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t launch_gemv_decode(const __half* x, const uint32_t* packed, const uint32_t* scales,
                               __half* y, int64_t M, int64_t K, int64_t N, void* workspace,
                               cudaStream_t stream, const __half* add, bool swiglu, int group, int64_t add_stride) {
  for (int64_t m0 = 0; m0 < M; m0 += 16) {
    const int Mc = (int)((M - m0) < 16 ? (M - m0) : 16);
    const int64_t stride = add_stride >= 0 ? add_stride : N;
    DecodeProblem q{x + m0 * K, packed, scales, y + m0 * (swiglu ? N / 2 : N), K, N, add ? add + m0 * stride : nullptr, swiglu, stride};
    const cudaError_t e = launch_batch_group<1>(&q, 1, Mc, workspace, stream, group);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------- a chain of dependent steps
namespace {

template <bool ROT, int G>
cudaError_t chain_kernel_setup(int* blocks_per_sm, size_t smem) {
  auto kernel = gemv_decode_kernel<1, ChainParams, ROT, 0, G>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 126 * 1024);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, kernel, kThreads, smem);
}

// How many clusters of `size` CTAs can be resident at once.
template <bool ROT, int G>
cudaError_t chain_max_clusters(int* clusters, size_t smem, int size) {
  int unused = 0;
  cudaError_t e = chain_kernel_setup<ROT, G>(&unused, smem);  // sets the shared-memory attribute
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(size * 64));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)size;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(clusters, gemv_decode_kernel<1, ChainParams, ROT, 0, G>, &cfg);
}

template <bool ROT, int G>
cudaError_t chain_kernel_launch(const ChainParams& p, int grid, size_t smem, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.cluster > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)p.cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, gemv_decode_kernel<1, ChainParams, ROT, 0, G>, p);
}

// One launch of at most kMaxChain steps.  Every CTA of the grid takes part in every phase, and a
// phase waits for CTAs of the one before, so the whole grid has to be resident at once: the grid is
// what the occupancy calculation says fits (two CTAs per SM).
template <int G>
cudaError_t launch_chain(const ChainStep* steps, int count, int M, void* workspace, cudaStream_t stream) {
  const int sms = sm_count();
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  static ChainParams p;  // 14 KB: too large for the stack of a small thread; guarded by the mutex below
  static std::mutex lock;
  std::lock_guard<std::mutex> guard(lock);
  p.ws = static_cast<uint8_t*>(workspace);
  p.status = status;
  p.sync = reinterpret_cast<unsigned int*>(p.ws + (size_t)kMaxSlots * kSlotBytes);
  p.M = M;
  p.count = count;
  p.wait_limit = wait_limit_cycles();
  p.skip_copies = tune(kTuneSkipCopies) == 1;
  p.xsum_offset = x_offset(G) + M * kXRowBytes;
  p.stage_bytes = (p.xsum_offset + kStageGroups * 32 * (int)sizeof(float) + 127) & ~127;
  int stages = (kRingBudget - (smem_tail_cluster(1) - kSmemTail)) / p.stage_bytes;
  stages = stages > kMaxStages ? kMaxStages : (stages < 2 ? 2 : stages);
  p.stages = stages;
  const size_t smem = 128 + (size_t)stages * p.stage_bytes + smem_tail_cluster(1);
  const bool rot = M >= 5;
  // Clusters of eight neighbouring CTAs, so that the CTAs that share a panel can add their sums up
  // in shared memory; the grid is what can be resident at once, in whole clusters.  Where clusters
  // would leave more than a quarter of the SMs' room unused, the launch does without them.
  int grid = 0;
  p.cluster = 1;
  if (tune(kTuneDecodeCluster) != 0) {
    int clusters = 0;
    const cudaError_t ce = rot ? chain_max_clusters<true, G>(&clusters, smem, 8) : chain_max_clusters<false, G>(&clusters, smem, 8);
    if (ce == cudaSuccess && clusters * 8 * 4 >= 2 * sms * 3) {
      p.cluster = 8;
      grid = clusters * 8 < 2 * sms / 8 * 8 ? clusters * 8 : 2 * sms / 8 * 8;
    }
    (void)cudaGetLastError();
  }
  if (p.cluster == 1) {
    int per_sm = 0;
    const cudaError_t e = rot ? chain_kernel_setup<true, G>(&per_sm, smem) : chain_kernel_setup<false, G>(&per_sm, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    if (per_sm > 2) per_sm = 2;
    grid = per_sm * sms;
  }
  if (grid > kMaxSlots - 1) grid = (kMaxSlots - 1) / 8 * 8;

  int phases = 0;
  unsigned int panels_before = 0;
  for (int j = 0; j < count; ++j) {
    const ChainStep& st = steps[j];
    if (j == 0 || st.after_previous) {
      ChainPhase& f = p.phase[phases];
      f.first = j;
      f.chunks = 0;
      f.wait_target = panels_before;
      ++phases;
    }
    ChainPhase& f = p.phase[phases - 1];
    ChainProb& q = p.prob[j];
    q.x = st.x;
    q.packed = reinterpret_cast<const uint8_t*>(st.packed);
    q.scales = reinterpret_cast<const uint8_t*>(st.scales);
    q.y = st.y;
    q.add = st.add;
    q.add_stride = st.add_stride;
    q.K = (int)st.K;
    q.N = (int)st.N;
    q.ng = (int)(st.K / kGroup);
    q.nbs = (int)(st.N / kTileN);
    q.panels = (q.nbs + kPanelTiles - 1) / kPanelTiles;
    q.chunk_begin = f.chunks;
    q.epi = st.epi;
    q.phase = phases - 1;
    q.rms_eps = st.rms_eps;
    if ((long long)f.chunks + (long long)q.panels * q.ng > 0x7FFFFFFFLL / 512) return cudaErrorInvalidValue;
    f.chunks += q.panels * q.ng;
    f.last = j + 1;
    panels_before += (unsigned)q.panels * kPanelTiles;
  }
  p.phases = phases;
  for (int i = 0; i < phases; ++i) {
    ChainPhase& f = p.phase[i];
    f.unit = 1;
    if (f.last - f.first == 1) {
      // a lone step is cut as a lone problem is: whole panels when that loads the CTAs evenly,
      // else a fixed number of CTAs per panel, each with a slice of the panel's groups
      const ChainProb& q = p.prob[f.first];
      const int per = (q.panels + grid - 1) / grid;
      if (q.panels >= grid && (double)q.panels / ((double)per * grid) >= 0.97) f.unit = q.ng;
      if (q.panels < grid) {
        int slices = grid / q.panels < q.ng ? grid / q.panels : q.ng;
        if (slices == 2 && q.ng <= 16) slices = 1;
        // in a cluster launch the CTAs of a panel are 2, 4 or 8 neighbours of one cluster
        if (p.cluster > 1) slices = slices >= 8 ? 8 : (slices >= 4 ? 4 : (slices >= 2 ? 2 : 1));
        f.unit = -slices;
      }
      // tl_e0m4_tuning_set("decode_split" / "decode_slices") force the cut, as for a lone problem
      if (tune(kTuneDecodeSplit) == 1) f.unit = q.ng;
      if (tune(kTuneDecodeSplit) == 2) f.unit = 1;
      const int64_t forced = tune(kTuneDecodeSlices);
      if (forced >= 1 && forced <= q.ng && forced * q.panels <= grid &&
          (p.cluster == 1 || forced == 1 || forced == 2 || forced == 4 || forced == 8))
        f.unit = -(int)forced;
    }
  }
  const cudaError_t e =
      rot ? chain_kernel_launch<true, G>(p, grid, smem, stream) : chain_kernel_launch<false, G>(p, grid, smem, stream);
  count_launch();
  return e;
}

}  // namespace

size_t decode_chain_workspace_bytes() { return (size_t)kMaxSlots * kSlotBytes + 256; }

cudaError_t launch_gemv_decode_chain(const ChainStep* steps, int count, int M, void* workspace, cudaStream_t stream,
                                     int group) {
  for (int j0 = 0; j0 < count; j0 += kMaxChain) {
    const int n = count - j0 < kMaxChain ? count - j0 : kMaxChain;
    const cudaError_t e = group == 32   ? launch_chain<32>(steps + j0, n, M, workspace, stream)
                          : group == 64 ? launch_chain<64>(steps + j0, n, M, workspace, stream)
                                        : launch_chain<kGroup>(steps + j0, n, M, workspace, stream);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------- variant with built-in scratch
namespace {

// Split-panel scratch of the decode kernel for callers that may not allocate device memory and
// so have no workspace to pass: the same kMaxSlots slots a caller-supplied workspace holds
// (about 2.6 MB), reserved in every GPU that loads this library for as long as it stays loaded.
static __device__ __align__(256) unsigned char g_builtin_scratch[kMaxSlots * kSlotBytes];

}  // namespace

size_t builtin_scratch_bytes() { return (size_t)kMaxSlots * kSlotBytes; }

cudaError_t launch_gemv_decode_builtin(const __half* x, const uint32_t* packed, const uint32_t* scales,
                                       __half* y, int M, int64_t K, int64_t N, cudaStream_t stream, int group) {
  // In host code `g_builtin_scratch` is only a handle; the kernel needs the device address,
  // which is looked up once per device while that device is current.
  // (Host threads may race to fill an entry; they all store the same address, atomically.)
  static std::atomic<void*> address[64];
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  void* ptr = (dev >= 0 && dev < 64) ? address[dev].load(std::memory_order_acquire) : nullptr;
  if (!ptr) {
    e = cudaGetSymbolAddress(&ptr, g_builtin_scratch);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorUnknown;
    if (dev >= 0 && dev < 64) address[dev].store(ptr, std::memory_order_release);
  }
  // The array keeps whatever the previous call left (zero after a call that ran to completion,
  // anything after one that was cut short), so it is cleared on the stream before every launch.
  e = cudaMemsetAsync(ptr, 0, builtin_scratch_bytes(), stream);
  if (e != cudaSuccess) return e;
  DecodeProblem q{x, packed, scales, y, K, N, nullptr, false};
  return launch_batch_group<1>(&q, 1, M, ptr, stream, group);
}

cudaError_t read_decode_status(unsigned int* out, cudaStream_t stream) {
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  cudaError_t e = cudaMemcpyAsync(out, status, sizeof(unsigned int), cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return e;
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return e;
  if (*out != 0) {
    const unsigned int zero = 0;
    e = cudaMemcpyAsync(status, &zero, sizeof(unsigned int), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  }
  return e;
}

}  // namespace tl
