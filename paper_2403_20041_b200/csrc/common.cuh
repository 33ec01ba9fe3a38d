// Shared device/host helpers of the E0M4 library (layout rule, bit construction).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tl_e0m4.h"

namespace tl {

constexpr int kGroup = 128;  // default quantization group along K (Section 3.1) = rows of a packed tile;
                             // groups of 64 and 32 rows split a tile row into 2 and 4 scale words per column
constexpr int kTileN = 16;   // columns per packed tile
constexpr int kTileWords = 256;  // uint32 words per packed tile (16 columns x 128 codes / 8)
constexpr int kPanelTiles = 8;   // column blocks per panel (128 columns)

// Position of tile (column n, group g) in the packed stream: panels of up to 8 column blocks
// are stored one after the other; inside a panel the tiles of one group are neighbours.
__host__ __device__ __forceinline__ size_t tile_index(int n, int g, int ng, int N) {
  const int nb = n / kTileN;
  const int p = nb / kPanelTiles;
  const int r = nb % kPanelTiles;
  const int rest = N / kTileN - kPanelTiles * p;
  const int R = rest < kPanelTiles ? rest : kPanelTiles;
  return (size_t)p * kPanelTiles * ng + (size_t)g * R + r;
}

// Dequantization constants of Section 2.3 for the binade [2, 4), replicated in both halves of
// a 32-bit register: CONST_EXP_BIN_PART = 0x4000, the nibble lands on fraction bits 9..6.
constexpr uint32_t kExpPart2 = 0x40004000u;
constexpr uint32_t kNibMask2 = 0x03C003C0u;

// One packed word holds eight consecutive k of one column; the code of k%8 = c sits in nibble
// c/2 + 4*(c%2).  The four shift/mask/OR steps below therefore yield the half2 pairs
// (k0,k1), (k2,k3), (k4,k5), (k6,k7) in natural order, each half being
// as_half(0x4000 | code << 6) = 2 + code/8.
__device__ __forceinline__ void e0m4_construct8(uint32_t w, uint32_t& e01, uint32_t& e23,
                                                uint32_t& e45, uint32_t& e67) {
  e01 = ((w << 6) & kNibMask2) | kExpPart2;
  e23 = ((w << 2) & kNibMask2) | kExpPart2;
  e45 = ((w >> 2) & kNibMask2) | kExpPart2;
  e67 = ((w >> 6) & kNibMask2) | kExpPart2;
}

__device__ __forceinline__ int nibble_pos(int k_local) { return (k_local >> 1) + 4 * (k_local & 1); }

// Counter of kernel launches issued by the library (host side).
void count_launch(int n = 1);

// Host launchers implemented in the .cu files; all return a cudaError_t from the launch.
cudaError_t launch_quantize(const void* w, tl_dtype dt, int64_t K, int64_t N, uint32_t* packed,
                            uint32_t* scales, cudaStream_t stream, int group = kGroup);
// Same container, codes of the group-wise asymmetric INT4 format (Section 3.4's comparison format).
cudaError_t launch_quantize_int4(const void* w, tl_dtype dt, int64_t K, int64_t N, uint32_t* packed,
                                 uint32_t* scales, cudaStream_t stream, int group = kGroup);
cudaError_t launch_dequant(const uint32_t* packed, const uint32_t* scales, int64_t K, int64_t N,
                           __half* out, cudaStream_t stream, int group = kGroup);
// In-place KV-cache append: cache[b, h, pos[b] + s, :] = fresh[b, h, s, :]; D % 8 == 0.
cudaError_t launch_kv_append(void* cache, const void* fresh, const int* pos, int64_t B, int64_t H, int64_t L, int64_t S,
                             int64_t D, unsigned int* status, cudaStream_t stream);
// Fused rms-norm with optional residual add; K % 8 == 0, K <= kMaxNormK.
constexpr int64_t kMaxNormK = 32768;
cudaError_t launch_rmsnorm(const __half* x, const __half* r, const __half* gamma, __half* s_out, __half* y, int64_t M,
                           int64_t K, float eps, cudaStream_t stream);
// Fused layer-norm (mean removed, biased variance, beta added); same limits.
cudaError_t launch_layernorm(const __half* x, const __half* r, const __half* gamma, const __half* beta, __half* s_out,
                             __half* y, int64_t M, int64_t K, float eps, cudaStream_t stream);
// Decode kernels.  `workspace` holds decode_workspace_bytes() bytes that are zero on entry and
// are left zero.  A batch is a list of independent problems sharing M (<= 16).
struct DecodeProblem {
  const __half* x;
  const uint32_t* packed;
  const uint32_t* scales;
  __half* y;
  int64_t K, N;
  const __half* add = nullptr;  // optional fp16 [M, N]: y = fp16(x W + add); may alias y
  bool swiglu = false;          // single-problem launches: y[M, N/2] = silu(gate) * up over column blocks of 8
  int64_t add_stride = -1;      // elements between the addend's token rows; -1 = N, 0 = one bias row for all tokens
};
constexpr int kMaxDecodeBatch = 192;  // problems per launch (the 160 matrices of a 40-layer stack fit one); longer lists take several
size_t decode_workspace_bytes();
cudaError_t launch_gemv_decode(const __half* x, const uint32_t* packed, const uint32_t* scales,
                               __half* y, int64_t M, int64_t K, int64_t N, void* workspace,
                               cudaStream_t stream, const __half* add = nullptr, bool swiglu = false,
                               int group = kGroup, int64_t add_stride = -1);
cudaError_t launch_gemv_decode_batch(const DecodeProblem* probs, int count, int M, void* workspace,
                                     cudaStream_t stream, int group = kGroup);
// A chain of decode steps (M <= 8) in one persistent launch per 128 steps: a step with
// `after_previous` set starts only when all earlier steps are complete, the others stream together
// with their predecessor.  epi: 0 plain, 1 addend (add_stride N: a matrix, 0: a bias row), 2 SwiGLU.
// rms_eps >= 0: every output row is scaled by rsqrt(mean_k x[m, k]^2 + eps) before the epilogue.
// `workspace` holds decode_chain_workspace_bytes() bytes, zero on entry and left zero.
struct ChainStep {
  const __half* x;
  const uint32_t* packed;
  const uint32_t* scales;
  __half* y;
  const __half* add;
  int64_t add_stride;
  int64_t K, N;
  int epi;
  bool after_previous;
  float rms_eps;
};
size_t decode_chain_workspace_bytes();
cudaError_t launch_gemv_decode_chain(const ChainStep* steps, int count, int M, void* workspace, cudaStream_t stream,
                                     int group = kGroup);
// Decode launch that uses the library's own file-scope scratch array instead of a workspace.
size_t builtin_scratch_bytes();
cudaError_t launch_gemv_decode_builtin(const __half* x, const uint32_t* packed, const uint32_t* scales,
                                       __half* y, int M, int64_t K, int64_t N, cudaStream_t stream,
                                       int group = kGroup);
// Tensor-core kernel (tcgen05, dequantized weights as the tensor-memory operand) for every M above
// the register decode kernel's range.  `workspace` holds gemm_tc_workspace_bytes(M, K, N) bytes
// (split-K scratch, zero on entry and left zero; 0 bytes when no split is used).  `status` is the
// device status word.
size_t gemm_tc_workspace_bytes(int64_t M, int64_t K, int64_t N, int bits = 4);
cudaError_t launch_gemm_tc(const __half* x, const uint32_t* packed, const uint32_t* scales, __half* y,
                           int64_t M, int64_t K, int64_t N, void* workspace, unsigned int* status,
                           cudaStream_t stream, const __half* add = nullptr, bool swiglu = false,
                           int group = kGroup, int64_t add_stride = -1, int bits = 4);
// E0M8 (eight fraction bits kept, one byte per code, groups of 128): quantizer and dequantizer; the
// matmul is launch_gemm_tc with bits = 8 (plain epilogue), for every M.
cudaError_t launch_quantize8(const void* w, tl_dtype dt, int64_t K, int64_t N, uint8_t* packed, uint32_t* scales,
                             cudaStream_t stream);
cudaError_t launch_dequant8(const uint8_t* packed, const uint32_t* scales, int64_t K, int64_t N, __half* out,
                            cudaStream_t stream);
// E0M3 / E0M5 (three or five fraction bits kept, units of eight codes in `bits` bytes, groups of 128):
// quantizer and dequantizer; the matmul is launch_gemm_tc with bits = 3 or 5 (plain epilogue), for every M.
cudaError_t launch_quantize_x(const void* w, tl_dtype dt, int64_t K, int64_t N, int bits, uint8_t* packed,
                              uint32_t* scales, cudaStream_t stream);
cudaError_t launch_dequant_x(const uint8_t* packed, const uint32_t* scales, int64_t K, int64_t N, int bits, __half* out,
                             cudaStream_t stream);
// Tensor-core kernel over a list of independent problems that share M (at most kMaxTcBatchM tokens;
// longer lists take several launches).  `workspace` holds gemm_tc_batch_workspace_bytes() bytes, zero
// on entry and left zero.
// Problems per launch: their tensor maps travel as kernel parameters, and the whole parameter
// block stays within the first 4 KB of parameter space (22 maps of 128 bytes + 22 descriptors):
// a tensor copy whose map lay beyond that offset faulted.
constexpr int kMaxTcBatch = 22;
constexpr int kMaxTcBatchM = 128;
size_t gemm_tc_batch_workspace_bytes();
cudaError_t launch_gemm_tc_batch(const DecodeProblem* probs, int count, int M, void* workspace, unsigned int* status,
                                 cudaStream_t stream, int group = kGroup, int bits = 4);
// Device address of the status word that kernels raise when a bounded wait gives up.
unsigned int* device_status_ptr();
// Copies the device status word to *out (synchronizes the stream) and clears it if set.
cudaError_t read_decode_status(unsigned int* out, cudaStream_t stream);

}  // namespace tl
