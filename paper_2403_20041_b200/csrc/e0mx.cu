// E0M3 and E0M5: the construction of Section 2.3 with three or five fraction bits kept (the section
// notes that the method carries over to other bit widths).  A code is the `bits` highest fraction
// bits of w1 in [2, 4): as_half(0x4000 | code << (10 - bits)) = 2 + code / 2^(bits - 1); range,
// stored scale, truncated bias, clip and rounding bit are the steps of the 4-bit quantizer with
// 2^bits for 16.
//
// Container: the tiles of the 4-bit layout in the same order.  Eight consecutive k of one column
// are a unit of `bits` bytes, a little-endian integer in which the code of k % 8 = c occupies bits
// c * bits .. (c + 1) * bits - 1; in a tile column n % 16 owns its 16 units one after the other
// (16 * bits bytes: 48 or 80, a multiple of 16), so the 128 codes of a column's tile row are one
// continuous bit string and a tile is 256 * bits bytes.  The coefficient words ({fp16 d, fp16 b}
// per group and column) do not change.  Group size 128 only.
//
// One thread owns one group (128 consecutive k of one column), as in the other quantizers: a
// warp's reads of W[K, N] and its writes of the dense output are coalesced row segments.
#include "common.cuh"
#include "ptx.cuh"

namespace tl {
namespace {

__device__ __forceinline__ float load_wx(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_wx(const __half* p) { return __half2float(__ldg(p)); }

template <typename T, int BITS>
__global__ void __launch_bounds__(128)
quantize_x_kernel(const T* __restrict__ w, int K, int N, uint8_t* __restrict__ packed, uint32_t* __restrict__ scales) {
  constexpr int kWords = kGroup * BITS / 32;       // 12 or 20 words of codes per column and tile
  constexpr uint32_t kTopCode = (1u << BITS) - 1u;
  constexpr float kPerUnit = (float)(1 << (BITS - 1));  // code steps per unit of w1
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (n >= N) return;
  const int ng = K / kGroup;
  const T* col = w + (size_t)g * kGroup * N + n;
  const size_t tile = tile_index(n, g, ng, N);

  // the group's values are read once and stay in registers for both passes
  float vals[kGroup];
#pragma unroll
  for (int k = 0; k < kGroup; ++k) vals[k] = load_wx(col + (size_t)k * N);
  // 1. range of the group, widened to contain 0
  float lo = 0.0f, hi = 0.0f;
#pragma unroll
  for (int k = 0; k < kGroup; ++k) {
    lo = fminf(lo, vals[k]);
    hi = fmaxf(hi, vals[k]);
  }
  const float kBase = 2.0f;
  const float kTop = 3.998046875f;   // 4 - 2^-9: the largest fp16 below 4
  const float kSpan = 1.998046875f;
  // 2. stored dequantization scale d (fp16), saturated at 65504
  __half d_h = __float2half_rn(__fdiv_rn(__fsub_rn(hi, lo), kSpan));
  if (__hisinf(d_h)) d_h = __ushort_as_half((unsigned short)0x7BFF);
  const float d_f = __half2float(d_h);
  const bool dead = (d_f == 0.0f);
  // 3. forward scale and the bias truncated to the 2^bits-point grid
  const float s = dead ? 0.0f : __fdiv_rn(1.0f, d_f);
  const float t = __fmul_rn(__fmul_rn(-lo, s), kPerUnit);
  const int z = dead ? 0 : (int)fminf(fmaxf(floorf(t), 0.0f), (float)kTopCode);
  const float b = __fadd_rn(kBase, __fmul_rn((float)z, 1.0f / kPerUnit));  // exact

  // 4. codes: the `bits` highest fraction bits of w1 plus the rounding bit, saturated; the column's
  //    128 codes are appended to one little-endian bit string
  uint32_t words[kWords];
#pragma unroll
  for (int i = 0; i < kWords; ++i) words[i] = 0u;
#pragma unroll
  for (int k = 0; k < kGroup; ++k) {
    float w1 = __fadd_rn(__fmul_rn(vals[k], s), b);
    w1 = fminf(fmaxf(w1, kBase), kTop);
    const uint32_t top = (__float_as_uint(w1) >> (23 - BITS - 1)) & ((2u << BITS) - 1u);
    uint32_t q = (top >> 1) + (top & 1u);
    q = q > kTopCode ? kTopCode : q;
    if (dead) q = 0;
    const int at = k * BITS, wi = at >> 5, sh = at & 31;
    words[wi] |= q << sh;
    if (sh + BITS > 32) words[wi + 1] |= q >> (32 - sh);
  }
  uint4* out = reinterpret_cast<uint4*>(packed + tile * (256 * BITS) + (n % kTileN) * (16 * BITS));
#pragma unroll
  for (int v = 0; v < kWords / 4; ++v) out[v] = make_uint4(words[4 * v], words[4 * v + 1], words[4 * v + 2], words[4 * v + 3]);
  const uint32_t b_bits = 0x4000u | ((uint32_t)z << (10 - BITS));
  scales[tile * kTileN + (n % kTileN)] = (uint32_t)__half_as_ushort(d_h) | (b_bits << 16);
}

template <int BITS>
__global__ void __launch_bounds__(128)
dequant_x_kernel(const uint8_t* __restrict__ packed, const uint32_t* __restrict__ scales, int K, int N,
                 __half* __restrict__ out) {
  constexpr int kWords = kGroup * BITS / 32;
  // programmatic dependent launch: the packed tensor may be the previous kernel's output
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (n >= N) return;
  const int ng = K / kGroup;
  const size_t tile = tile_index(n, g, ng, N);
  const uint4* src = reinterpret_cast<const uint4*>(packed + tile * (256 * BITS) + (n % kTileN) * (16 * BITS));
  uint32_t words[kWords + 1];
#pragma unroll
  for (int v = 0; v < kWords / 4; ++v) {
    const uint4 q = src[v];
    words[4 * v] = q.x;
    words[4 * v + 1] = q.y;
    words[4 * v + 2] = q.z;
    words[4 * v + 3] = q.w;
  }
  words[kWords] = 0u;
  const uint32_t sc = scales[tile * kTileN + (n % kTileN)];
  const __half d = __ushort_as_half((unsigned short)(sc & 0xFFFFu));
  const __half b = __ushort_as_half((unsigned short)(sc >> 16));
  __half* dst = out + (size_t)g * kGroup * N + n;
#pragma unroll
  for (int k = 0; k < kGroup; ++k) {
    const int at = k * BITS, wi = at >> 5, sh = at & 31;
    const uint32_t q = __funnelshift_r(words[wi], words[wi + 1], sh) & ((1u << BITS) - 1u);
    // the formula of Section 2.3: CONST_EXP_BIN_PART | (code << CONST_BIT_SHIFT_NUM), shift = 10 - bits
    const __half w1 = __ushort_as_half((unsigned short)(0x4000u | (q << (10 - BITS))));
    dst[(size_t)k * N] = __hmul(__hsub(w1, b), d);
  }
}

}  // namespace

cudaError_t launch_quantize_x(const void* w, tl_dtype dt, int64_t K, int64_t N, int bits, uint8_t* packed,
                              uint32_t* scales, cudaStream_t stream) {
  dim3 block(128);
  dim3 grid((unsigned)((N + 127) / 128), (unsigned)(K / kGroup));
  const int k = (int)K, n = (int)N;
  if (bits == 3) {
    if (dt == TL_F32) quantize_x_kernel<float, 3><<<grid, block, 0, stream>>>(static_cast<const float*>(w), k, n, packed, scales);
    else quantize_x_kernel<__half, 3><<<grid, block, 0, stream>>>(static_cast<const __half*>(w), k, n, packed, scales);
  } else if (bits == 5) {
    if (dt == TL_F32) quantize_x_kernel<float, 5><<<grid, block, 0, stream>>>(static_cast<const float*>(w), k, n, packed, scales);
    else quantize_x_kernel<__half, 5><<<grid, block, 0, stream>>>(static_cast<const __half*>(w), k, n, packed, scales);
  } else {
    return cudaErrorInvalidValue;
  }
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_dequant_x(const uint8_t* packed, const uint32_t* scales, int64_t K, int64_t N, int bits, __half* out,
                             cudaStream_t stream) {
  if (bits != 3 && bits != 5) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((N + 127) / 128), (unsigned)(K / kGroup));
  cfg.blockDim = dim3(128);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int k = (int)K, n = (int)N;
  const cudaError_t e = bits == 3 ? cudaLaunchKernelEx(&cfg, dequant_x_kernel<3>, packed, scales, k, n, out)
                                  : cudaLaunchKernelEx(&cfg, dequant_x_kernel<5>, packed, scales, k, n, out);
  count_launch();
  return e;
}

}  // namespace tl
