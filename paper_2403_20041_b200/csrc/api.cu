// extern "C" boundary: argument validation, the M-based dispatcher and the host-buffer variant.
#include <atomic>
#include <cstring>
#include <vector>

#include "common.cuh"
#include "tuning.h"

namespace tl {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// Overrides set by tl_e0m4_tuning_set; -1 = the library's own choice.
static std::atomic<int64_t> g_tuning[kTuneCount];
static struct TuningInit {
  TuningInit() {
    for (auto& v : g_tuning) v.store(-1, std::memory_order_relaxed);
  }
} g_tuning_init;
int64_t tune(TuneKey key) { return g_tuning[key].load(std::memory_order_relaxed); }

namespace {

constexpr int64_t kDecodeMaxM = 16;  // Section 2.2: decoding = vector-matrix, prefill = matrix-matrix
// Inside tl_e0m4_matmul two kernels share the range of M: the register-fragment GEMV kernel up to
// kRegisterMaxM tokens and the tensor-core kernel above.
constexpr int64_t kRegisterMaxM = 8;
inline int64_t register_max_m() {
  const int64_t v = tune(kTuneRegisterMaxM);
  return v >= 1 && v <= kDecodeMaxM ? v : kRegisterMaxM;
}
// Inside tl_e0m4_matmul_batch the GEMV kernel serves up to this many tokens and the tensor-core
// list kernel the rest (measured on a ChatGLM2-6B-shaped stack: equal at 8 tokens, the tensor-core
// kernel 1.3x faster at 9 and 1.5x at 16).
constexpr int64_t kBatchDecodeMaxM = 8;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline tl_status check_shape(int64_t K, int64_t N, int group) {
  if (group != 128 && group != 64 && group != 32) return TL_ERR_SHAPE;
  if (K <= 0 || N <= 0) return TL_ERR_SHAPE;
  if (K % kGroup != 0 || N % kTileN != 0) return TL_ERR_SHAPE;
  if (K > (int64_t)1 << 24 || N > (int64_t)1 << 24) return TL_ERR_SHAPE;
  return TL_OK;
}

// The current device must be a compute-capability 10.x part; the answer is cached per device.
tl_status check_device() {
  static std::atomic<int> cache[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return TL_ERR_CUDA;
  if (dev < 64) {
    const int c = cache[dev].load(std::memory_order_relaxed);
    if (c == 1) return TL_OK;
    if (c == 2) return TL_ERR_ARCH;
  }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return TL_ERR_CUDA;
  const bool ok = (major == 10);
  if (dev < 64) cache[dev].store(ok ? 1 : 2, std::memory_order_relaxed);
  return ok ? TL_OK : TL_ERR_ARCH;
}

inline size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace
}  // namespace tl

using namespace tl;

extern "C" {

tl_status tl_e0m4_packed_sizes(int64_t K, int64_t N, int group, size_t* packed_bytes,
                               size_t* scales_bytes) {
  const tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (packed_bytes) *packed_bytes = (size_t)K * (size_t)N / 2;
  if (scales_bytes) *scales_bytes = (size_t)(K / group) * (size_t)N * 4;
  return TL_OK;
}

namespace {

tl_status quantize_any(bool int4, const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group,
                       void* packed_dev, void* scales_dev, void* stream) {
  if (!w_dev || !packed_dev || !scales_dev) return TL_ERR_NULL;
  if (w_dtype != TL_F32 && w_dtype != TL_F16) return TL_ERR_DTYPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (!aligned16(w_dev) || !aligned16(packed_dev) || !aligned16(scales_dev)) return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e =
      (int4 ? launch_quantize_int4 : launch_quantize)(w_dev, w_dtype, K, N, static_cast<uint32_t*>(packed_dev),
                                                      static_cast<uint32_t*>(scales_dev),
                                                      static_cast<cudaStream_t>(stream), group);
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

}  // namespace

tl_status tl_e0m4_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group,
                           void* packed_dev, void* scales_dev, void* stream) {
  return quantize_any(false, w_dev, w_dtype, K, N, group, packed_dev, scales_dev, stream);
}

tl_status tl_int4_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group,
                           void* packed_dev, void* scales_dev, void* stream) {
  return quantize_any(true, w_dev, w_dtype, K, N, group, packed_dev, scales_dev, stream);
}

tl_status tl_e0m4_dequant(const void* packed_dev, const void* scales_dev, int64_t K, int64_t N,
                          int group, void* w_f16_dev, void* stream) {
  if (!packed_dev || !scales_dev || !w_f16_dev) return TL_ERR_NULL;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (!aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(w_f16_dev)) return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e =
      launch_dequant(static_cast<const uint32_t*>(packed_dev), static_cast<const uint32_t*>(scales_dev),
                     K, N, static_cast<__half*>(w_f16_dev), static_cast<cudaStream_t>(stream), group);
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

// ---------------------------------------------------------------- E0M8 (eight fraction bits kept)

tl_status tl_e0m8_packed_sizes(int64_t K, int64_t N, int group, size_t* packed_bytes, size_t* scales_bytes) {
  if (group != kGroup) return TL_ERR_SHAPE;
  const tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (packed_bytes) *packed_bytes = (size_t)K * (size_t)N;
  if (scales_bytes) *scales_bytes = (size_t)(K / group) * (size_t)N * 4;
  return TL_OK;
}

tl_status tl_e0m8_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group, void* packed_dev,
                           void* scales_dev, void* stream) {
  if (!w_dev || !packed_dev || !scales_dev) return TL_ERR_NULL;
  if (w_dtype != TL_F32 && w_dtype != TL_F16) return TL_ERR_DTYPE;
  if (group != kGroup) return TL_ERR_SHAPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (!aligned16(w_dev) || !aligned16(packed_dev) || !aligned16(scales_dev)) return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e = launch_quantize8(w_dev, w_dtype, K, N, static_cast<uint8_t*>(packed_dev),
                                         static_cast<uint32_t*>(scales_dev), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_e0m8_dequant(const void* packed_dev, const void* scales_dev, int64_t K, int64_t N, int group,
                          void* w_f16_dev, void* stream) {
  if (!packed_dev || !scales_dev || !w_f16_dev) return TL_ERR_NULL;
  if (group != kGroup) return TL_ERR_SHAPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (!aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(w_f16_dev)) return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e =
      launch_dequant8(static_cast<const uint8_t*>(packed_dev), static_cast<const uint32_t*>(scales_dev), K, N,
                      static_cast<__half*>(w_f16_dev), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

size_t tl_e0m8_matmul_workspace(int64_t M, int64_t K, int64_t N) {
  if (M <= 0 || K <= 0 || N <= 0 || K % kGroup != 0 || N % kTileN != 0) return 0;
  return gemm_tc_workspace_bytes(M, K, N, 8);
}

namespace {

tl_status matmul8_any(const void* x_dev, const void* packed_dev, const void* scales_dev, const void* addend_dev,
                      bool swiglu, int64_t add_stride, void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                      void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!x_dev || !packed_dev || !scales_dev || !y_dev) return TL_ERR_NULL;
  if (group != kGroup) return TL_ERR_SHAPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (M <= 0 || M > (int64_t)1 << 20) return TL_ERR_SHAPE;
  if (!aligned16(x_dev) || !aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(y_dev) ||
      !aligned16(addend_dev))
    return TL_ERR_ALIGN;
  const size_t need = tl_e0m8_matmul_workspace(M, K, N);
  if (need > 0) {
    if (!workspace_dev || workspace_bytes < need) return TL_ERR_WORKSPACE;
    if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  }
  if ((st = check_device()) != TL_OK) return st;
  unsigned int* status = device_status_ptr();
  if (!status) return TL_ERR_CUDA;
  // every M runs on the tensor-core kernel: with a byte per weight its tensor time per byte is half
  // the 4-bit kernel's, below the memory time even at one token
  const cudaError_t e =
      launch_gemm_tc(static_cast<const __half*>(x_dev), static_cast<const uint32_t*>(packed_dev),
                     static_cast<const uint32_t*>(scales_dev), static_cast<__half*>(y_dev), M, K, N, workspace_dev,
                     status, static_cast<cudaStream_t>(stream), static_cast<const __half*>(addend_dev), swiglu, kGroup,
                     add_stride, 8);
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

}  // namespace

tl_status tl_e0m8_matmul(const void* x_dev, const void* packed_dev, const void* scales_dev, void* y_dev, int64_t M,
                         int64_t K, int64_t N, int group, void* workspace_dev, size_t workspace_bytes, void* stream) {
  return matmul8_any(x_dev, packed_dev, scales_dev, nullptr, false, -1, y_dev, M, K, N, group, workspace_dev,
                     workspace_bytes, stream);
}

tl_status tl_e0m8_matmul_add(const void* x_dev, const void* packed_dev, const void* scales_dev, const void* addend_dev,
                             void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                             size_t workspace_bytes, void* stream) {
  if (!addend_dev) return TL_ERR_NULL;
  return matmul8_any(x_dev, packed_dev, scales_dev, addend_dev, false, -1, y_dev, M, K, N, group, workspace_dev,
                     workspace_bytes, stream);
}

tl_status tl_e0m8_matmul_bias(const void* x_dev, const void* packed_dev, const void* scales_dev, const void* bias_dev,
                              void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                              size_t workspace_bytes, void* stream) {
  if (!bias_dev) return TL_ERR_NULL;
  return matmul8_any(x_dev, packed_dev, scales_dev, bias_dev, false, 0, y_dev, M, K, N, group, workspace_dev,
                     workspace_bytes, stream);
}

tl_status tl_e0m8_matmul_swiglu(const void* x_dev, const void* packed_dev, const void* scales_dev, void* y_dev,
                                int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                                size_t workspace_bytes, void* stream) {
  return matmul8_any(x_dev, packed_dev, scales_dev, nullptr, true, -1, y_dev, M, K, N, group, workspace_dev,
                     workspace_bytes, stream);
}

tl_status tl_e0m8_matmul_batch(const tl_e0m4_problem* problems_host, int count, int64_t M, int group,
                               void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!problems_host) return TL_ERR_NULL;
  if (count <= 0 || count > 65536) return TL_ERR_SHAPE;
  if (M <= 0 || M > kMaxTcBatchM || group != kGroup) return TL_ERR_SHAPE;
  if (!workspace_dev) return TL_ERR_NULL;
  for (int j = 0; j < count; ++j) {
    const tl_e0m4_problem& q = problems_host[j];
    if (!q.x_dev || !q.packed_dev || !q.scales_dev || !q.y_dev) return TL_ERR_NULL;
    const tl_status st = check_shape(q.K, q.N, group);
    if (st != TL_OK) return st;
    if (!aligned16(q.x_dev) || !aligned16(q.packed_dev) || !aligned16(q.scales_dev) || !aligned16(q.y_dev))
      return TL_ERR_ALIGN;
  }
  if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  if (workspace_bytes < gemm_tc_batch_workspace_bytes()) return TL_ERR_WORKSPACE;
  const tl_status st = check_device();
  if (st != TL_OK) return st;
  unsigned int* status = device_status_ptr();
  if (!status) return TL_ERR_CUDA;
  DecodeProblem local[kMaxTcBatch];
  for (int j0 = 0; j0 < count; j0 += kMaxTcBatch) {
    const int n = count - j0 < kMaxTcBatch ? count - j0 : kMaxTcBatch;
    for (int j = 0; j < n; ++j) {
      const tl_e0m4_problem& q = problems_host[j0 + j];
      local[j] = DecodeProblem{static_cast<const __half*>(q.x_dev), static_cast<const uint32_t*>(q.packed_dev),
                               static_cast<const uint32_t*>(q.scales_dev), static_cast<__half*>(q.y_dev), q.K, q.N};
    }
    if (launch_gemm_tc_batch(local, n, (int)M, workspace_dev, status, static_cast<cudaStream_t>(stream), kGroup, 8) !=
        cudaSuccess)
      return TL_ERR_CUDA;
  }
  return TL_OK;
}

// ---------------------------------------------------------------- E0M3 / E0M5 (three or five fraction bits kept)

tl_status tl_e0mx_packed_sizes(int64_t K, int64_t N, int group, int bits, size_t* packed_bytes, size_t* scales_bytes) {
  if (group != kGroup || (bits != 3 && bits != 5)) return TL_ERR_SHAPE;
  const tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (packed_bytes) *packed_bytes = (size_t)K * (size_t)N * (size_t)bits / 8;
  if (scales_bytes) *scales_bytes = (size_t)(K / group) * (size_t)N * 4;
  return TL_OK;
}

tl_status tl_e0mx_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group, int bits,
                           void* packed_dev, void* scales_dev, void* stream) {
  if (!w_dev || !packed_dev || !scales_dev) return TL_ERR_NULL;
  if (w_dtype != TL_F32 && w_dtype != TL_F16) return TL_ERR_DTYPE;
  if (group != kGroup || (bits != 3 && bits != 5)) return TL_ERR_SHAPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (!aligned16(w_dev) || !aligned16(packed_dev) || !aligned16(scales_dev)) return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e = launch_quantize_x(w_dev, w_dtype, K, N, bits, static_cast<uint8_t*>(packed_dev),
                                          static_cast<uint32_t*>(scales_dev), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_e0mx_dequant(const void* packed_dev, const void* scales_dev, int64_t K, int64_t N, int group, int bits,
                          void* w_f16_dev, void* stream) {
  if (!packed_dev || !scales_dev || !w_f16_dev) return TL_ERR_NULL;
  if (group != kGroup || (bits != 3 && bits != 5)) return TL_ERR_SHAPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (!aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(w_f16_dev)) return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e =
      launch_dequant_x(static_cast<const uint8_t*>(packed_dev), static_cast<const uint32_t*>(scales_dev), K, N, bits,
                       static_cast<__half*>(w_f16_dev), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

size_t tl_e0mx_matmul_workspace(int64_t M, int64_t K, int64_t N, int bits) {
  if (M <= 0 || K <= 0 || N <= 0 || K % kGroup != 0 || N % kTileN != 0 || (bits != 3 && bits != 5)) return 0;
  return gemm_tc_workspace_bytes(M, K, N, bits);
}

tl_status tl_e0mx_matmul(const void* x_dev, const void* packed_dev, const void* scales_dev, void* y_dev, int64_t M,
                         int64_t K, int64_t N, int group, int bits, void* workspace_dev, size_t workspace_bytes,
                         void* stream) {
  if (!x_dev || !packed_dev || !scales_dev || !y_dev) return TL_ERR_NULL;
  if (group != kGroup || (bits != 3 && bits != 5)) return TL_ERR_SHAPE;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (M <= 0 || M > (int64_t)1 << 20) return TL_ERR_SHAPE;
  if (!aligned16(x_dev) || !aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(y_dev)) return TL_ERR_ALIGN;
  const size_t need = tl_e0mx_matmul_workspace(M, K, N, bits);
  if (need > 0) {
    if (!workspace_dev || workspace_bytes < need) return TL_ERR_WORKSPACE;
    if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  }
  if ((st = check_device()) != TL_OK) return st;
  unsigned int* status = device_status_ptr();
  if (!status) return TL_ERR_CUDA;
  // every M runs on the tensor-core kernel, as for E0M8
  const cudaError_t e =
      launch_gemm_tc(static_cast<const __half*>(x_dev), static_cast<const uint32_t*>(packed_dev),
                     static_cast<const uint32_t*>(scales_dev), static_cast<__half*>(y_dev), M, K, N, workspace_dev,
                     status, static_cast<cudaStream_t>(stream), nullptr, false, kGroup, -1, bits);
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_kernel tl_e0m4_matmul_kernel(int64_t M, int64_t K, int64_t N) {
  (void)K;
  (void)N;
  return M <= register_max_m() ? TL_KERNEL_REGISTER : TL_KERNEL_TENSOR;
}

tl_stage tl_e0m4_matmul_stage(int64_t M) { return M <= kDecodeMaxM ? TL_STAGE_DECODE : TL_STAGE_PREFILL; }

size_t tl_e0m4_matmul_workspace(int64_t M, int64_t K, int64_t N) {
  if (M <= 0 || K <= 0 || N <= 0 || K % kGroup != 0 || N % kTileN != 0) return 0;
  if (M <= register_max_m()) return decode_workspace_bytes();
  const size_t pre = gemm_tc_workspace_bytes(M, K, N);
  return pre > decode_workspace_bytes() ? pre : decode_workspace_bytes();
}

size_t tl_e0m4_matmul_batch_workspace(void) {
  const size_t a = decode_workspace_bytes(), b = gemm_tc_batch_workspace_bytes();
  return a > b ? a : b;
}

tl_status tl_e0m4_matmul_batch(const tl_e0m4_problem* problems_host, int count, int64_t M, int group,
                               void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!problems_host) return TL_ERR_NULL;
  if (count <= 0 || count > 65536) return TL_ERR_SHAPE;
  if (M <= 0 || M > kMaxTcBatchM) return TL_ERR_SHAPE;
  if (!workspace_dev) return TL_ERR_NULL;
  for (int j = 0; j < count; ++j) {
    const tl_e0m4_problem& q = problems_host[j];
    if (!q.x_dev || !q.packed_dev || !q.scales_dev || !q.y_dev) return TL_ERR_NULL;
    const tl_status st = check_shape(q.K, q.N, group);
    if (st != TL_OK) return st;
    if (!aligned16(q.x_dev) || !aligned16(q.packed_dev) || !aligned16(q.scales_dev) || !aligned16(q.y_dev))
      return TL_ERR_ALIGN;
  }
  if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  if (workspace_bytes < tl_e0m4_matmul_batch_workspace()) return TL_ERR_WORKSPACE;
  const tl_status st = check_device();
  if (st != TL_OK) return st;
  // Up to kBatchDecodeMaxM tokens the register-fragment kernel streams the list, above it the
  // tensor-core kernel does (measured crossover; tl_e0m4_tuning_set("batch_tc_min", m) moves it).
  const int64_t tc_min = tune(kTuneBatchTcMin) >= 1 ? tune(kTuneBatchTcMin) : kBatchDecodeMaxM + 1;
  const bool tensor = M > kDecodeMaxM || M >= tc_min;
  unsigned int* status = tensor ? device_status_ptr() : nullptr;
  if (tensor && !status) return TL_ERR_CUDA;
  DecodeProblem local[kMaxDecodeBatch];
  for (int j0 = 0; j0 < count; j0 += kMaxDecodeBatch) {
    const int n = count - j0 < kMaxDecodeBatch ? count - j0 : kMaxDecodeBatch;
    for (int j = 0; j < n; ++j) {
      const tl_e0m4_problem& q = problems_host[j0 + j];
      local[j] = DecodeProblem{static_cast<const __half*>(q.x_dev), static_cast<const uint32_t*>(q.packed_dev),
                               static_cast<const uint32_t*>(q.scales_dev), static_cast<__half*>(q.y_dev),
                               q.K, q.N};
    }
    const cudaError_t e =
        tensor ? launch_gemm_tc_batch(local, n, (int)M, workspace_dev, status, static_cast<cudaStream_t>(stream), group)
               : launch_gemv_decode_batch(local, n, (int)M, workspace_dev, static_cast<cudaStream_t>(stream), group);
    if (e != cudaSuccess) return TL_ERR_CUDA;
  }
  return TL_OK;
}

namespace {

tl_status matmul_any(const void* x_dev, const void* packed_dev, const void* scales_dev, const void* addend_dev,
                     bool swiglu, void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                     size_t workspace_bytes, void* stream, int64_t add_stride = -1) {
  if (!x_dev || !packed_dev || !scales_dev || !y_dev) return TL_ERR_NULL;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (M <= 0 || M > (int64_t)1 << 20) return TL_ERR_SHAPE;
  if (!aligned16(x_dev) || !aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(y_dev) ||
      !aligned16(addend_dev))
    return TL_ERR_ALIGN;
  const size_t need = tl_e0m4_matmul_workspace(M, K, N);
  if (need > 0) {
    if (!workspace_dev || workspace_bytes < need) return TL_ERR_WORKSPACE;
    if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  }
  if ((st = check_device()) != TL_OK) return st;
  const cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* add = static_cast<const __half*>(addend_dev);
  cudaError_t e;
  if (M <= register_max_m()) {
    e = launch_gemv_decode(static_cast<const __half*>(x_dev), static_cast<const uint32_t*>(packed_dev),
                           static_cast<const uint32_t*>(scales_dev), static_cast<__half*>(y_dev), M, K,
                           N, workspace_dev, s, add, swiglu, group, add_stride);
  } else {
    unsigned int* status = device_status_ptr();
    if (!status) return TL_ERR_CUDA;
    e = launch_gemm_tc(static_cast<const __half*>(x_dev), static_cast<const uint32_t*>(packed_dev),
                       static_cast<const uint32_t*>(scales_dev), static_cast<__half*>(y_dev), M, K, N,
                       workspace_dev, status, s, add, swiglu, group, add_stride);
  }
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

}  // namespace

tl_status tl_e0m4_matmul(const void* x_dev, const void* packed_dev, const void* scales_dev,
                         void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                         void* workspace_dev, size_t workspace_bytes, void* stream) {
  return matmul_any(x_dev, packed_dev, scales_dev, nullptr, false, y_dev, M, K, N, group, workspace_dev,
                    workspace_bytes, stream);
}

tl_status tl_e0m4_matmul_add(const void* x_dev, const void* packed_dev, const void* scales_dev,
                             const void* addend_dev, void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                             void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!addend_dev) return TL_ERR_NULL;
  return matmul_any(x_dev, packed_dev, scales_dev, addend_dev, false, y_dev, M, K, N, group, workspace_dev,
                    workspace_bytes, stream);
}

tl_status tl_e0m4_matmul_bias(const void* x_dev, const void* packed_dev, const void* scales_dev,
                              const void* bias_dev, void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                              void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!bias_dev) return TL_ERR_NULL;
  return matmul_any(x_dev, packed_dev, scales_dev, bias_dev, false, y_dev, M, K, N, group, workspace_dev,
                    workspace_bytes, stream, 0);
}

tl_status tl_e0m4_matmul_swiglu(const void* x_dev, const void* packed_dev, const void* scales_dev,
                                void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                                void* workspace_dev, size_t workspace_bytes, void* stream) {
  return matmul_any(x_dev, packed_dev, scales_dev, nullptr, true, y_dev, M, K, N, group, workspace_dev,
                    workspace_bytes, stream);
}

size_t tl_e0m4_matmul_chain_workspace(void) { return decode_chain_workspace_bytes(); }

tl_status tl_e0m4_matmul_chain(const tl_e0m4_step* steps_host, int count, int64_t M, int group,
                               void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!steps_host || !workspace_dev) return TL_ERR_NULL;
  if (count <= 0 || count > 65536) return TL_ERR_SHAPE;
  if (M <= 0 || M > kRegisterMaxM) return TL_ERR_SHAPE;
  std::vector<ChainStep> steps((size_t)count);
  for (int j = 0; j < count; ++j) {
    const tl_e0m4_step& q = steps_host[j];
    if (!q.x_dev || !q.packed_dev || !q.scales_dev || !q.y_dev) return TL_ERR_NULL;
    const tl_status st = check_shape(q.K, q.N, group);
    if (st != TL_OK) return st;
    if (q.epilogue < TL_EPILOGUE_NONE || q.epilogue > TL_EPILOGUE_SWIGLU) return TL_ERR_SHAPE;
    const bool wants_addend = q.epilogue == TL_EPILOGUE_ADD || q.epilogue == TL_EPILOGUE_BIAS;
    if (wants_addend && !q.addend_dev) return TL_ERR_NULL;
    if (q.rms_scale && !(q.rms_eps >= 0.0f)) return TL_ERR_SHAPE;
    if (!aligned16(q.x_dev) || !aligned16(q.packed_dev) || !aligned16(q.scales_dev) || !aligned16(q.y_dev) ||
        (wants_addend && !aligned16(q.addend_dev)))
      return TL_ERR_ALIGN;
    ChainStep& c = steps[(size_t)j];
    c.x = static_cast<const __half*>(q.x_dev);
    c.packed = static_cast<const uint32_t*>(q.packed_dev);
    c.scales = static_cast<const uint32_t*>(q.scales_dev);
    c.y = static_cast<__half*>(q.y_dev);
    c.add = wants_addend ? static_cast<const __half*>(q.addend_dev) : nullptr;
    c.add_stride = q.epilogue == TL_EPILOGUE_ADD ? q.N : 0;
    c.K = q.K;
    c.N = q.N;
    c.epi = wants_addend ? 1 : (q.epilogue == TL_EPILOGUE_SWIGLU ? 2 : 0);
    c.after_previous = q.after_previous != 0;
    c.rms_eps = q.rms_scale ? q.rms_eps : -1.0f;
  }
  if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  if (workspace_bytes < decode_chain_workspace_bytes()) return TL_ERR_WORKSPACE;
  const tl_status st = check_device();
  if (st != TL_OK) return st;
  const cudaError_t e =
      launch_gemv_decode_chain(steps.data(), count, (int)M, workspace_dev, static_cast<cudaStream_t>(stream), group);
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_e0m4_matmul_noalloc(const void* x_dev, const void* packed_dev, const void* scales_dev,
                                 void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* stream) {
  if (!x_dev || !packed_dev || !scales_dev || !y_dev) return TL_ERR_NULL;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (M <= 0) return TL_ERR_SHAPE;
  if (M > kDecodeMaxM) return TL_ERR_LIMIT;  // the built-in scratch holds 16 tokens per column
  if (!aligned16(x_dev) || !aligned16(packed_dev) || !aligned16(scales_dev) || !aligned16(y_dev))
    return TL_ERR_ALIGN;
  if ((st = check_device()) != TL_OK) return st;
  const cudaError_t e = launch_gemv_decode_builtin(
      static_cast<const __half*>(x_dev), static_cast<const uint32_t*>(packed_dev),
      static_cast<const uint32_t*>(scales_dev), static_cast<__half*>(y_dev), (int)M, K, N,
      static_cast<cudaStream_t>(stream), group);
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

size_t tl_e0m4_matmul_noalloc_scratch_bytes(void) { return builtin_scratch_bytes(); }

tl_status tl_e0m4_matmul_batch_host(const tl_e0m4_problem* problems_host, int count, int64_t M,
                                    int group, const void* x_host, void* x_stage_dev, size_t x_bytes,
                                    void* y_host, const void* y_stage_dev, size_t y_bytes,
                                    void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!x_host || !x_stage_dev || !y_host || !y_stage_dev) return TL_ERR_NULL;
  if (!problems_host) return TL_ERR_NULL;
  if (count <= 0) return TL_ERR_SHAPE;
  const char* xs = static_cast<const char*>(x_stage_dev);
  const char* ys = static_cast<const char*>(y_stage_dev);
  for (int j = 0; j < count; ++j) {
    const tl_e0m4_problem& q = problems_host[j];
    if (!q.x_dev || !q.y_dev) return TL_ERR_NULL;
    if (q.K <= 0 || q.N <= 0 || M <= 0) return TL_ERR_SHAPE;
    const char* xq = static_cast<const char*>(q.x_dev);
    const char* yq = static_cast<const char*>(q.y_dev);
    if (xq < xs || xq + (size_t)M * q.K * 2 > xs + x_bytes) return TL_ERR_SHAPE;
    if (yq < ys || yq + (size_t)M * q.N * 2 > ys + y_bytes) return TL_ERR_SHAPE;
  }
  const cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(x_stage_dev, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return TL_ERR_CUDA;
  const tl_status st =
      tl_e0m4_matmul_batch(problems_host, count, M, group, workspace_dev, workspace_bytes, stream);
  if (st != TL_OK) return st;
  if (cudaMemcpyAsync(y_host, y_stage_dev, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return TL_ERR_CUDA;
  return TL_OK;
}

size_t tl_e0m4_matmul_host_staging(int64_t M, int64_t K, int64_t N) {
  if (M <= 0 || K <= 0 || N <= 0) return 0;
  return round256((size_t)M * K * 2) + round256((size_t)M * N * 2) +
         round256(tl_e0m4_matmul_workspace(M, K, N));
}

tl_status tl_e0m4_matmul_host(const void* x_host, const void* packed_dev, const void* scales_dev,
                              void* y_host, int64_t M, int64_t K, int64_t N, int group,
                              void* staging_dev, size_t staging_bytes, void* stream) {
  if (!x_host || !y_host || !packed_dev || !scales_dev || !staging_dev) return TL_ERR_NULL;
  tl_status st = check_shape(K, N, group);
  if (st != TL_OK) return st;
  if (M <= 0 || M > (int64_t)1 << 20) return TL_ERR_SHAPE;
  if (!aligned16(staging_dev)) return TL_ERR_ALIGN;
  if (staging_bytes < tl_e0m4_matmul_host_staging(M, K, N)) return TL_ERR_WORKSPACE;
  if ((st = check_device()) != TL_OK) return st;
  const cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t x_bytes = (size_t)M * K * 2, y_bytes = (size_t)M * N * 2;
  char* base = static_cast<char*>(staging_dev);
  void* x_dev = base;
  void* y_dev = base + round256(x_bytes);
  void* ws = base + round256(x_bytes) + round256(y_bytes);
  const size_t ws_bytes = tl_e0m4_matmul_workspace(M, K, N);
  if (cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return TL_ERR_CUDA;
  st = tl_e0m4_matmul(x_dev, packed_dev, scales_dev, y_dev, M, K, N, group, ws_bytes ? ws : nullptr,
                      ws_bytes, stream);
  if (st != TL_OK) return st;
  if (cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return TL_ERR_CUDA;
  return TL_OK;
}

tl_status tl_rmsnorm(const void* x_dev, const void* residual_dev, const void* gamma_dev, void* sum_out_dev,
                     void* y_dev, int64_t M, int64_t K, float eps, void* stream) {
  if (!x_dev || !gamma_dev || !y_dev) return TL_ERR_NULL;
  if (sum_out_dev && !residual_dev) return TL_ERR_NULL;
  if (M <= 0 || M > (int64_t)1 << 24 || K <= 0 || K % 8 != 0 || K > kMaxNormK) return TL_ERR_SHAPE;
  if (!(eps >= 0.0f)) return TL_ERR_SHAPE;
  if (!aligned16(x_dev) || !aligned16(gamma_dev) || !aligned16(y_dev) || !aligned16(residual_dev) ||
      !aligned16(sum_out_dev))
    return TL_ERR_ALIGN;
  const tl_status st = check_device();
  if (st != TL_OK) return st;
  const cudaError_t e = launch_rmsnorm(static_cast<const __half*>(x_dev), static_cast<const __half*>(residual_dev),
                                       static_cast<const __half*>(gamma_dev), static_cast<__half*>(sum_out_dev),
                                       static_cast<__half*>(y_dev), M, K, eps, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_layernorm(const void* x_dev, const void* residual_dev, const void* gamma_dev, const void* beta_dev,
                       void* sum_out_dev, void* y_dev, int64_t M, int64_t K, float eps, void* stream) {
  if (!x_dev || !gamma_dev || !beta_dev || !y_dev) return TL_ERR_NULL;
  if (sum_out_dev && !residual_dev) return TL_ERR_NULL;
  if (M <= 0 || M > (int64_t)1 << 24 || K <= 0 || K % 8 != 0 || K > kMaxNormK) return TL_ERR_SHAPE;
  if (!(eps >= 0.0f)) return TL_ERR_SHAPE;
  if (!aligned16(x_dev) || !aligned16(gamma_dev) || !aligned16(beta_dev) || !aligned16(y_dev) ||
      !aligned16(residual_dev) || !aligned16(sum_out_dev))
    return TL_ERR_ALIGN;
  const tl_status st = check_device();
  if (st != TL_OK) return st;
  const cudaError_t e =
      launch_layernorm(static_cast<const __half*>(x_dev), static_cast<const __half*>(residual_dev),
                       static_cast<const __half*>(gamma_dev), static_cast<const __half*>(beta_dev),
                       static_cast<__half*>(sum_out_dev), static_cast<__half*>(y_dev), M, K, eps,
                       static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_kv_append(void* cache_dev, const void* new_dev, const void* position_ids_dev, int64_t B, int64_t H,
                       int64_t L, int64_t S, int64_t D, void* stream) {
  if (!cache_dev || !new_dev || !position_ids_dev) return TL_ERR_NULL;
  if (B <= 0 || H <= 0 || L <= 0 || S <= 0 || D <= 0 || S > L || D % 8 != 0) return TL_ERR_SHAPE;
  if (B > (int64_t)1 << 20 || H > (int64_t)1 << 20 || L > (int64_t)1 << 28 || D > (int64_t)1 << 20) return TL_ERR_SHAPE;
  if (B * H * S * (D / 8) > (int64_t)1 << 40) return TL_ERR_SHAPE;
  if (!aligned16(cache_dev) || !aligned16(new_dev) || (reinterpret_cast<uintptr_t>(position_ids_dev) & 3u)) return TL_ERR_ALIGN;
  const tl_status st = check_device();
  if (st != TL_OK) return st;
  unsigned int* status = device_status_ptr();
  if (!status) return TL_ERR_CUDA;
  const cudaError_t e = launch_kv_append(cache_dev, new_dev, static_cast<const int*>(position_ids_dev), B, H, L, S, D,
                                         status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_e0m4_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!workspace_dev) return TL_ERR_NULL;
  if (!aligned16(workspace_dev)) return TL_ERR_ALIGN;
  if (workspace_bytes == 0) return TL_OK;
  const cudaError_t e =
      cudaMemsetAsync(workspace_dev, 0, workspace_bytes, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TL_OK : TL_ERR_CUDA;
}

tl_status tl_e0m4_device_status(void* stream) {
  unsigned int word = 0;
  if (read_decode_status(&word, static_cast<cudaStream_t>(stream)) != cudaSuccess) return TL_ERR_CUDA;
  return word == 0 ? TL_OK : static_cast<tl_status>(word);
}

uint64_t tl_e0m4_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

tl_status tl_e0m4_tuning_set(const char* key, int64_t value) {
  static const char* const names[kTuneCount] = {
      "ksplit", "tc_pair", "tc_big", "tc_mtiles", "list_pair", "batch_tc_min", "decode_split", "decode_slices",
      "decode_ctas_per_sm", "decode_rot_min", "wait_limit_cycles", "skip_copies", "register_max_m", "decode_cluster"};
  if (!key) {
    for (auto& v : g_tuning) v.store(-1, std::memory_order_relaxed);
    return TL_OK;
  }
  for (int k = 0; k < kTuneCount; ++k) {
    if (std::strcmp(key, names[k]) == 0) {
      g_tuning[k].store(value < 0 ? -1 : value, std::memory_order_relaxed);
      return TL_OK;
    }
  }
  return TL_ERR_KEY;
}

const char* tl_status_string(tl_status status) {
  switch (status) {
    case TL_OK: return "ok";
    case TL_ERR_NULL: return "null pointer";
    case TL_ERR_SHAPE: return "unsupported shape or group size";
    case TL_ERR_ALIGN: return "device pointer not 16-byte aligned";
    case TL_ERR_DTYPE: return "unknown dtype";
    case TL_ERR_WORKSPACE: return "workspace missing or too small";
    case TL_ERR_ARCH: return "device is not compute capability 10.x";
    case TL_ERR_CUDA: return "CUDA call or kernel launch failed";
    case TL_ERR_TIMEOUT: return "bounded device-side wait expired";
    case TL_ERR_LIMIT: return "problem exceeds the built-in scratch of the no-alloc entry point (M <= 16)";
    case TL_ERR_KEY: return "unknown tuning key";
  }
  return "unknown status";
}

}  // extern "C"
