// In-place KV-cache append (the paper's "KV cache copy optimization"): one cache tensor of the
// maximum sequence length is both input and output of the concatenation, and position_ids says
// where the new keys (or values) go, so nothing is copied but the new rows.
//
//   cache[b, h, pos[b] + s, :] = fresh[b, h, s, :]        cache [B, H, L, D], fresh [B, H, S, D], fp16
//
// One thread moves one 16-byte vector; consecutive threads move consecutive vectors of a row, and
// the rows of one (b, h) are contiguous on both sides, so reads and writes are fully coalesced.
// A batch entry whose rows would not fit (pos < 0 or pos + S > L) is skipped and the device status
// word is raised.  Pure data movement: HBM-bound, 4 bytes of traffic per element.
#include "common.cuh"
#include "ptx.cuh"

namespace tl {
namespace {

__global__ void __launch_bounds__(256)
kv_append_kernel(uint4* __restrict__ cache, const uint4* __restrict__ fresh, const int* __restrict__ pos, int H, int L,
                 int S, int vec_per_row, long long total, unsigned int* status) {
  // Programmatic dependent launch: the next kernel may begin its set-up now; the new rows (and the
  // positions) may be the previous kernel's output, so they are read after griddepcontrol.wait.
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();
  const long long per_b = (long long)H * S * vec_per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int b = (int)(i / per_b);
    const long long r = i - (long long)b * per_b;
    const int h = (int)(r / ((long long)S * vec_per_row));
    const long long in_head = r - (long long)h * S * vec_per_row;  // vector inside the S new rows of (b, h)
    const int p = pos[b];
    // S <= L is checked on the host, so L - S cannot wrap whatever the position holds
    if (p < 0 || p > L - S) {
      if (in_head == 0 && h == 0) atomicExch(status, (unsigned)TL_ERR_SHAPE);
      continue;
    }
    cache[(((long long)b * H + h) * L + p) * vec_per_row + in_head] = fresh[i];
  }
}

}  // namespace

cudaError_t launch_kv_append(void* cache, const void* fresh, const int* pos, int64_t B, int64_t H, int64_t L, int64_t S,
                             int64_t D, unsigned int* status, cudaStream_t stream) {
  const int vec_per_row = (int)(D / 8);
  const long long total = (long long)B * H * S * vec_per_row;
  // one vector per thread up to 2^22 blocks, a grid-stride loop beyond (the grid's x limit is 2^31 - 1)
  const long long blocks = (total + 255) / 256;
  const unsigned grid = (unsigned)(blocks < (1LL << 22) ? blocks : (1LL << 22));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kv_append_kernel, static_cast<uint4*>(cache),
                                           static_cast<const uint4*>(fresh), pos, (int)H, (int)L, (int)S, vec_per_row,
                                           total, status);
  count_launch();
  return e;
}

}  // namespace tl
