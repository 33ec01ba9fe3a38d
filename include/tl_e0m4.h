/*
 * tl_e0m4.h -- C ABI of the E0M4 weight-only FP4 matmul library for NVIDIA B200 (sm_100a).
 *
 * The operation is the one the Transformer-Lite paper states in Section 2.2 ("Operator
 * optimizations": half-precision activations times 4-bit group-wise quantized weights,
 * dequantized inside the matmul, with one implementation for prefill and one for decoding)
 * and Section 2.3 ("E0M4 FP4 quantization": the 4-bit code is the four highest fraction bits
 * of a weight that was mapped into one binade; dequantization is one shift and one OR).
 *
 * General rules for every entry point
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; pointers named *_host
 *     are HOST pointers.  The library allocates no device memory and frees none.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue
 *     work on that stream and return without synchronizing unless stated otherwise.
 *   - Argument errors are detected on the host and returned before anything is launched.
 *     Launch failures are returned as TL_ERR_CUDA.  No exception crosses this boundary.
 *   - Outputs are fully overwritten.  Weights must be finite.
 *   - Shapes: weights are logically W[K, N] (K = input features, N = output features);
 *     the quantization group is `group` consecutive k of one column n: 128 (the size Section
 *     3.1 uses), 64 or 32; every other value is TL_ERR_SHAPE.  K must be a multiple of 128 and
 *     N a multiple of 16 for every group size.  The same `group` must be given to the call
 *     that packs a tensor and to every call that reads it.
 *   - All device pointers must be 16-byte aligned.
 *
 * Packed layout (the paper prescribes none; this is the library's own rule)
 *   tile   : 16 columns x 128 rows (one group) of codes = 256 little-endian uint32 words.
 *   panel  : up to 8 neighbouring tiles (128 columns); panel p = n/128 holds
 *            R = min(8, N/16 - 8p) column blocks.  Panels follow each other; inside a panel the
 *            tiles are ordered group by group:  tile number = p*8*(K/128) + (k/128)*R + (n%128)/16.
 *   packed : K*N/2 bytes, tile after tile.  In a tile, column n%16 owns 16 consecutive words,
 *            word (k%128)/8 holds eight consecutive k, and the code of k%8 = c sits in nibble
 *            c/2 + 4*(c%2) of the word (nibble q = bits 4q..4q+3).
 *   scales : (K/group)*N uint32 words.  Group 128: 16 per tile in the same tile order
 *            (word = tile*16 + n%16).  Groups 64 and 32 keep the tile of 128 rows; a tile then
 *            owns 128/group runs of 16 words, one per group of its rows:
 *            word = (tile*(128/group) + (k%128)/group)*16 + n%16.
 *            Low half = fp16 dequantization scale d, high half = fp16 bias b.
 *   A weight is recovered as  w = (as_half(0x4000 | code << 6) - b) * d  (one fp16 rounding).
 */
#ifndef TL_E0M4_H_
#define TL_E0M4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TL_OK = 0,
  TL_ERR_NULL = 1,      /* a required pointer is NULL                          */
  TL_ERR_SHAPE = 2,     /* M, K, N or group violates the rules above           */
  TL_ERR_ALIGN = 3,     /* a device pointer is not 16-byte aligned             */
  TL_ERR_DTYPE = 4,     /* unknown tl_dtype                                    */
  TL_ERR_WORKSPACE = 5, /* workspace missing or smaller than required          */
  TL_ERR_ARCH = 6,      /* the current device is not compute capability 10.x   */
  TL_ERR_CUDA = 7,      /* a CUDA runtime/driver call or a launch failed       */
  TL_ERR_TIMEOUT = 8,   /* a bounded device-side wait gave up (see status word) */
  TL_ERR_LIMIT = 9,     /* tl_e0m4_matmul_noalloc: problem larger than its built-in scratch serves */
  TL_ERR_KEY = 10       /* tl_e0m4_tuning_set: unknown key                     */
} tl_status;

typedef enum { TL_F32 = 0, TL_F16 = 1 } tl_dtype;

/* Section 2.2 has one matmul implementation for the decoding stage (vector-matrix, bound by the
 * weight bytes) and one for prefill (matrix-matrix, bound by arithmetic).  The stage of a call is
 * set by M alone: decoding up to 16 tokens, prefill above. */
typedef enum { TL_STAGE_DECODE = 0, TL_STAGE_PREFILL = 1 } tl_stage;

/* The two kernels tl_e0m4_matmul dispatches to.  TL_KERNEL_REGISTER: the vector-matrix kernel that
 * builds the weights in registers (mma.sync fragments).  TL_KERNEL_TENSOR: the tcgen05 kernel with
 * the dequantized weights in tensor memory.  The cut between them lies inside the decoding stage
 * (measured: the register kernel wins up to 8 tokens). */
typedef enum { TL_KERNEL_REGISTER = 0, TL_KERNEL_TENSOR = 1 } tl_kernel;

/* Sizes in bytes of the `packed` and `scales` buffers for a [K, N] weight (host only, no
 * CUDA call).  Section 2.3: 4 bits per weight plus a scaling and a bias coefficient per
 * group.  Either output pointer may be NULL. */
tl_status tl_e0m4_packed_sizes(int64_t K, int64_t N, int group,
                               size_t* packed_bytes, size_t* scales_bytes);

/* Section 2.3 "Quantization".  w_dev: [K, N] row-major (n fastest), TL_F32 or TL_F16.
 * Per group of `group` k of one column: range widened to contain 0; d = range / (4 - 2^-9 - 2)
 * rounded to fp16 (stored); s = 1/d; bias = 2 + floor(-min * s * 8)/8 (stored, fp16);
 * w1 = clip(w*s + bias, 2, 4 - 2^-9) in fp32 (product and sum rounded separately);
 * code = min(y1 + y2, 15) with y1 the four highest and y2 the fifth fraction bit of w1.
 * Writes packed_dev and scales_dev in the layout above. */
tl_status tl_e0m4_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group,
                           void* packed_dev, void* scales_dev, void* stream);

/* The comparison format of Section 3.4 (Tables 1 and 2): group-wise asymmetric INT4 with an
 * integer zero point, written into the SAME packed container, so that tl_e0m4_dequant and
 * every tl_e0m4_matmul* entry point serve it unchanged.  The paper names the format and gives
 * no formulas; this is the usual min-max one.  Per group of `group` k of one column:
 * step = (max - min) / 15 rounded to fp16 (at most 8188); s = 1/step; zero point
 * z = clamp(rint(-min * s), 0, 15); code = clamp(rint(w * s) + z, 0, 15) in fp32, ties to even.
 * Stored: d = 8 * step (exact in fp16) and b = as_half(0x4000 | z << 6), for which the E0M4
 * dequantization (w1 - b) * d equals (code - z) * step exactly.  Same arguments, layout and
 * errors as tl_e0m4_quantize. */
tl_status tl_int4_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group,
                           void* packed_dev, void* scales_dev, void* stream);

/* Section 2.2 "Operator optimizations": the small operators that make up rms-norm, fused into
 * one kernel, with the residual add that precedes the norm in a transformer block folded in.
 *   s = x (residual_dev == NULL)  or  s = fp16(x + residual);
 *   y[m, k] = s[m, k] * rsqrt(mean_k(s[m, :]^2) + eps) * gamma[k]      (fp32 arithmetic, fp16 out)
 * x_dev, residual_dev, y_dev, sum_out_dev: fp16 [M, K] row-major; gamma_dev: fp16 [K].
 * sum_out_dev (may be NULL; needs a residual) receives s; it may be x_dev or residual_dev, and
 * y_dev may be x_dev when no residual is given (every element is read before it is written by
 * the same thread).  K % 8 == 0, K <= 32768, eps >= 0, pointers 16-byte aligned; errors are
 * returned before the launch.  The paper names the operator and gives no formula: this is the
 * rms-norm of the models it runs. */
tl_status tl_rmsnorm(const void* x_dev, const void* residual_dev, const void* gamma_dev, void* sum_out_dev,
                     void* y_dev, int64_t M, int64_t K, float eps, void* stream);

/* Section 2.2 "operator fusions", the other norm the paper names: layer-norm over the last axis,
 *   y[m, k] = (s[m, k] - mean_k s[m, :]) / sqrt(var_k s[m, :] + eps) * gamma[k] + beta[k]
 * with the biased variance (sum of squared deviations / K), fp32 arithmetic, one fp16 rounding.
 * beta_dev: fp16 [K].  Residual, sum_out, aliasing, limits and errors exactly as tl_rmsnorm. */
tl_status tl_layernorm(const void* x_dev, const void* residual_dev, const void* gamma_dev, const void* beta_dev,
                       void* sum_out_dev, void* y_dev, int64_t M, int64_t K, float eps, void* stream);

/* "KV cache copy optimization" (the paper's second Section 2.3): the in-place operator that
 * replaces the concatenation of cached and new keys (or values).  One tensor of the maximum
 * sequence length is input and output; position_ids gives, per batch entry, the row at which the
 * new rows are written:
 *   cache[b, h, position_ids[b] + s, :] = new[b, h, s, :]     for s < S
 * cache_dev: fp16 [B, H, L, D] row-major; new_dev: fp16 [B, H, S, D]; position_ids_dev: int32 [B]
 * (device).  D % 8 == 0, S <= L, tensors 16-byte aligned.  A batch entry whose rows would not fit
 * (position < 0 or position + S > L) is left untouched and raises the device status word
 * (tl_e0m4_device_status returns TL_ERR_SHAPE).  Nothing else of the cache is read or written. */
tl_status tl_kv_append(void* cache_dev, const void* new_dev, const void* position_ids_dev, int64_t B, int64_t H,
                       int64_t L, int64_t S, int64_t D, void* stream);

/* Section 2.3 "Dequantization": w1 = as_half(EXP | (code << 6)), then (w1 - b) * d.
 * w_f16_dev: [K, N] row-major fp16, fully overwritten. */
tl_status tl_e0m4_dequant(const void* packed_dev, const void* scales_dev, int64_t K, int64_t N,
                          int group, void* w_f16_dev, void* stream);

/* Which of Section 2.2's two stages a call with M tokens belongs to (host only, no CUDA call). */
tl_stage tl_e0m4_matmul_stage(int64_t M);

/* Which kernel tl_e0m4_matmul really launches for this shape (host only, no CUDA call). */
tl_kernel tl_e0m4_matmul_kernel(int64_t M, int64_t K, int64_t N);

/* Bytes of device scratch tl_e0m4_matmul needs for this shape (0 = none).  Host only. */
size_t tl_e0m4_matmul_workspace(int64_t M, int64_t K, int64_t N);

/* Zero-fills a matmul workspace on `stream` (a cudaMemsetAsync).  A workspace must be zeroed
 * once before its first use; every tl_e0m4_matmul call that returns TL_OK and runs to
 * completion leaves it zeroed again, so one buffer can serve any sequence of calls that are
 * ordered on one stream.  Calls that may run concurrently need separate workspaces. */
tl_status tl_e0m4_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream);

/* Section 2.2: y[M, N] = x[M, K] . W[K, N] with W given in packed E0M4 form and
 * dequantized inside the kernel; fp16 in, fp32 accumulation, fp16 out.
 * x_dev: [M, K] row-major fp16.  y_dev: [M, N] row-major fp16.  M >= 1.
 * workspace_dev / workspace_bytes: scratch of at least tl_e0m4_matmul_workspace(M, K, N)
 * bytes (may be NULL when that is 0), zeroed as tl_e0m4_workspace_init describes; the decode
 * kernels keep split-K partial sums and tile counters there and return it zeroed.
 * The matmul kernels use programmatic dependent launch: a call begins fetching `packed_dev` and
 * `scales_dev` as soon as the kernels before it on the stream let their successors start, which
 * every kernel of this library does at its very beginning.  So the weights of a call must be
 * complete before the kernel that precedes the call on the stream STARTS: weights written by the
 * kernels enqueued directly before it (a tl_e0m4_quantize, a copy kernel, another matmul) need an
 * event, a synchronization or any operation that is not a kernel of this library in between.
 * Weights are static in inference, which is what this rule relies on; x_dev, y_dev, the addend and
 * the workspace are ordered as usual. */
tl_status tl_e0m4_matmul(const void* x_dev, const void* packed_dev, const void* scales_dev,
                         void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                         void* workspace_dev, size_t workspace_bytes, void* stream);

/* Section 2.2 "operator fusions" (an element-wise operator fused with the operator before it):
 * the matmul with the residual add that follows it in a transformer block,
 *   y[m, n] = fp16( sum_k x[m, k] * W[k, n]  +  addend[m, n] ),
 * the sum in fp32, rounded once.  addend_dev: fp16 [M, N] row-major, 16-byte aligned; it may be
 * y_dev (every element is read before it is written).  Everything else as tl_e0m4_matmul. */
tl_status tl_e0m4_matmul_add(const void* x_dev, const void* packed_dev, const void* scales_dev,
                             const void* addend_dev, void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                             void* workspace_dev, size_t workspace_bytes, void* stream);

/* The same fusion with a bias row (the q/k/v projections of several of the paper's models carry
 * one): y[m, n] = fp16( sum_k x[m, k] W[k, n] + bias[n] ), the sum in fp32, rounded once.
 * bias_dev: fp16 [N], 16-byte aligned.  Everything else as tl_e0m4_matmul_add. */
tl_status tl_e0m4_matmul_bias(const void* x_dev, const void* packed_dev, const void* scales_dev,
                              const void* bias_dev, void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                              void* workspace_dev, size_t workspace_bytes, void* stream);

/* Section 2.2 "operator fusions": the joined gate and up projections of a gated MLP with the
 * activation fused in.  W[K, N] holds gate and up columns interleaved in blocks of eight
 * (columns 16 j .. 16 j + 7 gate, 16 j + 8 .. 16 j + 15 the matching up columns; the caller
 * permutes the columns before tl_e0m4_quantize), Y = x . W stays in fp32 and
 *   y[m, 8 j + c] = fp16( silu(Y[m, 16 j + c]) * Y[m, 16 j + 8 + c] ),  silu(g) = g / (1 + exp(-g)).
 * y_dev: fp16 [M, N / 2] row-major.  Everything else as tl_e0m4_matmul (workspace included). */
tl_status tl_e0m4_matmul_swiglu(const void* x_dev, const void* packed_dev, const void* scales_dev,
                                void* y_dev, int64_t M, int64_t K, int64_t N, int group,
                                void* workspace_dev, size_t workspace_bytes, void* stream);

/* One problem of a batch: the arguments of tl_e0m4_matmul that differ between problems. */
typedef struct tl_e0m4_problem {
  const void* x_dev;      /* fp16 [M, K] row-major */
  const void* packed_dev; /* packed codes of W[K, N] */
  const void* scales_dev; /* scale words of W[K, N] */
  void* y_dev;            /* fp16 [M, N] row-major, fully overwritten */
  int64_t K;
  int64_t N;
} tl_e0m4_problem;

/* Bytes of device scratch tl_e0m4_matmul_batch needs (a constant, about 9.7 MB).  Host only. */
size_t tl_e0m4_matmul_batch_workspace(void);

/* Section 2.2, decoding stage and batched decoding: the same product for `count` INDEPENDENT
 * problems that share M (1 <= M <= 128; larger M is TL_ERR_SHAPE), e.g. the q/k/v projections of
 * one layer, gate and up, or a whole stack of layers whose inputs are all known.  All problems run
 * in one persistent kernel that streams their packed weights back to back (longer lists than 192
 * take one launch per 192): the register-fragment vector-matrix kernel up to 8 tokens, the
 * tensor-core kernel from 9 tokens on.  problems_host: HOST array of `count` descriptors; it is
 * read during the call only.  No problem may read what another problem of the same batch writes
 * (no y_dev may alias an x_dev or another y_dev).  The workspace follows the rules of
 * tl_e0m4_workspace_init; panels cut between two CTAs meet in fp32 atomics, so two runs may
 * differ in the last fp16 bit. */
tl_status tl_e0m4_matmul_batch(const tl_e0m4_problem* problems_host, int count, int64_t M, int group,
                               void* workspace_dev, size_t workspace_bytes, void* stream);

/* The batch for callers whose activations live in host memory.  The problems' x_dev / y_dev
 * must point into two device staging ranges [x_stage_dev, +x_bytes) and [y_stage_dev, +y_bytes).
 * Enqueues on `stream`: one copy x_host -> x_stage_dev (x_bytes), tl_e0m4_matmul_batch, one copy
 * y_stage_dev -> y_host (y_bytes).  x_host / y_host should be pinned; the result is valid once
 * the stream has been synchronized. */
tl_status tl_e0m4_matmul_batch_host(const tl_e0m4_problem* problems_host, int count, int64_t M,
                                    int group, const void* x_host, void* x_stage_dev, size_t x_bytes,
                                    void* y_host, const void* y_stage_dev, size_t y_bytes,
                                    void* workspace_dev, size_t workspace_bytes, void* stream);

/* One step of a decode chain: a matmul of tl_e0m4_matmul with the element-wise operators around it
 * fused in (Section 2.2, operator fusions), as one descriptor. */
typedef enum {
  TL_EPILOGUE_NONE = 0,   /* y[M, N] = Y                                                     */
  TL_EPILOGUE_ADD = 1,    /* y[M, N] = Y + addend[M, N]   (addend_dev may be y_dev)          */
  TL_EPILOGUE_BIAS = 2,   /* y[M, N] = Y + bias[N]                                            */
  TL_EPILOGUE_SWIGLU = 3  /* y[M, N / 2] = silu(gate) * up over column blocks of eight of Y,
                             as tl_e0m4_matmul_swiglu                                        */
} tl_epilogue;

typedef struct tl_e0m4_step {
  const void* x_dev;       /* fp16 [M, K] row-major */
  const void* packed_dev;  /* packed codes of W[K, N] */
  const void* scales_dev;  /* scale words of W[K, N] */
  void* y_dev;             /* fp16 [M, N] ([M, N / 2] with TL_EPILOGUE_SWIGLU), fully overwritten */
  const void* addend_dev;  /* fp16 [M, N] (ADD) or [N] (BIAS), else NULL */
  int64_t K;
  int64_t N;
  int32_t epilogue;        /* a tl_epilogue */
  int32_t after_previous;  /* non-zero: this step reads (x_dev, addend_dev) or overwrites what an EARLIER step of
                              the list writes, so it begins only when all earlier steps are complete;
                              zero: it is independent of every step since the last such barrier */
  int32_t rms_scale;       /* non-zero: Y is x . W with every row multiplied by 1 / sqrt(mean_k x[m, k]^2 + rms_eps):
                              the rms-norm that precedes the matmul, its gain folded into W by the caller
                              (quantize diag(gamma) . W) */
  float rms_eps;
} tl_e0m4_step;

/* Bytes of device scratch tl_e0m4_matmul_chain needs (a constant, about 2.7 MB).  Host only. */
size_t tl_e0m4_matmul_chain_workspace(void);

/* Section 2.2, the decoding stage as a model runs it: a sequence of matmuls in which one consumes
 * what another produces (norm -> qkv + bias -> ... -> o + residual -> norm -> gate_up + SwiGLU ->
 * down + residual, layer after layer).  Y = x . W (fp32 accumulation), optionally scaled per row
 * (rms_scale), then the epilogue, rounded once to fp16.  1 <= M <= 8 (TL_ERR_SHAPE above; batches
 * of more tokens take one tl_e0m4_matmul call per step).
 * All steps run in ONE persistent kernel per 128 steps.  Steps are processed in list order by all
 * CTAs together; where a step has after_previous set, the kernel waits (on the device, per CTA,
 * only for the activations: the packed weights of later steps keep streaming into shared memory
 * meanwhile) until every earlier step is complete.  Steps without it run as the problems of
 * tl_e0m4_matmul_batch do and must be independent of the steps since the last barrier.
 * steps_host: HOST array, read during the call only.  Weights must be complete before the kernel
 * preceding this call on the stream starts (see tl_e0m4_matmul).  The workspace
 * (tl_e0m4_matmul_chain_workspace() bytes) follows the rules of tl_e0m4_workspace_init.
 * The kernel's CTAs wait for one another, so all of them must be resident at once: the launch is
 * sized to fit an otherwise idle GPU, and a call should not share the GPU with another long-running
 * kernel (every wait is bounded: if the grid cannot become resident within about two seconds the
 * call ends with TL_ERR_TIMEOUT in the status word instead of hanging). */
tl_status tl_e0m4_matmul_chain(const tl_e0m4_step* steps_host, int count, int64_t M, int group,
                               void* workspace_dev, size_t workspace_bytes, void* stream);

/* (No counterpart in the paper: this entry point exists for deployment reasons only.)
 * The decoding product of tl_e0m4_matmul for callers that cannot obtain device memory at the
 * time of the call and therefore have no workspace to pass: code running between the
 * reservation of a fixed memory budget and its release (an inference server that hands its
 * whole device pool to a framework allocator at start-up), code on a latency-critical path
 * where cudaMalloc's implicit device synchronization is not acceptable, and plug-ins that are
 * forbidden to allocate by their host.  The scratch that tl_e0m4_matmul takes from the caller
 * lives here in an array inside the library image instead: tl_e0m4_matmul_noalloc_scratch_bytes()
 * bytes (about 2.6 MB), held by every GPU that has loaded the library until the process exits.
 * The call itself allocates and frees nothing.
 * Limits: 1 <= M <= 16 (more tokens than the array has room for per output column are refused
 * with TL_ERR_LIMIT; use tl_e0m4_matmul with a workspace for those); K, N, alignment and `group`
 * as for tl_e0m4_matmul.  The arguments are those of tl_e0m4_matmul; the result agrees with
 * tl_e0m4_matmul's within the library's matmul tolerance, not bit for bit (from 9 tokens on the
 * two entry points run different kernels, and cut panels meet in atomics in either).
 * The first call on each device looks up the array's device address (the device must be
 * current); make that first call outside any stream capture.  Every call clears the array on
 * `stream` before it launches, because the array keeps whatever the previous call left behind.
 * All calls on a device share the one array: calls that can overlap on the GPU (different
 * streams without an ordering between them) race on it and must not be issued. */
tl_status tl_e0m4_matmul_noalloc(const void* x_dev, const void* packed_dev, const void* scales_dev,
                                 void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* stream);

/* Size in bytes of the array tl_e0m4_matmul_noalloc keeps inside the library.  Host only. */
size_t tl_e0m4_matmul_noalloc_scratch_bytes(void);

/* Bytes of device staging tl_e0m4_matmul_host needs: room for x and y plus the matmul
 * workspace, each rounded up to 256 bytes.  Host only. */
size_t tl_e0m4_matmul_host_staging(int64_t M, int64_t K, int64_t N);

/* The same product for callers whose activations live in host memory: copies x_host
 * (fp16 [M, K], ideally pinned) to the device staging buffer, runs tl_e0m4_matmul and copies
 * y (fp16 [M, N]) back to y_host, all on `stream`; the result is valid once the stream has
 * been synchronized.  Weights stay on the device.  staging_dev must hold at least
 * tl_e0m4_matmul_host_staging(M, K, N) bytes; its workspace part (the last
 * tl_e0m4_matmul_workspace bytes, rounded up to 256) must be zeroed once, which
 * tl_e0m4_workspace_init on the whole staging buffer does. */
tl_status tl_e0m4_matmul_host(const void* x_host, const void* packed_dev, const void* scales_dev,
                              void* y_host, int64_t M, int64_t K, int64_t N, int group,
                              void* staging_dev, size_t staging_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * E0M8: the construction of Section 2.3 with eight fraction bits kept (the section notes that the
 * method carries over to other bit widths).  A code is the eight highest fraction bits of w1 in
 * [2, 4): as_half(0x4000 | code << 2) = 2 + code / 128, 256 grid points.  The steps are those of
 * tl_e0m4_quantize with 128 for 8, 255 for 15 and "eight highest / ninth" for "four highest /
 * fifth": d = range / (4 - 2^-9 - 2) rounded to fp16; s = 1 / d; bias = 2 + floor(-min * s * 128) / 128;
 * w1 = clip(w * s + bias, 2, 4 - 2^-9); code = min(y1 + y2, 255); dequantization (w1 - b) * d
 * rounded once to fp16.
 * Container: the 4-bit layout's tiles (16 columns x 128 rows) in the same order, one byte per
 * code: packed_dev holds K * N bytes, tile t at byte 2048 * t, made of eight chunks of 256 bytes
 * (one per 16 rows); in a chunk column n % 16 owns 16 consecutive bytes and byte k % 16 is the code
 * of row k: byte 2048 t + 256 ((k % 128) / 16) + 16 (n % 16) + k % 16.  scales_dev is laid out as
 * for E0M4.
 * group must be 128 (TL_ERR_SHAPE otherwise); other arguments, ownership, alignment rules and
 * errors are those of the E0M4 entry points of the same name.
 * tl_e0m8_matmul runs every M on the tensor-core kernel; its workspace
 * (tl_e0m8_matmul_workspace(M, K, N) bytes, possibly 0) is zero on entry and left zero. */
tl_status tl_e0m8_packed_sizes(int64_t K, int64_t N, int group, size_t* packed_bytes, size_t* scales_bytes);
tl_status tl_e0m8_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group, void* packed_dev,
                           void* scales_dev, void* stream);
tl_status tl_e0m8_dequant(const void* packed_dev, const void* scales_dev, int64_t K, int64_t N, int group,
                          void* w_f16_dev, void* stream);
size_t tl_e0m8_matmul_workspace(int64_t M, int64_t K, int64_t N);
tl_status tl_e0m8_matmul(const void* x_dev, const void* packed_dev, const void* scales_dev, void* y_dev, int64_t M,
                         int64_t K, int64_t N, int group, void* workspace_dev, size_t workspace_bytes, void* stream);
/* The fused forms of Section 2.2 for E0M8 weights: residual add, bias row and SwiGLU, with the
 * meaning, layouts and rules of tl_e0m4_matmul_add, tl_e0m4_matmul_bias and tl_e0m4_matmul_swiglu. */
tl_status tl_e0m8_matmul_add(const void* x_dev, const void* packed_dev, const void* scales_dev, const void* addend_dev,
                             void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                             size_t workspace_bytes, void* stream);
tl_status tl_e0m8_matmul_bias(const void* x_dev, const void* packed_dev, const void* scales_dev, const void* bias_dev,
                              void* y_dev, int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                              size_t workspace_bytes, void* stream);
tl_status tl_e0m8_matmul_swiglu(const void* x_dev, const void* packed_dev, const void* scales_dev, void* y_dev,
                                int64_t M, int64_t K, int64_t N, int group, void* workspace_dev,
                                size_t workspace_bytes, void* stream);
/* A list of independent E0M8 problems that share M (1 <= M <= 128), as tl_e0m4_matmul_batch: one
 * persistent tensor-core kernel per 22 problems walks the 128-k rounds of all of them.  The workspace
 * is that of tl_e0m4_matmul_batch (tl_e0m4_matmul_batch_workspace() bytes, zero on entry, left zero). */
tl_status tl_e0m8_matmul_batch(const tl_e0m4_problem* problems_host, int count, int64_t M, int group,
                               void* workspace_dev, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * E0M3 and E0M5: the construction of Section 2.3 with three or five fraction bits kept ("other
 * bit-width quantization").  `bits` is 3 or 5 (TL_ERR_SHAPE otherwise; 4 and 8 have the entry points
 * above).  A code is the `bits` highest fraction bits of w1 in [2, 4):
 * as_half(0x4000 | code << (10 - bits)) = 2 + code / 2^(bits - 1); the steps are those of
 * tl_e0m4_quantize with 2^bits for 16, 2^bits - 1 for 15 and 2^(bits - 1) for 8.
 * Container: the 4-bit layout's tiles (16 columns x 128 rows) in the same order; eight consecutive k
 * of one column are a unit of `bits` bytes, a little-endian integer in which the code of k % 8 = c
 * occupies bits c * bits .. (c + 1) * bits - 1, and column n % 16 of a tile owns its 16 units one
 * after the other: byte 256 * bits * tile + 16 * bits * (n % 16) + bits * ((k % 128) / 8) is the
 * first byte of the unit of row k.  packed_dev holds K * N * bits / 8 bytes; scales_dev is laid
 * out as for E0M4.  group must be 128.  Other arguments, ownership, alignment rules and errors
 * are those of the E0M4 entry points of the same name.  tl_e0mx_matmul runs every M on the
 * tensor-core kernel (plain product; its workspace, tl_e0mx_matmul_workspace(M, K, N, bits) bytes,
 * possibly 0, is zero on entry and left zero). */
tl_status tl_e0mx_packed_sizes(int64_t K, int64_t N, int group, int bits, size_t* packed_bytes, size_t* scales_bytes);
tl_status tl_e0mx_quantize(const void* w_dev, tl_dtype w_dtype, int64_t K, int64_t N, int group, int bits,
                           void* packed_dev, void* scales_dev, void* stream);
tl_status tl_e0mx_dequant(const void* packed_dev, const void* scales_dev, int64_t K, int64_t N, int group, int bits,
                          void* w_f16_dev, void* stream);
size_t tl_e0mx_matmul_workspace(int64_t M, int64_t K, int64_t N, int bits);
tl_status tl_e0mx_matmul(const void* x_dev, const void* packed_dev, const void* scales_dev, void* y_dev, int64_t M,
                         int64_t K, int64_t N, int group, int bits, void* workspace_dev, size_t workspace_bytes,
                         void* stream);

/* Reads the device status word that kernels set when a bounded device-side wait gives up
 * (TL_ERR_TIMEOUT), clears it, and returns it.  Synchronizes `stream`.  Diagnostics only. */
tl_status tl_e0m4_device_status(void* stream);

/* Number of kernels this library has launched in this process so far (all entry points). */
uint64_t tl_e0m4_launch_count(void);

/* Diagnostics and tests (no counterpart in the paper): overrides one launch heuristic for the whole
 * process until it is set back.  value < 0 restores the library's own choice; key == NULL restores
 * all of them.  The overrides are read at every call (sizing calls included), never from the
 * environment.  Keys: "ksplit" (1..8 CTAs share a tile along K in the tensor-core kernel),
 * "tc_pair" (0 / 1: pairs of CTAs), "tc_big" (0: rounds of 64 k), "tc_mtiles" (1, 2, 4, 8 times the
 * fewest token tiles), "list_pair" (0 / 1), "batch_tc_min" (first token count of a list that takes
 * the tensor-core kernel), "register_max_m" (most tokens of a single call on the register kernel,
 * 1..16), "decode_split" (1 whole panels per CTA, 2 stream-K ranges), "decode_slices" (CTAs per
 * panel), "decode_ctas_per_sm" (1, 2), "decode_rot_min", "decode_cluster" (0: CTAs that share a panel add
 * their sums up in the global scratch instead of a cluster's shared memory), "wait_limit_cycles" (SM cycles after
 * which a device-side wait gives up and raises TL_ERR_TIMEOUT in the status word; about two seconds
 * by default), "skip_copies" (1: the producers of the matmul kernels issue no copies, so that with
 * a short wait limit every wait runs out while nothing is in flight: the safe way to see the
 * time-out path work).  Unknown key: TL_ERR_KEY. */
tl_status tl_e0m4_tuning_set(const char* key, int64_t value);

/* Static, human-readable name of a status code. */
const char* tl_status_string(tl_status status);

#ifdef __cplusplus
}
#endif

#endif /* TL_E0M4_H_ */
