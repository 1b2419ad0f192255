/*
 * litevggt.h - C ABI of the B200 (sm_100a) library for geometry-aware cached token
 * merging around VGGT's frame-global attention layer (LiteVGGT, Sec. 3.4 of the paper).
 *
 * Path (one global layer):
 *   grad map (once per sequence) -> merge plan [var map + norms -> GA map -> partition
 *   -> cosine match + row argmax -> select -> index build] -> merge -> global
 *   attention over the merged tokens -> unmerge.  The plan is the cached index set that
 *   is reused by the following global layers and refreshed every k-th layer.
 *
 * Conventions
 *   - F frames, patch grid gh x gw, P = gh*gw patch tokens + S special tokens per frame
 *     (Sec. 3.1: 1 camera + 4 register), T = P + S, N = F*T tokens, D channels.
 *   - token index i = f*T + t; t < S special, t = S + py*gw + px patch (row-major grid).
 *   - "dev" pointers are device memory on the ctx's device, "host" pointers are host
 *     memory.  All tensors are row-major, contiguous and 16-byte aligned
 *     (LITEVGGT_ERR_ALIGN otherwise).  bf16 tensors are passed as void*.
 *   - The caller owns every tensor and the stream.  The library owns the ctx workspace
 *     (allocated once in litevggt_create, sized for the config) and the plan arrays.
 *   - Every call validates its arguments and returns a status; nothing throws or
 *     aborts.  Compute calls enqueue work on `stream` (a cudaStream_t passed as void*)
 *     and return without synchronising, unless stated otherwise.
 *   - Device-side pipeline waits are bounded; a kernel that gives up records it in the
 *     ctx's device status word, which litevggt_poll_device_status reads.
 *   - There is no CPU or non-sm_100 fallback: LITEVGGT_ERR_ARCH on other devices.
 */
#ifndef LITEVGGT_H_
#define LITEVGGT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LITEVGGT_OK = 0,
  LITEVGGT_ERR_NULL = 1,           /* a required pointer is NULL */
  LITEVGGT_ERR_BAD_CONFIG = 2,     /* config field out of range / unsupported */
  LITEVGGT_ERR_SHAPE = 3,          /* a size argument disagrees with the config */
  LITEVGGT_ERR_ALIGN = 4,          /* a tensor is not 16-byte aligned */
  LITEVGGT_ERR_ALLOC = 5,          /* device or host allocation failed */
  LITEVGGT_ERR_CUDA = 6,           /* a CUDA runtime/driver call failed */
  LITEVGGT_ERR_ARCH = 7,           /* device is not compute capability 10.x */
  LITEVGGT_ERR_STALE_PLAN = 8,     /* plan belongs to another ctx, or was never built */
  LITEVGGT_ERR_DEVICE_TIMEOUT = 9, /* a kernel gave up on a bounded wait */
  LITEVGGT_ERR_DEVICE_BOUNDS = 10  /* a kernel met an out-of-range index and skipped it */
} litevggt_status;

/* Token classes written by the partition (Sec. 3.4, "GA Token Partitioning"). */
enum {
  LITEVGGT_CLS_PROTECTED = 0, /* special tokens: never merged, never anchors */
  LITEVGGT_CLS_GA = 1,        /* top geometric-importance tokens: excluded from merging */
  LITEVGGT_CLS_DST = 2,       /* anchors */
  LITEVGGT_CLS_SRC = 3        /* merge candidates */
};

typedef struct {
  int32_t frames;             /* F >= 1 */
  int32_t grid_h, grid_w;     /* patch grid; image is (14*grid_h) x (14*grid_w) pixels; grid_w <= 64 */
  int32_t patch_px;           /* 14; at most 30 */
  int32_t n_special;          /* 5 (1 camera + 4 register tokens, ahead of the patches) */
  int32_t dim;                /* 1024 */
  int32_t heads;              /* 16 (head dim must be 64) */
  float merge_ratio;          /* r in [0,1]: R = min(|Src|, floor(r*N)) src tokens are merged
                                 away, most similar first.  r >= |Src|/N is the paper's
                                 rule (every src token is merged); r = 0 is the identity. */
  float ga_keep_frac;         /* 0.10: fraction of patches per frame kept as GA tokens */
  float alpha, beta;          /* 0.5, 0.5: weights of norm(Grad map), norm(Var map) */
  int32_t cell_h, cell_w;     /* 2, 2: one anchor per cell in frames 1..F-1 */
  int32_t var_window;         /* 3: window of the Var map */
  int32_t recompute_interval; /* 6: refresh the plan every this many global layers */
  int32_t qkv_dtype;          /* 0 = bf16; 1 = E4M3: litevggt_global_attn / _ext quantise the projected Q, K, V head
                                 by head (scale = amax / 448 of the head, taken from the tensor itself) and
                                 run both attention products on 8-bit operands, the probabilities rounded to
                                 E4M3 as well (Sec. 3.5 and supplementary "FP8 Quantization Details").  The
                                 projections, merge and unmerge stay bf16. */
} litevggt_config;

typedef struct litevggt_ctx litevggt_ctx;   /* workspace, tensor maps, device status word */
typedef struct litevggt_plan litevggt_plan; /* the cached merge indices */

/* Fill `cfg` with the paper's defaults for the given sequence shape. */
litevggt_status litevggt_default_config(int32_t frames, int32_t grid_h, int32_t grid_w,
                                        float merge_ratio, litevggt_config* cfg);

/* Create a context on `device`: validates the config, allocates the workspace, builds
 * the tensor maps.  Synchronous.  *out is NULL on failure. */
litevggt_status litevggt_create(const litevggt_config* cfg, int device, litevggt_ctx** out);
litevggt_status litevggt_destroy(litevggt_ctx* ctx);

/* Sizes that follow from the config (host arithmetic only; any output may be NULL):
 * N tokens, M merged rows, |Src|, |Dst|, bytes of device workspace held by the ctx. */
litevggt_status litevggt_sizes(const litevggt_ctx* ctx, int64_t* n_tokens, int64_t* n_merged,
                               int64_t* n_src, int64_t* n_dst, size_t* workspace_bytes);

/* Grad map (Sec. 3.4, "Pixel Gradient"): Sobel on the channel-mean intensity with
 * replicate padding, magnitude, mean over each patch.
 * images: dev fp32 [F,3,14*gh,14*gw] in [0,1];  grad: dev fp32 [F,gh,gw] (written). */
litevggt_status litevggt_grad_map(litevggt_ctx* ctx, const float* images, float* grad, void* stream);

/* Merge plan (Sec. 3.4): Var map of x (3x3 clipped window, population variance per
 * channel, mean over channels), GA map = alpha*norm(grad)+beta*norm(var) with per-frame
 * min-max normalisation, partition into GA/dst/src tokens, cosine matching of every
 * src token against all anchors of all frames (row argmax, ties to the lowest anchor),
 * selection of the R most similar src tokens and the index arrays.
 * x: dev bf16 [N,D] (read);  grad: dev fp32 [F,gh,gw] (read).
 * *plan_inout == NULL: a plan is created; otherwise it is refreshed in place. */
litevggt_status litevggt_merge_plan(litevggt_ctx* ctx, const void* x, const float* grad,
                                    litevggt_plan** plan_inout, void* stream);

/* Same as litevggt_merge_plan from the matching step onwards, with the partition given
 * by the caller (cls: dev uint8 [N], LITEVGGT_CLS_* values with exactly the per-frame
 * class counts the config implies; LITEVGGT_ERR_DEVICE_BOUNDS is flagged otherwise).
 * Used for stage-isolated tests and for other anchor rules. */
litevggt_status litevggt_merge_plan_with_partition(litevggt_ctx* ctx, const void* x,
                                                   const uint8_t* cls, litevggt_plan** plan_inout,
                                                   void* stream);

/* Merge (Sec. 3.4, merge equation): x'_d = (x_d + sum_{s in S_d} x_s) / (1 + |S_d|),
 * fp32 accumulation in ascending token order, one rounding to bf16; rows that absorb
 * nothing are copied bit-exactly.  x: dev bf16 [N,D];  x_merged: dev bf16 [M,D]. */
litevggt_status litevggt_merge(litevggt_ctx* ctx, const litevggt_plan* plan, const void* x,
                               void* x_merged, void* stream);

/* Global self-attention over the merged sequence (Sec. 3.1): qkv = x' W_qkv^T + b_qkv,
 * per head softmax(Q K^T / sqrt(64)) V (non-causal), y' = o W_o^T + b_o.
 * x_merged: dev bf16 [m,D]; m must equal M.  w_qkv: dev bf16 [3D,D], rows [0,D) Q,
 * [D,2D) K, [2D,3D) V, head h = channels [64h,64h+64);  b_qkv: dev bf16 [3D] or NULL;
 * w_o: dev bf16 [D,D] (output-feature-major);  b_o: dev bf16 [D] or NULL;
 * y_merged: dev bf16 [m,D] (written). */
litevggt_status litevggt_global_attn(litevggt_ctx* ctx, const void* x_merged, int64_t m,
                                     const void* w_qkv, const void* b_qkv, const void* w_o,
                                     const void* b_o, void* y_merged, void* stream);

/* Options of litevggt_global_attn_ext.  The paper prints neither; VGGT's attention layer, which
 * the method keeps (Sec. 3.1), normalises queries and keys per head and rotates them by their 2-D
 * position, so weights trained that way need both. */
typedef struct litevggt_attn_ext {
  /* Per-head LayerNorm of Q and K over the 64 channels of a head (population variance):
   * dev bf16 [64] each, 16-byte aligned; all four NULL = no normalisation, otherwise all four. */
  const void* q_norm_gamma;
  const void* q_norm_beta;
  const void* k_norm_gamma;
  const void* k_norm_beta;
  float norm_eps;   /* > 0 when the normalisation is on (VGGT: 1e-5) */
  /* 2-D rotary embedding of Q and K, after the normalisation: non-zero = on.  A head's channels
   * [0,32) turn with the row position, [32,64) with the column position; inside a half, channel i
   * (< 16) and channel i+16 form a plane rotated by position * rope_base^(-i/16).  Row r of the
   * merged sequence has the position of the token that owns it (the plan's kept token): special
   * tokens (0,0), the patch at grid row py, column px (py+1, px+1). */
  int32_t rope;
  float rope_base;  /* > 1 when the rotation is on (VGGT: 100) */
} litevggt_attn_ext;

/* litevggt_global_attn with the options above applied to the projected Q and K before the scores
 * (normalisation first, then rotation), fp32 arithmetic, one rounding back to bf16.  plan: the plan
 * the merged rows came from (read for the rows' positions; may be NULL when ext->rope == 0).
 * Everything else as in litevggt_global_attn.  A LayerScale factor on the layer's output needs no
 * option: scale the rows of w_o and the entries of b_o by it. */
litevggt_status litevggt_global_attn_ext(litevggt_ctx* ctx, const litevggt_plan* plan,
                                         const void* x_merged, int64_t m, const void* w_qkv,
                                         const void* b_qkv, const void* w_o, const void* b_o,
                                         const litevggt_attn_ext* ext, void* y_merged, void* stream);

/* The same attention layer as litevggt_global_attn for callers that must not allocate (the paper
 * has no counterpart; this is a property of the library, not of the method).  It needs no
 * context: a context's workspace comes from cudaMalloc, which is off limits for code running
 * under a memory manager that owns the device, for plug-ins entered after their host froze the
 * memory map, and for loops that cannot afford the device-wide synchronisation an allocation
 * brings.  The two intermediates (projected Q/K/V rows and the per-head attention output) live
 * in a fixed 8 MiB array inside the library image instead, which every GPU that loads the
 * library holds until the process exits.  Neither this call nor anything it calls allocates or
 * frees memory.
 *   - Works on the CURRENT device, for D = 1024 and 16 heads, and for 1 <= m <= 1024 merged rows;
 *     any other m is refused with LITEVGGT_ERR_SHAPE before anything is launched.  The extents
 *     are taken on trust from m: x_merged and y_merged are read / written as [m, 1024], w_qkv as
 *     [3072, 1024], w_o as [1024, 1024], b_qkv as [3072], b_o as [1024], all bf16; a shorter
 *     buffer is overrun.
 *   - The first call on a device looks up the array's device address and the device's
 *     properties and raises the kernels' shared-memory limits; it is also the call on which the
 *     driver loads the library's kernels and the array itself onto that device.  Make it outside
 *     any stream capture and before any region in which allocation is forbidden.  Later calls
 *     only enqueue (one memset, the kernels) and encode tensor maps on the host.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.  The
 *     call clears what has to start at zero (the status word) itself; two calls whose work
 *     overlaps on the GPU (different streams, no ordering between them) race on the array.
 *   - Tensors as in litevggt_global_attn (dev bf16, 16-byte aligned).  device_status: dev pointer
 *     to one 32-bit word, or NULL; it is zeroed on the stream and afterwards holds 1 if a kernel
 *     gave up on a bounded wait, 0 otherwise (with NULL the word inside the array is used and
 *     cannot be read back).  Asynchronous on `stream`. */
litevggt_status litevggt_global_attn_static(const void* x_merged, int64_t m, const void* w_qkv,
                                            const void* b_qkv, const void* w_o, const void* b_o,
                                            void* y_merged, uint32_t* device_status, void* stream);

/* The other sub-layers of an aggregator block (Sec. 3.1: the aggregator alternates frame-wise and
 * global self-attention; pre-norm transformer blocks with an MLP of ratio 4 are the reading taken).
 * They run at the full length N, outside the merged path.  Their workspace (N x 4D bf16 plus 1 GiB)
 * is allocated on the first of these calls.
 *
 * LayerNorm over the D channels of each row: y = (x - mean) / sqrt(var + eps) * gamma + beta with
 * the population variance.  x, out: dev bf16 [rows, D]; gamma, beta: dev bf16 [D]. */
litevggt_status litevggt_layernorm(litevggt_ctx* ctx, const void* x, int64_t rows, const void* gamma, const void* beta,
                                   float eps, void* out, void* stream);

/* Frame-local self-attention: the same attention layer as litevggt_global_attn applied to every
 * frame's T = P + S tokens separately (Sec. 3.1), y = residual + attn(x) (residual may be NULL).
 * x, residual, y: dev bf16 [N, D]; weights as in litevggt_global_attn. */
litevggt_status litevggt_frame_attn(litevggt_ctx* ctx, const void* x, const void* w_qkv, const void* b_qkv,
                                    const void* w_o, const void* b_o, const void* residual, void* y, void* stream);

/* Transformer MLP: y = residual + gelu(x w1^T + b1) w2^T + b2 with the erf form of GELU, 0.5 x (1 + erf(x / sqrt 2))
 * (erf by a rational approximation with absolute error below 1.5e-7, far under the bf16 rounding of the result).
 * x, residual (nullable), y: dev bf16 [rows, D], rows <= N; w1: dev bf16 [4D, D]; b1: dev bf16 [4D] or
 * NULL; w2: dev bf16 [D, 4D]; b2: dev bf16 [D] or NULL. */
litevggt_status litevggt_mlp(litevggt_ctx* ctx, const void* x, int64_t rows, const void* w1, const void* b1,
                             const void* w2, const void* b2, const void* residual, void* y, void* stream);

/* Unmerge (Sec. 3.4, "Token Unmerging"): out_i = y'[dst_of[i]] (+ residual_i).
 * y_merged: dev bf16 [M,D];  residual: dev bf16 [N,D] or NULL;  out: dev bf16 [N,D]. */
litevggt_status litevggt_unmerge(litevggt_ctx* ctx, const litevggt_plan* plan, const void* y_merged,
                                 const void* residual, void* out, void* stream);

/* One whole global layer from host memory: copies x (host bf16 [N,D]) to the device,
 * optionally (re)builds the plan from it (grad != NULL: dev fp32 [F,gh,gw], as in
 * litevggt_merge_plan; *plan_inout may then be NULL), runs merge -> global attention ->
 * unmerge with residual x, and copies the result to out (host bf16 [N,D]).  Weights are
 * dev pointers as in litevggt_global_attn.  Copies are asynchronous on `stream` when the
 * host buffers are pinned.  The device staging buffers are allocated on the first call. */
litevggt_status litevggt_global_layer_host(litevggt_ctx* ctx, litevggt_plan** plan_inout,
                                           const float* grad, const void* x_host, const void* w_qkv,
                                           const void* b_qkv, const void* w_o, const void* b_o,
                                           void* out_host, void* stream);

/* litevggt_global_layer_host for a sequence of independent calls (one batch of frames after the
 * other, as a server would run them): the host-to-device copy of a call's input and the
 * device-to-host copy of its output run on two copy streams of the context, with double-buffered
 * staging, so they overlap the neighbouring calls' kernels instead of adding to them (at 1000
 * frames the two copies are 2 x 2.13 GB, about 6 % of a layer).  Kernels run on `stream`, in call
 * order.  Arguments as in litevggt_global_layer_host; both host buffers should be pinned.
 *   - x_host must stay unchanged, and out_host is NOT complete, until litevggt_host_drain has been
 *     called on `stream` after this call and that point of the stream has been reached.
 *   - A call does not wait for the output copies of earlier calls: feeding one call's out_host to
 *     the next call's x_host needs a drain in between (or the plain entry point, which is ordered).
 *   - The first call allocates the second pair of staging buffers (2 x N x D bf16) and creates the
 *     streams and events. */
litevggt_status litevggt_global_layer_host_pipelined(litevggt_ctx* ctx, litevggt_plan** plan_inout,
                                                     const float* grad, const void* x_host,
                                                     const void* w_qkv, const void* b_qkv,
                                                     const void* w_o, const void* b_o,
                                                     void* out_host, void* stream);

/* Makes `stream` wait for every output copy started by litevggt_global_layer_host_pipelined so far
 * (no host synchronisation; a no-op when none was started). */
litevggt_status litevggt_host_drain(litevggt_ctx* ctx, void* stream);

/* Plain bf16 linear layer on the tensor cores: out[m,n] = a[m,k] w[n,k]^T + bias[n].
 * a: dev bf16 [m,k]; w: dev bf16 [n,k]; bias: dev bf16 [n] or NULL; out: dev bf16 [m,n].
 * k and n must be multiples of 64.  This is the projection step of the attention layer. */
litevggt_status litevggt_linear(litevggt_ctx* ctx, const void* a, int64_t m, int64_t k,
                                const void* w, int64_t n, const void* bias, void* out, void* stream);

/* Index cache policy (Sec. 3.4: indices are computed once every `recompute_interval`
 * global layers): *yes = 1 when the plan must be (re)built at this global layer. */
litevggt_status litevggt_should_refresh(const litevggt_ctx* ctx, const litevggt_plan* plan,
                                        int32_t global_layer_idx, int32_t* yes);

/* Copy plan contents to host arrays (synchronises `stream`; any output may be NULL):
 * dst_of [N] merged row of every token; size [M]; kept_idx [M] token index of each row;
 * cls [N]; best_dst [|Src|] anchor token index per src (ascending src token order);
 * best_sim [|Src|] its cosine; var / ga [F*P] Var map and GA map (0 for a plan built
 * from a caller's partition or imported). */
litevggt_status litevggt_plan_export(litevggt_ctx* ctx, const litevggt_plan* plan, int32_t* dst_of,
                                     int32_t* size, int32_t* kept_idx, uint8_t* cls, int32_t* best_dst,
                                     float* best_sim, float* var, float* ga, void* stream);

/* Build a plan from a host dst_of [N] array (tests; synchronous).  The array must map
 * kept tokens to consecutive rows 0..M-1 in ascending token order. */
litevggt_status litevggt_plan_import(litevggt_ctx* ctx, const int32_t* dst_of, litevggt_plan** out);
litevggt_status litevggt_plan_destroy(litevggt_plan* plan);

/* Pointer to an internal device buffer of the last litevggt_global_attn call (tests):
 * which = 0: qkv bf16 [M,3D], whose K third is stored multiplied by the softmax scale in base-2
 * units, 1/sqrt(64) log2(e), rounded once (the attention kernels take 2^(q . k) as it comes from the
 * tensor core);  which = 1: attention output o bf16 [M,D];  with qkv_dtype = 1 also
 * 2: Q as E4M3 bytes [M,D];  3: K likewise;  4: V transposed, bytes [D, round_up(M,128)] (row =
 * head * 64 + channel, column = key, zero beyond M);  5: float [3, heads], the largest magnitude of
 * Q, K, V per head (scale = amax / 448). */
litevggt_status litevggt_debug_buffer(litevggt_ctx* ctx, int which, void** dev_ptr, size_t* bytes);

/* Synchronise `stream` and report whether any kernel flagged a bounded-wait timeout or
 * an out-of-range index since the last poll (the flag is cleared). */
litevggt_status litevggt_poll_device_status(litevggt_ctx* ctx, void* stream);

/* Self-test of the bounded waits (the paper has no counterpart; Sec. 3.4's kernels are this
 * library's own).  Every pipelined kernel here waits on its barriers with a cycle limit; a wait
 * that runs out raises the status word and the kernel returns instead of hanging.  This call
 * launches a one-CTA kernel that waits, through the same device helpers, on a barrier that nobody
 * arrives on, with `limit_cycles` (1,000 .. 2^32) as the limit.  Afterwards
 * litevggt_poll_device_status must return LITEVGGT_ERR_DEVICE_TIMEOUT once and LITEVGGT_OK again
 * on the next poll, and the context stays usable.  outcome (host, nullable; the call then
 * synchronises the stream): bit 2 = the kernel ran to its end, bits 0 / 1 = a wait wrongly reported
 * the barrier as complete (must be clear).  Nothing faults, traps or spins without a bound. */
litevggt_status litevggt_selftest_bounded_wait(litevggt_ctx* ctx, int64_t limit_cycles, uint32_t* outcome,
                                               void* stream);

/* Device-time stopwatches.  Each step of the path is bracketed by CUDA events recorded on
 * the launching stream: which = 0 grad map, 1 var map, 2 partition + token lists, 3 cosine
 * matching (pack + GEMM/argmax), 4 selection + index build, 5 merge, 6 qkv projection,
 * 7 attention core, 8 output projection, 9 unmerge, 10 LayerNorm, 11 frame-local attention layer,
 * 12 MLP, 13 Q/K normalisation + rotary embedding, 14 E4M3 quantisation of Q/K/V.
 * litevggt_timers_reset forgets all
 * records; litevggt_timer_read synchronises on the recorded events and returns the summed
 * device time (ms) and the number of records (at most 64 are kept per step). */
litevggt_status litevggt_timers_reset(litevggt_ctx* ctx);
litevggt_status litevggt_timer_read(litevggt_ctx* ctx, int which, float* total_ms, int32_t* count);
/* The individual records of one stopwatch, oldest first: up to `capacity` device times (ms) are
 * written to `ms` (host), *count receives how many.  Synchronises on the recorded events. */
litevggt_status litevggt_timer_samples(litevggt_ctx* ctx, int which, float* ms, int32_t capacity, int32_t* count);

/* Number of kernels this library has launched on behalf of ctx since creation. */
litevggt_status litevggt_launch_count(const litevggt_ctx* ctx, int64_t* launches);

const char* litevggt_status_string(litevggt_status s);

#ifdef __cplusplus
}
#endif
#endif /* LITEVGGT_H_ */
