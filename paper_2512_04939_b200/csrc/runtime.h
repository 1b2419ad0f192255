// Host-side runtime objects behind the C ABI: context (workspace, device status word,
// launch counter), plan (cached merge indices) and the launchers of each kernel group.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "../../include/litevggt.h"

namespace lv {

struct Sizes {
  int frames, grid_h, grid_w, n_special, dim, heads;
  int patches;        // P
  int tokens_frame;   // T
  long long n_tokens; // N
  int n_dst_frame, n_ga_frame, n_src_frame;
  long long n_src, n_dst;
  long long n_remove; // R
  long long n_merged; // M
};

inline long long round_up(long long v, long long a) { return (v + a - 1) / a * a; }

// Raises a kernel's dynamic shared-memory limit once per device (`done` holds one bit per device,
// one object per kernel), so that a launcher's later calls only enqueue work.
inline cudaError_t set_max_dynamic_smem_once(const void* kernel, int bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) done.fetch_or(bit, std::memory_order_release);
  return e;
}

// The attention kernels take the exponentials in base 2 of scores that already carry the softmax
// scale: 1/sqrt(64) log2(e) is folded into K where K is last rounded to bf16 (the QKV projection's
// epilogue, or the Q/K normalisation pass), so that no arithmetic stands between the tensor core's
// scores and the exponential, at no extra rounding.
constexpr float kKeyScaleLog2e = 0.125f * 1.4426950408889634f;

constexpr long long kMlpChunkRows = 131072;  // rows of the 4D-wide hidden activations held at a time (1 GiB)

// One device allocation carved into named regions.
struct Workspace {
  uint8_t* base = nullptr;
  size_t bytes = 0;
  // scoring
  float* var_map = nullptr;     // [F*P]
  float* ga_score = nullptr;    // [F*P]
  uint8_t* cls = nullptr;       // [N]
  int* src_list = nullptr;      // [|Src|] token index, ascending
  int* dst_list = nullptr;      // [|Dst|] token index, ascending
  // matching
  __nv_bfloat16* panel_src = nullptr;  // [|Src|, D] packed rows
  __nv_bfloat16* panel_dst = nullptr;  // [|Dst|, D]
  float* inv_norm_src = nullptr;       // [|Src|]
  float* inv_norm_dst = nullptr;       // [round_up(|Dst|,256)]
  // index build
  unsigned long long* sort_keys = nullptr;  // [pow2 >= max(|Src|, R)]
  int* scan_tmp = nullptr;                  // [N] kept flags / scan output
  int* scan_blocks = nullptr;               // block sums
  int* row_of = nullptr;                    // [N]
  // attention
  __nv_bfloat16* qkv = nullptr;    // [M, 3D]
  __nv_bfloat16* attn_o = nullptr; // [M, D]
  float* attn_o_state = nullptr;   // [M, D] running output between key chunks (long sequences only)
  float* attn_ml_state = nullptr;  // [M, heads, 4] reference maximum and partial row sums
  float* attn_kmax = nullptr;      // [max(frames, 1), heads] largest |k|^2 per sequence and head
  // E4M3 variant of the attention operands (qkv_dtype = 1)
  uint8_t* q8 = nullptr;           // [M, D] bytes
  uint8_t* k8 = nullptr;           // [M, D] bytes
  uint8_t* v8t = nullptr;          // [D, round_up(M, 128)] bytes: V transposed, head-major rows
  float* qkv_amax = nullptr;       // [3, heads] largest magnitude of Q, K, V per head
  // whole-layer-from-host staging
  __nv_bfloat16* stage_x = nullptr;   // [N, D]
  __nv_bfloat16* stage_xm = nullptr;  // [M, D]
  __nv_bfloat16* stage_ym = nullptr;  // [M, D]
  __nv_bfloat16* stage_out = nullptr; // [N, D]
  // block workspace of the frame-local attention and the MLP (allocated on first use)
  __nv_bfloat16* blk_qkv = nullptr;   // [N, 3D]
  __nv_bfloat16* blk_o = nullptr;     // [N, D]
  __nv_bfloat16* blk_hidden = nullptr; // [kMlpChunkRows, 4D]
  uint32_t* status = nullptr;         // device status word
};

}  // namespace lv

namespace lv {
// Device-time stopwatches, one per step of the path: CUDA event pairs recorded on the
// launching stream around the step's kernels, kept in a small ring per step.
constexpr int kNumTimers = 15;
constexpr int kTimerSlots = 64;
struct Timers {
  cudaEvent_t start[kNumTimers][kTimerSlots];
  cudaEvent_t stop[kNumTimers][kTimerSlots];
  int used[kNumTimers];  // launches recorded since the last reset
  bool created;
};
}  // namespace lv

// Streams, events and the second pair of staging buffers behind litevggt_global_layer_host_pipelined.
struct HostPipe {
  bool created = false;
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t in_ready[2] = {}, x_free[2] = {}, out_ready[2] = {}, out_free[2] = {};
  bool used[2] = {false, false};
  unsigned long long calls = 0;
  __nv_bfloat16* x[2] = {nullptr, nullptr};    // [N, D] each
  __nv_bfloat16* out[2] = {nullptr, nullptr};  // [N, D] each
  uint8_t* extra = nullptr;                     // allocation that holds x[1] and out[1]
};

struct litevggt_ctx {
  uint32_t magic;
  litevggt_config cfg;
  lv::Sizes sz;
  int device;
  int num_sms;
  lv::Workspace ws;
  long long launches;
  void* encode_tiled;  // cuTensorMapEncodeTiled, resolved at run time
  lv::Timers timers;
  HostPipe pipe;
};

struct litevggt_plan {
  uint32_t magic;
  const litevggt_ctx* owner;
  int built;
  int last_refresh_layer;
  bool has_maps;       // var/ga/best_* valid (plan built by the library's own scoring)
  uint8_t* base;       // one device allocation
  int* dst_of;         // [N]
  int* size;           // [M]
  int* kept_idx;       // [M]
  int* seg_off;        // [M+1]
  int* seg_src;        // [R]
  int* best_dst;       // [|Src|] anchor token index
  float* best_sim;     // [|Src|]
};

namespace lv {

// bits of the device status word
constexpr uint32_t kStatusTimeout = 1u;
constexpr uint32_t kStatusBounds = 2u;

constexpr uint32_t kCtxMagic = 0x4c564358u;
constexpr uint32_t kPlanMagic = 0x4c56504cu;

// tensor_map.cu
bool resolve_encode_tiled(void** fn);
// 2-D bf16 tensor [outer, inner] row-major with row pitch `pitch_elems`; box [box_outer, box_inner],
// 128-byte swizzle, zero fill outside the tensor.
bool make_tmap_bf16_2d(void* encode_fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                       uint64_t pitch_elems, uint32_t box_inner, uint32_t box_outer);
bool make_tmap_u8_2d(void* encode_fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                     uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer);

// scoring.cu
cudaError_t launch_grad_map(const litevggt_ctx* ctx, const float* images, float* grad, cudaStream_t s, int* launches);
cudaError_t launch_var_map(const litevggt_ctx* ctx, const __nv_bfloat16* x, float* var,
                           cudaStream_t s, int* launches);
cudaError_t launch_partition(const litevggt_ctx* ctx, const float* grad, const float* var, float* ga, uint8_t* cls,
                             cudaStream_t s, int* launches);
cudaError_t launch_build_lists(const litevggt_ctx* ctx, const uint8_t* cls, int* src_list, int* dst_list,
                               cudaStream_t s, int* launches);

// similarity.cu
cudaError_t launch_match(litevggt_ctx* ctx, const __nv_bfloat16* x, int* best_dst, float* best_sim, cudaStream_t s,
                         int* launches);

// index_build.cu
cudaError_t launch_index_build(litevggt_ctx* ctx, litevggt_plan* plan, cudaStream_t s, int* launches);
size_t sort_capacity(long long n);

// merge_unmerge.cu
cudaError_t launch_merge(const litevggt_ctx* ctx, const litevggt_plan* plan, const __nv_bfloat16* x,
                         __nv_bfloat16* xm, cudaStream_t s, int* launches);
cudaError_t launch_unmerge(const litevggt_ctx* ctx, const litevggt_plan* plan, const __nv_bfloat16* ym,
                           const __nv_bfloat16* residual, __nv_bfloat16* out, cudaStream_t s, int* launches);

// linear.cu
cudaError_t launch_linear(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k, const __nv_bfloat16* w,
                          long long n, const __nv_bfloat16* bias, __nv_bfloat16* out, cudaStream_t s, int* launches);
// The same with output columns [scale_begin, scale_end) (multiples of 64) multiplied by `scale` in
// fp32 before the one rounding to bf16: the QKV projection of an attention layer scales its K columns.
cudaError_t launch_linear_scaled(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k,
                                 const __nv_bfloat16* w, long long n, const __nv_bfloat16* bias, int scale_begin,
                                 int scale_end, float scale, __nv_bfloat16* out, cudaStream_t s, int* launches);

cudaError_t launch_linear_mlp(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k,
                              const __nv_bfloat16* w, long long n, const __nv_bfloat16* bias, int gelu,
                              const __nv_bfloat16* residual, __nv_bfloat16* out, cudaStream_t s, int* launches);
cudaError_t launch_layernorm(const __nv_bfloat16* x, const __nv_bfloat16* gamma, const __nv_bfloat16* beta,
                             __nv_bfloat16* out, long long rows, float eps, cudaStream_t s, int* launches);

// selftest.cu: one CTA waits on a barrier that nobody arrives on, with the given cycle limit
cudaError_t launch_bounded_wait_selftest(litevggt_ctx* ctx, long long limit_cycles, uint32_t* outcome, cudaStream_t s,
                                         int* launches);

// attention.cu
// n_seq independent sequences of seq_len rows each, laid back to back in qkv / o
// qk_embed.cu: optional per-head LayerNorm and 2-D rotary embedding of Q and K, in place on [m, 3D]
cudaError_t launch_qk_embed(const litevggt_ctx* ctx, __nv_bfloat16* qkv, const int* kept_idx, long long m,
                            const __nv_bfloat16* q_gamma, const __nv_bfloat16* q_beta, const __nv_bfloat16* k_gamma,
                            const __nv_bfloat16* k_beta, float eps, int rope, float rope_base, cudaStream_t s,
                            int* launches);
cudaError_t launch_flash_attention(litevggt_ctx* ctx, const __nv_bfloat16* qkv, long long seq_len, int n_seq,
                                   __nv_bfloat16* o, cudaStream_t s, int* launches);
size_t attention_state_bytes(long long m, int dim, int heads, size_t* ml_offset);
// E4M3 variant: per-head amax of Q, K, V and their quantised copies (fp8_quant.cu), then the
// attention core on those (attention.cu); one sequence of m rows
cudaError_t launch_qkv_quantize(litevggt_ctx* ctx, const __nv_bfloat16* qkv, long long m, cudaStream_t s, int* launches);
cudaError_t launch_flash_attention_fp8(litevggt_ctx* ctx, long long m, __nv_bfloat16* o, cudaStream_t s, int* launches);

}  // namespace lv
