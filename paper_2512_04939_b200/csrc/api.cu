// extern "C" boundary: argument validation, context / plan life cycle, launch sequencing.
// Every step of the path runs in the kernels behind the launch_* functions; this file
// only checks arguments, carves the workspace and orders the launches on the caller's
// stream.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "runtime.h"

using namespace lv;

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool ctx_ok(const litevggt_ctx* c) { return c != nullptr && c->magic == kCtxMagic; }
inline bool plan_ok(const litevggt_plan* p) { return p != nullptr && p->magic == kPlanMagic; }

// fractions arrive as float; snap them to 1e-6 so that 0.7f means 0.7
inline double snap(float v) { return round((double)v * 1e6) / 1e6; }

litevggt_status compute_sizes(const litevggt_config& c, Sizes* out) {
  if (c.frames < 1 || c.grid_h < 1 || c.grid_w < 1 || c.patch_px < 1 || c.n_special < 0) return LITEVGGT_ERR_BAD_CONFIG;
  if (c.dim != 1024 || c.heads != 16) return LITEVGGT_ERR_BAD_CONFIG;  // kernels are specialised for D=1024, 16x64
  if (c.cell_h < 1 || c.cell_w < 1 || c.var_window != 3 || c.recompute_interval < 1) return LITEVGGT_ERR_BAD_CONFIG;
  if (!(c.merge_ratio >= 0.0f && c.merge_ratio <= 1.0f)) return LITEVGGT_ERR_BAD_CONFIG;
  if (!(c.ga_keep_frac >= 0.0f && c.ga_keep_frac <= 1.0f)) return LITEVGGT_ERR_BAD_CONFIG;
  if (c.qkv_dtype != 0 && c.qkv_dtype != 1) return LITEVGGT_ERR_BAD_CONFIG;  // bf16 or E4M3 attention operands
  if (c.patch_px > 30) return LITEVGGT_ERR_BAD_CONFIG;  // a patch and its two halo columns share a warp in the Grad map
  Sizes z;
  z.frames = c.frames; z.grid_h = c.grid_h; z.grid_w = c.grid_w; z.n_special = c.n_special;
  z.dim = c.dim; z.heads = c.heads;
  const long long p = (long long)c.grid_h * c.grid_w;
  if (p > 8192 || c.grid_w > 64) return LITEVGGT_ERR_BAD_CONFIG;  // the Var map kernel keeps per-row results of <= 64 columns in shared memory
  z.patches = (int)p;
  z.tokens_frame = (int)p + c.n_special;
  z.n_tokens = (long long)c.frames * z.tokens_frame;
  if (z.n_tokens > (1ll << 22)) return LITEVGGT_ERR_BAD_CONFIG;  // scans and sorts are sized for <= 4 Mi tokens
  z.n_dst_frame = ((c.grid_h + c.cell_h - 1) / c.cell_h) * ((c.grid_w + c.cell_w - 1) / c.cell_w);
  long long n_ga = (long long)floor(snap(c.ga_keep_frac) * (double)p + 1e-9);
  if (n_ga > p - z.n_dst_frame) n_ga = p - z.n_dst_frame;
  z.n_ga_frame = (int)n_ga;
  z.n_src_frame = (int)(p - z.n_dst_frame - n_ga);
  z.n_src = (long long)(c.frames - 1) * z.n_src_frame;
  z.n_dst = p + (long long)(c.frames - 1) * z.n_dst_frame;
  long long r = (long long)floor(snap(c.merge_ratio) * (double)z.n_tokens + 1e-9);
  if (r > z.n_src) r = z.n_src;
  z.n_remove = r;
  z.n_merged = z.n_tokens - r;
  *out = z;
  return LITEVGGT_OK;
}

struct Carver {
  size_t off = 0;
  template <class T>
  size_t take(long long count) {
    const size_t at = off;
    off += (size_t)round_up((long long)sizeof(T) * (count > 0 ? count : 1), 256);
    return at;
  }
};

void bump(litevggt_ctx* ctx, int n) { ctx->launches += n; }

// Brackets the launches of one step with an event pair on the launching stream.
struct StepTimer {
  litevggt_ctx* ctx;
  cudaStream_t s;
  int which, slot;
  StepTimer(litevggt_ctx* c, int w, cudaStream_t st) : ctx(c), s(st), which(w), slot(-1) {
    Timers& t = ctx->timers;
    if (!t.created) return;
    slot = t.used[which] % kTimerSlots;
    cudaEventRecord(t.start[which][slot], s);
  }
  ~StepTimer() {
    if (slot < 0) return;
    cudaEventRecord(ctx->timers.stop[which][slot], s);
    ++ctx->timers.used[which];
  }
};

litevggt_status cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return LITEVGGT_OK;
  (void)cudaGetLastError();
  return e == cudaErrorMemoryAllocation ? LITEVGGT_ERR_ALLOC : LITEVGGT_ERR_CUDA;
}

litevggt_status alloc_plan(litevggt_ctx* ctx, litevggt_plan** out) {
  const Sizes& z = ctx->sz;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  litevggt_plan* p = new (std::nothrow) litevggt_plan();
  if (p == nullptr) return LITEVGGT_ERR_ALLOC;
  Carver c;
  const size_t o_dst_of = c.take<int>(z.n_tokens), o_size = c.take<int>(z.n_merged);
  const size_t o_kept = c.take<int>(z.n_merged), o_off = c.take<int>(z.n_merged + 1);
  const size_t o_seg = c.take<int>(z.n_remove), o_bd = c.take<int>(z.n_src), o_bs = c.take<float>(z.n_src);
  if (cudaMalloc(&p->base, c.off) != cudaSuccess) {
    (void)cudaGetLastError();
    delete p;
    return LITEVGGT_ERR_ALLOC;
  }
  cudaMemset(p->base, 0, c.off);
  p->magic = kPlanMagic;
  p->owner = ctx;
  p->built = 0;
  p->last_refresh_layer = -1;
  p->has_maps = false;
  p->dst_of = reinterpret_cast<int*>(p->base + o_dst_of);
  p->size = reinterpret_cast<int*>(p->base + o_size);
  p->kept_idx = reinterpret_cast<int*>(p->base + o_kept);
  p->seg_off = reinterpret_cast<int*>(p->base + o_off);
  p->seg_src = reinterpret_cast<int*>(p->base + o_seg);
  p->best_dst = reinterpret_cast<int*>(p->base + o_bd);
  p->best_sim = reinterpret_cast<float*>(p->base + o_bs);
  *out = p;
  return LITEVGGT_OK;
}

// matching -> selection -> index arrays, from the class array in ctx->ws.cls
litevggt_status plan_from_classes(litevggt_ctx* ctx, const __nv_bfloat16* x, litevggt_plan* plan, cudaStream_t s) {
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 2, s);
    e = launch_build_lists(ctx, ctx->ws.cls, ctx->ws.src_list, ctx->ws.dst_list, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 3, s);
    e = launch_match(ctx, x, plan->best_dst, plan->best_sim, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 4, s);
    e = launch_index_build(ctx, plan, s, &n);
  }
  bump(ctx, n);
  if (e != cudaSuccess) return cuda_status(e);
  plan->built = 1;
  return LITEVGGT_OK;
}

litevggt_status ensure_staging(litevggt_ctx* ctx) {
  if (ctx->ws.stage_x != nullptr) return LITEVGGT_OK;
  const Sizes& z = ctx->sz;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  const size_t big = (size_t)z.n_tokens * z.dim * 2, small = (size_t)z.n_merged * z.dim * 2;
  uint8_t* base = nullptr;
  const size_t total = 2 * (size_t)round_up((long long)big, 256) + 2 * (size_t)round_up((long long)small, 256);
  if (cudaMalloc(&base, total) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVGGT_ERR_ALLOC;
  }
  size_t off = 0;
  ctx->ws.stage_x = reinterpret_cast<__nv_bfloat16*>(base + off); off += (size_t)round_up((long long)big, 256);
  ctx->ws.stage_out = reinterpret_cast<__nv_bfloat16*>(base + off); off += (size_t)round_up((long long)big, 256);
  ctx->ws.stage_xm = reinterpret_cast<__nv_bfloat16*>(base + off); off += (size_t)round_up((long long)small, 256);
  ctx->ws.stage_ym = reinterpret_cast<__nv_bfloat16*>(base + off);
  ctx->ws.bytes += total;
  return LITEVGGT_OK;
}

// Copy streams, events and the second pair of [N, D] staging buffers of the pipelined host entry.
litevggt_status ensure_host_pipe(litevggt_ctx* ctx) {
  litevggt_status st = ensure_staging(ctx);
  if (st != LITEVGGT_OK) return st;
  HostPipe& hp = ctx->pipe;
  if (hp.created) return LITEVGGT_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  const size_t big = (size_t)round_up(ctx->sz.n_tokens * ctx->sz.dim * 2, 256);
  if (cudaMalloc(&hp.extra, 2 * big) != cudaSuccess) {
    (void)cudaGetLastError();
    hp.extra = nullptr;
    return LITEVGGT_ERR_ALLOC;
  }
  cudaError_t e = cudaStreamCreateWithFlags(&hp.copy_in, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&hp.copy_out, cudaStreamNonBlocking);
  cudaEvent_t* sets[4] = {hp.in_ready, hp.x_free, hp.out_ready, hp.out_free};
  for (int k = 0; k < 4 && e == cudaSuccess; ++k)
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&sets[k][i], cudaEventDisableTiming);
  if (e != cudaSuccess) {
    // partial set-up is released at destroy time only if `created`; release it here instead
    if (hp.copy_in) cudaStreamDestroy(hp.copy_in);
    if (hp.copy_out) cudaStreamDestroy(hp.copy_out);
    for (int k = 0; k < 4; ++k)
      for (int i = 0; i < 2; ++i)
        if (sets[k][i]) cudaEventDestroy(sets[k][i]);
    cudaFree(hp.extra);
    hp = HostPipe();
    return cuda_status(e);
  }
  hp.x[0] = ctx->ws.stage_x;
  hp.out[0] = ctx->ws.stage_out;
  hp.x[1] = reinterpret_cast<__nv_bfloat16*>(hp.extra);
  hp.out[1] = reinterpret_cast<__nv_bfloat16*>(hp.extra + big);
  ctx->ws.bytes += 2 * big;
  hp.created = true;
  return LITEVGGT_OK;
}

litevggt_status ensure_block_ws(litevggt_ctx* ctx) {
  if (ctx->ws.blk_qkv != nullptr) return LITEVGGT_OK;
  const Sizes& z = ctx->sz;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  const size_t qkv = (size_t)round_up(z.n_tokens * 3 * z.dim * 2, 256), o = (size_t)round_up(z.n_tokens * z.dim * 2, 256);
  const long long hid_rows = z.n_tokens < kMlpChunkRows ? z.n_tokens : kMlpChunkRows;
  const size_t hid = (size_t)round_up(hid_rows * 4 * z.dim * 2, 256);
  uint8_t* base = nullptr;
  if (cudaMalloc(&base, qkv + o + hid) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVGGT_ERR_ALLOC;
  }
  ctx->ws.blk_qkv = reinterpret_cast<__nv_bfloat16*>(base);
  ctx->ws.blk_o = reinterpret_cast<__nv_bfloat16*>(base + qkv);
  ctx->ws.blk_hidden = reinterpret_cast<__nv_bfloat16*>(base + qkv + o);
  ctx->ws.bytes += qkv + o + hid;
  return LITEVGGT_OK;
}

}  // namespace

extern "C" {

litevggt_status litevggt_default_config(int32_t frames, int32_t grid_h, int32_t grid_w, float merge_ratio,
                                        litevggt_config* cfg) {
  if (cfg == nullptr) return LITEVGGT_ERR_NULL;
  memset(cfg, 0, sizeof(*cfg));
  cfg->frames = frames; cfg->grid_h = grid_h; cfg->grid_w = grid_w;
  cfg->patch_px = 14; cfg->n_special = 5; cfg->dim = 1024; cfg->heads = 16;
  cfg->merge_ratio = merge_ratio; cfg->ga_keep_frac = 0.10f; cfg->alpha = 0.5f; cfg->beta = 0.5f;
  cfg->cell_h = 2; cfg->cell_w = 2; cfg->var_window = 3; cfg->recompute_interval = 6; cfg->qkv_dtype = 0;
  Sizes z;
  return compute_sizes(*cfg, &z);
}

litevggt_status litevggt_create(const litevggt_config* cfg, int device, litevggt_ctx** out) {
  if (cfg == nullptr || out == nullptr) return LITEVGGT_ERR_NULL;
  *out = nullptr;
  Sizes z;
  litevggt_status st = compute_sizes(*cfg, &z);
  if (st != LITEVGGT_OK) return st;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    (void)cudaGetLastError();
    return LITEVGGT_ERR_CUDA;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return cuda_status(cudaGetLastError());
  if (prop.major != 10) return LITEVGGT_ERR_ARCH;
  DeviceGuard g(device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  litevggt_ctx* ctx = new (std::nothrow) litevggt_ctx();
  if (ctx == nullptr) return LITEVGGT_ERR_ALLOC;
  ctx->magic = kCtxMagic;
  ctx->cfg = *cfg;
  ctx->sz = z;
  ctx->device = device;
  ctx->num_sms = prop.multiProcessorCount;
  ctx->launches = 0;
  ctx->encode_tiled = nullptr;
  ctx->timers.created = false;
  if (!resolve_encode_tiled(&ctx->encode_tiled)) {
    delete ctx;
    return LITEVGGT_ERR_CUDA;
  }
  Carver c;
  const long long fp = (long long)z.frames * z.patches;
  const long long cap = (long long)sort_capacity(z.n_src);
  const size_t o_var = c.take<float>(fp), o_ga = c.take<float>(fp), o_cls = c.take<uint8_t>(z.n_tokens);
  const size_t o_src = c.take<int>(z.n_src), o_dst = c.take<int>(z.n_dst);
  const size_t o_ps = c.take<__nv_bfloat16>(z.n_src * z.dim), o_pd = c.take<__nv_bfloat16>(z.n_dst * z.dim);
  const size_t o_ns = c.take<float>(z.n_src), o_nd = c.take<float>(round_up(z.n_dst, 256));
  const size_t o_keys = c.take<unsigned long long>(cap);
  const size_t o_tmp = c.take<int>(z.n_tokens + 1), o_blk = c.take<int>(2048), o_row = c.take<int>(z.n_tokens);
  const size_t o_qkv = c.take<__nv_bfloat16>(z.n_merged * 3 * z.dim), o_o = c.take<__nv_bfloat16>(z.n_merged * z.dim);
  size_t ml_off = 0;
  const size_t state_bytes = attention_state_bytes(z.n_merged, z.dim, z.heads, &ml_off);
  const size_t o_state = c.take<uint8_t>((long long)state_bytes);
  const size_t o_kmax = c.take<float>((long long)z.frames * z.heads);
  const bool fp8 = cfg->qkv_dtype == 1;
  const long long m_pad = round_up(z.n_merged, 128);
  const size_t o_q8 = c.take<uint8_t>(fp8 ? z.n_merged * z.dim : 0), o_k8 = c.take<uint8_t>(fp8 ? z.n_merged * z.dim : 0);
  const size_t o_v8 = c.take<uint8_t>(fp8 ? m_pad * z.dim : 0), o_amax = c.take<float>(48);
  const size_t o_status = c.take<uint32_t>(4);
  Workspace& ws = ctx->ws;
  if (cudaMalloc(&ws.base, c.off) != cudaSuccess) {
    (void)cudaGetLastError();
    delete ctx;
    return LITEVGGT_ERR_ALLOC;
  }
  ws.bytes = c.off;
  ws.var_map = reinterpret_cast<float*>(ws.base + o_var);
  ws.ga_score = reinterpret_cast<float*>(ws.base + o_ga);
  ws.cls = ws.base + o_cls;
  ws.src_list = reinterpret_cast<int*>(ws.base + o_src);
  ws.dst_list = reinterpret_cast<int*>(ws.base + o_dst);
  ws.panel_src = reinterpret_cast<__nv_bfloat16*>(ws.base + o_ps);
  ws.panel_dst = reinterpret_cast<__nv_bfloat16*>(ws.base + o_pd);
  ws.inv_norm_src = reinterpret_cast<float*>(ws.base + o_ns);
  ws.inv_norm_dst = reinterpret_cast<float*>(ws.base + o_nd);
  ws.sort_keys = reinterpret_cast<unsigned long long*>(ws.base + o_keys);
  ws.scan_tmp = reinterpret_cast<int*>(ws.base + o_tmp);
  ws.scan_blocks = reinterpret_cast<int*>(ws.base + o_blk);
  ws.row_of = reinterpret_cast<int*>(ws.base + o_row);
  ws.qkv = reinterpret_cast<__nv_bfloat16*>(ws.base + o_qkv);
  ws.attn_o = reinterpret_cast<__nv_bfloat16*>(ws.base + o_o);
  if (state_bytes > 0) {
    ws.attn_o_state = reinterpret_cast<float*>(ws.base + o_state);
    ws.attn_ml_state = reinterpret_cast<float*>(ws.base + o_state + ml_off);
  }
  ws.attn_kmax = reinterpret_cast<float*>(ws.base + o_kmax);
  if (fp8) {
    ws.q8 = ws.base + o_q8;
    ws.k8 = ws.base + o_k8;
    ws.v8t = ws.base + o_v8;
    ws.qkv_amax = reinterpret_cast<float*>(ws.base + o_amax);
  }
  ws.status = reinterpret_cast<uint32_t*>(ws.base + o_status);
  if (cudaMemset(ws.base + o_var, 0, o_src - o_var) != cudaSuccess ||
      cudaMemset(ws.status, 0, 16) != cudaSuccess) {
    (void)cudaGetLastError();
    cudaFree(ws.base);
    delete ctx;
    return LITEVGGT_ERR_CUDA;
  }
  Timers& tm = ctx->timers;
  tm.created = true;
  for (int w = 0; w < kNumTimers; ++w) {
    tm.used[w] = 0;
    for (int i = 0; i < kTimerSlots; ++i)
      if (cudaEventCreate(&tm.start[w][i]) != cudaSuccess || cudaEventCreate(&tm.stop[w][i]) != cudaSuccess)
        tm.created = false;
  }
  (void)cudaGetLastError();
  *out = ctx;
  return LITEVGGT_OK;
}

litevggt_status litevggt_timers_reset(litevggt_ctx* ctx) {
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  for (int w = 0; w < kNumTimers; ++w) ctx->timers.used[w] = 0;
  return LITEVGGT_OK;
}

litevggt_status litevggt_timer_read(litevggt_ctx* ctx, int which, float* total_ms, int32_t* count) {
  if (!ctx_ok(ctx) || total_ms == nullptr || count == nullptr) return LITEVGGT_ERR_NULL;
  if (which < 0 || which >= kNumTimers) return LITEVGGT_ERR_SHAPE;
  Timers& tm = ctx->timers;
  *total_ms = 0.0f;
  *count = 0;
  if (!tm.created) return LITEVGGT_ERR_CUDA;
  const int n = tm.used[which] < kTimerSlots ? tm.used[which] : kTimerSlots;
  for (int i = 0; i < n; ++i) {
    float ms = 0.0f;
    if (cudaEventSynchronize(tm.stop[which][i]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, tm.start[which][i], tm.stop[which][i]) != cudaSuccess)
      return cuda_status(cudaGetLastError());
    *total_ms += ms;
  }
  *count = n;
  return LITEVGGT_OK;
}

litevggt_status litevggt_timer_samples(litevggt_ctx* ctx, int which, float* ms, int32_t capacity, int32_t* count) {
  if (!ctx_ok(ctx) || ms == nullptr || count == nullptr) return LITEVGGT_ERR_NULL;
  if (which < 0 || which >= kNumTimers || capacity < 0) return LITEVGGT_ERR_SHAPE;
  Timers& tm = ctx->timers;
  *count = 0;
  if (!tm.created) return LITEVGGT_ERR_CUDA;
  // the ring keeps the latest kTimerSlots records; slot i holds record i, i + kTimerSlots, ...
  const int used = tm.used[which];
  const int kept = used < kTimerSlots ? used : kTimerSlots;
  const int n = kept < capacity ? kept : capacity;
  for (int i = 0; i < n; ++i) {
    const int slot = (used - kept + i) % kTimerSlots;
    if (cudaEventSynchronize(tm.stop[which][slot]) != cudaSuccess ||
        cudaEventElapsedTime(&ms[i], tm.start[which][slot], tm.stop[which][slot]) != cudaSuccess)
      return cuda_status(cudaGetLastError());
  }
  *count = n;
  return LITEVGGT_OK;
}

litevggt_status litevggt_destroy(litevggt_ctx* ctx) {
  if (ctx == nullptr) return LITEVGGT_OK;
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  DeviceGuard g(ctx->device);
  cudaDeviceSynchronize();
  if (ctx->timers.created)
    for (int w = 0; w < kNumTimers; ++w)
      for (int i = 0; i < kTimerSlots; ++i) {
        cudaEventDestroy(ctx->timers.start[w][i]);
        cudaEventDestroy(ctx->timers.stop[w][i]);
      }
  if (ctx->pipe.created) {
    cudaStreamDestroy(ctx->pipe.copy_in);
    cudaStreamDestroy(ctx->pipe.copy_out);
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(ctx->pipe.in_ready[i]);
      cudaEventDestroy(ctx->pipe.x_free[i]);
      cudaEventDestroy(ctx->pipe.out_ready[i]);
      cudaEventDestroy(ctx->pipe.out_free[i]);
    }
    if (ctx->pipe.extra != nullptr) cudaFree(ctx->pipe.extra);
  }
  if (ctx->ws.stage_x != nullptr) cudaFree(ctx->ws.stage_x);
  if (ctx->ws.blk_qkv != nullptr) cudaFree(ctx->ws.blk_qkv);
  if (ctx->ws.base != nullptr) cudaFree(ctx->ws.base);
  (void)cudaGetLastError();
  ctx->magic = 0;
  delete ctx;
  return LITEVGGT_OK;
}

litevggt_status litevggt_sizes(const litevggt_ctx* ctx, int64_t* n_tokens, int64_t* n_merged, int64_t* n_src,
                               int64_t* n_dst, size_t* workspace_bytes) {
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  if (n_tokens) *n_tokens = ctx->sz.n_tokens;
  if (n_merged) *n_merged = ctx->sz.n_merged;
  if (n_src) *n_src = ctx->sz.n_src;
  if (n_dst) *n_dst = ctx->sz.n_dst;
  if (workspace_bytes) *workspace_bytes = ctx->ws.bytes;
  return LITEVGGT_OK;
}

litevggt_status litevggt_grad_map(litevggt_ctx* ctx, const float* images, float* grad, void* stream) {
  if (!ctx_ok(ctx) || images == nullptr || grad == nullptr) return LITEVGGT_ERR_NULL;
  if (!aligned16(images) || !aligned16(grad)) return LITEVGGT_ERR_ALIGN;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 0, (cudaStream_t)stream);
    e = launch_grad_map(ctx, images, grad, (cudaStream_t)stream, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_merge_plan(litevggt_ctx* ctx, const void* x, const float* grad, litevggt_plan** plan_inout,
                                    void* stream) {
  if (!ctx_ok(ctx) || x == nullptr || grad == nullptr || plan_inout == nullptr) return LITEVGGT_ERR_NULL;
  if (!aligned16(x) || !aligned16(grad)) return LITEVGGT_ERR_ALIGN;
  if (*plan_inout != nullptr && (!plan_ok(*plan_inout) || (*plan_inout)->owner != ctx)) return LITEVGGT_ERR_STALE_PLAN;
  if (*plan_inout == nullptr) {
    litevggt_status st = alloc_plan(ctx, plan_inout);
    if (st != LITEVGGT_OK) return st;
  }
  litevggt_plan* plan = *plan_inout;
  cudaStream_t s = (cudaStream_t)stream;
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 1, s);
    e = launch_var_map(ctx, xb, ctx->ws.var_map, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 2, s);
    e = launch_partition(ctx, grad, ctx->ws.var_map, ctx->ws.ga_score, ctx->ws.cls, s, &n);
  }
  bump(ctx, n);
  if (e != cudaSuccess) return cuda_status(e);
  plan->has_maps = true;
  return plan_from_classes(ctx, xb, plan, s);
}

litevggt_status litevggt_merge_plan_with_partition(litevggt_ctx* ctx, const void* x, const uint8_t* cls,
                                                   litevggt_plan** plan_inout, void* stream) {
  if (!ctx_ok(ctx) || x == nullptr || cls == nullptr || plan_inout == nullptr) return LITEVGGT_ERR_NULL;
  if (!aligned16(x)) return LITEVGGT_ERR_ALIGN;
  if (*plan_inout != nullptr && (!plan_ok(*plan_inout) || (*plan_inout)->owner != ctx)) return LITEVGGT_ERR_STALE_PLAN;
  if (*plan_inout == nullptr) {
    litevggt_status st = alloc_plan(ctx, plan_inout);
    if (st != LITEVGGT_OK) return st;
  }
  litevggt_plan* plan = *plan_inout;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(ctx->ws.cls, cls, (size_t)ctx->sz.n_tokens, cudaMemcpyDeviceToDevice, s);
  if (e != cudaSuccess) return cuda_status(e);
  plan->has_maps = false;
  return plan_from_classes(ctx, static_cast<const __nv_bfloat16*>(x), plan, s);
}

litevggt_status litevggt_merge(litevggt_ctx* ctx, const litevggt_plan* plan, const void* x, void* x_merged,
                               void* stream) {
  if (!ctx_ok(ctx) || x == nullptr || x_merged == nullptr) return LITEVGGT_ERR_NULL;
  if (!plan_ok(plan) || plan->owner != ctx || !plan->built) return LITEVGGT_ERR_STALE_PLAN;
  if (!aligned16(x) || !aligned16(x_merged)) return LITEVGGT_ERR_ALIGN;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 5, (cudaStream_t)stream);
    e = launch_merge(ctx, plan, static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(x_merged),
                     (cudaStream_t)stream, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_linear(litevggt_ctx* ctx, const void* a, int64_t m, int64_t k, const void* w, int64_t n,
                                const void* bias, void* out, void* stream) {
  if (!ctx_ok(ctx) || a == nullptr || w == nullptr || out == nullptr) return LITEVGGT_ERR_NULL;
  if (m < 0 || k <= 0 || n <= 0 || k % 64 != 0 || n % 64 != 0 || m > INT32_MAX || n > INT32_MAX || k > INT32_MAX)
    return LITEVGGT_ERR_SHAPE;
  if (!aligned16(a) || !aligned16(w) || !aligned16(out) || (bias != nullptr && !aligned16(bias)))
    return LITEVGGT_ERR_ALIGN;
  int nl = 0;
  cudaError_t e = launch_linear(ctx, static_cast<const __nv_bfloat16*>(a), m, k, static_cast<const __nv_bfloat16*>(w),
                                n, static_cast<const __nv_bfloat16*>(bias), static_cast<__nv_bfloat16*>(out),
                                (cudaStream_t)stream, &nl);
  bump(ctx, nl);
  return cuda_status(e);
}

litevggt_status litevggt_global_attn(litevggt_ctx* ctx, const void* x_merged, int64_t m, const void* w_qkv,
                                     const void* b_qkv, const void* w_o, const void* b_o, void* y_merged,
                                     void* stream) {
  if (!ctx_ok(ctx) || x_merged == nullptr || w_qkv == nullptr || w_o == nullptr || y_merged == nullptr)
    return LITEVGGT_ERR_NULL;
  if (m != ctx->sz.n_merged) return LITEVGGT_ERR_SHAPE;
  if (!aligned16(x_merged) || !aligned16(w_qkv) || !aligned16(w_o) || !aligned16(y_merged) ||
      (b_qkv != nullptr && !aligned16(b_qkv)) || (b_o != nullptr && !aligned16(b_o)))
    return LITEVGGT_ERR_ALIGN;
  const int d = ctx->sz.dim;
  cudaStream_t s = (cudaStream_t)stream;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 6, s);
    e = launch_linear_scaled(ctx, static_cast<const __nv_bfloat16*>(x_merged), m, d,
                             static_cast<const __nv_bfloat16*>(w_qkv), 3 * d, static_cast<const __nv_bfloat16*>(b_qkv), d,
                             2 * d, kKeyScaleLog2e, ctx->ws.qkv, s, &n);
  }
  if (e == cudaSuccess && ctx->cfg.qkv_dtype == 1) {
    StepTimer t(ctx, 14, s);
    e = launch_qkv_quantize(ctx, ctx->ws.qkv, m, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 7, s);
    e = ctx->cfg.qkv_dtype == 1 ? launch_flash_attention_fp8(ctx, m, ctx->ws.attn_o, s, &n)
                                : launch_flash_attention(ctx, ctx->ws.qkv, m, 1, ctx->ws.attn_o, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 8, s);
    e = launch_linear(ctx, ctx->ws.attn_o, m, d, static_cast<const __nv_bfloat16*>(w_o), d,
                      static_cast<const __nv_bfloat16*>(b_o), static_cast<__nv_bfloat16*>(y_merged), s, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_global_attn_ext(litevggt_ctx* ctx, const litevggt_plan* plan, const void* x_merged, int64_t m,
                                         const void* w_qkv, const void* b_qkv, const void* w_o, const void* b_o,
                                         const litevggt_attn_ext* ext, void* y_merged, void* stream) {
  if (!ctx_ok(ctx) || x_merged == nullptr || w_qkv == nullptr || w_o == nullptr || y_merged == nullptr ||
      ext == nullptr)
    return LITEVGGT_ERR_NULL;
  if (m != ctx->sz.n_merged) return LITEVGGT_ERR_SHAPE;
  if (!aligned16(x_merged) || !aligned16(w_qkv) || !aligned16(w_o) || !aligned16(y_merged) ||
      (b_qkv != nullptr && !aligned16(b_qkv)) || (b_o != nullptr && !aligned16(b_o)))
    return LITEVGGT_ERR_ALIGN;
  const void* affine[4] = {ext->q_norm_gamma, ext->q_norm_beta, ext->k_norm_gamma, ext->k_norm_beta};
  int given = 0;
  for (const void* a : affine) given += a != nullptr;
  if (given != 0 && given != 4) return LITEVGGT_ERR_NULL;  // the four vectors come together or not at all
  for (const void* a : affine)
    if (a != nullptr && !aligned16(a)) return LITEVGGT_ERR_ALIGN;
  if (given == 4 && !(ext->norm_eps > 0.0f)) return LITEVGGT_ERR_SHAPE;
  if (ext->rope != 0) {
    if (!(ext->rope_base > 1.0f)) return LITEVGGT_ERR_SHAPE;
    if (plan == nullptr) return LITEVGGT_ERR_NULL;
    if (!plan_ok(plan) || plan->owner != ctx || !plan->built) return LITEVGGT_ERR_STALE_PLAN;
  }
  const int d = ctx->sz.dim;
  cudaStream_t s = (cudaStream_t)stream;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 6, s);
    e = launch_linear(ctx, static_cast<const __nv_bfloat16*>(x_merged), m, d, static_cast<const __nv_bfloat16*>(w_qkv),
                      3 * d, static_cast<const __nv_bfloat16*>(b_qkv), ctx->ws.qkv, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 13, s);
    e = launch_qk_embed(ctx, ctx->ws.qkv, ext->rope != 0 ? plan->kept_idx : nullptr, m,
                        static_cast<const __nv_bfloat16*>(ext->q_norm_gamma),
                        static_cast<const __nv_bfloat16*>(ext->q_norm_beta),
                        static_cast<const __nv_bfloat16*>(ext->k_norm_gamma),
                        static_cast<const __nv_bfloat16*>(ext->k_norm_beta), ext->norm_eps, ext->rope != 0,
                        ext->rope_base, s, &n);
  }
  if (e == cudaSuccess && ctx->cfg.qkv_dtype == 1) {
    StepTimer t(ctx, 14, s);
    e = launch_qkv_quantize(ctx, ctx->ws.qkv, m, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 7, s);
    e = ctx->cfg.qkv_dtype == 1 ? launch_flash_attention_fp8(ctx, m, ctx->ws.attn_o, s, &n)
                                : launch_flash_attention(ctx, ctx->ws.qkv, m, 1, ctx->ws.attn_o, s, &n);
  }
  if (e == cudaSuccess) {
    StepTimer t(ctx, 8, s);
    e = launch_linear(ctx, ctx->ws.attn_o, m, d, static_cast<const __nv_bfloat16*>(w_o), d,
                      static_cast<const __nv_bfloat16*>(b_o), static_cast<__nv_bfloat16*>(y_merged), s, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_layernorm(litevggt_ctx* ctx, const void* x, int64_t rows, const void* gamma, const void* beta,
                                   float eps, void* out, void* stream) {
  if (!ctx_ok(ctx) || x == nullptr || gamma == nullptr || beta == nullptr || out == nullptr) return LITEVGGT_ERR_NULL;
  if (rows < 0 || !(eps > 0.0f)) return LITEVGGT_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta) || !aligned16(out)) return LITEVGGT_ERR_ALIGN;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 10, (cudaStream_t)stream);
    e = launch_layernorm(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(gamma),
                         static_cast<const __nv_bfloat16*>(beta), static_cast<__nv_bfloat16*>(out), rows, eps,
                         (cudaStream_t)stream, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_frame_attn(litevggt_ctx* ctx, const void* x, const void* w_qkv, const void* b_qkv,
                                    const void* w_o, const void* b_o, const void* residual, void* y, void* stream) {
  if (!ctx_ok(ctx) || x == nullptr || w_qkv == nullptr || w_o == nullptr || y == nullptr) return LITEVGGT_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_qkv) || !aligned16(w_o) || !aligned16(y) ||
      (b_qkv != nullptr && !aligned16(b_qkv)) || (b_o != nullptr && !aligned16(b_o)) ||
      (residual != nullptr && !aligned16(residual)))
    return LITEVGGT_ERR_ALIGN;
  litevggt_status st = ensure_block_ws(ctx);
  if (st != LITEVGGT_OK) return st;
  const Sizes& z = ctx->sz;
  const int d = z.dim;
  cudaStream_t s = (cudaStream_t)stream;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 11, s);
    e = launch_linear_scaled(ctx, static_cast<const __nv_bfloat16*>(x), z.n_tokens, d,
                             static_cast<const __nv_bfloat16*>(w_qkv), 3 * d, static_cast<const __nv_bfloat16*>(b_qkv), d,
                             2 * d, kKeyScaleLog2e, ctx->ws.blk_qkv, s, &n);
    if (e == cudaSuccess) e = launch_flash_attention(ctx, ctx->ws.blk_qkv, z.tokens_frame, z.frames, ctx->ws.blk_o, s, &n);
    if (e == cudaSuccess)
      e = launch_linear_mlp(ctx, ctx->ws.blk_o, z.n_tokens, d, static_cast<const __nv_bfloat16*>(w_o), d,
                            static_cast<const __nv_bfloat16*>(b_o), 0, static_cast<const __nv_bfloat16*>(residual),
                            static_cast<__nv_bfloat16*>(y), s, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_mlp(litevggt_ctx* ctx, const void* x, int64_t rows, const void* w1, const void* b1,
                             const void* w2, const void* b2, const void* residual, void* y, void* stream) {
  if (!ctx_ok(ctx) || x == nullptr || w1 == nullptr || w2 == nullptr || y == nullptr) return LITEVGGT_ERR_NULL;
  if (rows < 0 || rows > ctx->sz.n_tokens) return LITEVGGT_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(w1) || !aligned16(w2) || !aligned16(y) || (b1 != nullptr && !aligned16(b1)) ||
      (b2 != nullptr && !aligned16(b2)) || (residual != nullptr && !aligned16(residual)))
    return LITEVGGT_ERR_ALIGN;
  litevggt_status st = ensure_block_ws(ctx);
  if (st != LITEVGGT_OK) return st;
  const int d = ctx->sz.dim;
  cudaStream_t s = (cudaStream_t)stream;
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  const __nv_bfloat16* rb = static_cast<const __nv_bfloat16*>(residual);
  __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(y);
  int n = 0;
  cudaError_t e = cudaSuccess;
  {
    StepTimer t(ctx, 12, s);
    for (long long r0 = 0; r0 < rows && e == cudaSuccess; r0 += kMlpChunkRows) {
      const long long nr = rows - r0 < kMlpChunkRows ? rows - r0 : kMlpChunkRows;
      e = launch_linear_mlp(ctx, xb + r0 * d, nr, d, static_cast<const __nv_bfloat16*>(w1), 4 * d,
                            static_cast<const __nv_bfloat16*>(b1), 1, nullptr, ctx->ws.blk_hidden, s, &n);
      if (e == cudaSuccess)
        e = launch_linear_mlp(ctx, ctx->ws.blk_hidden, nr, 4 * d, static_cast<const __nv_bfloat16*>(w2), d,
                              static_cast<const __nv_bfloat16*>(b2), 0, rb != nullptr ? rb + r0 * d : nullptr,
                              yb + r0 * d, s, &n);
    }
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_unmerge(litevggt_ctx* ctx, const litevggt_plan* plan, const void* y_merged,
                                 const void* residual, void* out, void* stream) {
  if (!ctx_ok(ctx) || y_merged == nullptr || out == nullptr) return LITEVGGT_ERR_NULL;
  if (!plan_ok(plan) || plan->owner != ctx || !plan->built) return LITEVGGT_ERR_STALE_PLAN;
  if (!aligned16(y_merged) || !aligned16(out) || (residual != nullptr && !aligned16(residual)))
    return LITEVGGT_ERR_ALIGN;
  int n = 0;
  cudaError_t e;
  {
    StepTimer t(ctx, 9, (cudaStream_t)stream);
    e = launch_unmerge(ctx, plan, static_cast<const __nv_bfloat16*>(y_merged),
                       static_cast<const __nv_bfloat16*>(residual), static_cast<__nv_bfloat16*>(out),
                       (cudaStream_t)stream, &n);
  }
  bump(ctx, n);
  return cuda_status(e);
}

litevggt_status litevggt_global_layer_host(litevggt_ctx* ctx, litevggt_plan** plan_inout, const float* grad,
                                           const void* x_host, const void* w_qkv, const void* b_qkv, const void* w_o,
                                           const void* b_o, void* out_host, void* stream) {
  if (!ctx_ok(ctx) || plan_inout == nullptr || x_host == nullptr || out_host == nullptr) return LITEVGGT_ERR_NULL;
  if (grad == nullptr) {
    const litevggt_plan* plan = *plan_inout;
    if (!plan_ok(plan) || plan->owner != ctx || !plan->built) return LITEVGGT_ERR_STALE_PLAN;
  }
  litevggt_status st = ensure_staging(ctx);
  if (st != LITEVGGT_OK) return st;
  const Sizes& z = ctx->sz;
  Workspace& ws = ctx->ws;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t bytes = (size_t)z.n_tokens * z.dim * 2;
  cudaError_t e = cudaMemcpyAsync(ws.stage_x, x_host, bytes, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return cuda_status(e);
  if (grad != nullptr) {
    st = litevggt_merge_plan(ctx, ws.stage_x, grad, plan_inout, stream);
    if (st != LITEVGGT_OK) return st;
  }
  const litevggt_plan* plan = *plan_inout;
  st = litevggt_merge(ctx, plan, ws.stage_x, ws.stage_xm, stream);
  if (st == LITEVGGT_OK)
    st = litevggt_global_attn(ctx, ws.stage_xm, z.n_merged, w_qkv, b_qkv, w_o, b_o, ws.stage_ym, stream);
  if (st == LITEVGGT_OK) st = litevggt_unmerge(ctx, plan, ws.stage_ym, ws.stage_x, ws.stage_out, stream);
  if (st != LITEVGGT_OK) return st;
  e = cudaMemcpyAsync(out_host, ws.stage_out, bytes, cudaMemcpyDeviceToHost, s);
  return cuda_status(e);
}

litevggt_status litevggt_global_layer_host_pipelined(litevggt_ctx* ctx, litevggt_plan** plan_inout, const float* grad,
                                                     const void* x_host, const void* w_qkv, const void* b_qkv,
                                                     const void* w_o, const void* b_o, void* out_host, void* stream) {
  if (!ctx_ok(ctx) || plan_inout == nullptr || x_host == nullptr || out_host == nullptr) return LITEVGGT_ERR_NULL;
  if (grad == nullptr) {
    const litevggt_plan* plan = *plan_inout;
    if (!plan_ok(plan) || plan->owner != ctx || !plan->built) return LITEVGGT_ERR_STALE_PLAN;
  }
  litevggt_status st = ensure_host_pipe(ctx);
  if (st != LITEVGGT_OK) return st;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  const Sizes& z = ctx->sz;
  Workspace& ws = ctx->ws;
  HostPipe& hp = ctx->pipe;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t bytes = (size_t)z.n_tokens * z.dim * 2;
  const int slot = (int)(hp.calls & 1ull);
  // copy-in stream: the buffer is free once the unmerge two calls ago has read its residual from it
  cudaError_t e = cudaSuccess;
  if (hp.used[slot]) e = cudaStreamWaitEvent(hp.copy_in, hp.x_free[slot], 0);
  if (e == cudaSuccess) e = cudaMemcpyAsync(hp.x[slot], x_host, bytes, cudaMemcpyHostToDevice, hp.copy_in);
  if (e == cudaSuccess) e = cudaEventRecord(hp.in_ready[slot], hp.copy_in);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(s, hp.in_ready[slot], 0);
  if (e != cudaSuccess) return cuda_status(e);
  if (grad != nullptr) {
    st = litevggt_merge_plan(ctx, hp.x[slot], grad, plan_inout, stream);
    if (st != LITEVGGT_OK) return st;
  }
  const litevggt_plan* plan = *plan_inout;
  st = litevggt_merge(ctx, plan, hp.x[slot], ws.stage_xm, stream);
  if (st == LITEVGGT_OK)
    st = litevggt_global_attn(ctx, ws.stage_xm, z.n_merged, w_qkv, b_qkv, w_o, b_o, ws.stage_ym, stream);
  if (st != LITEVGGT_OK) return st;
  // the output buffer is free once the copy-out two calls ago has drained it
  if (hp.used[slot]) e = cudaStreamWaitEvent(s, hp.out_free[slot], 0);
  if (e != cudaSuccess) return cuda_status(e);
  st = litevggt_unmerge(ctx, plan, ws.stage_ym, hp.x[slot], hp.out[slot], stream);
  if (st != LITEVGGT_OK) return st;
  e = cudaEventRecord(hp.out_ready[slot], s);
  if (e == cudaSuccess) e = cudaEventRecord(hp.x_free[slot], s);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hp.copy_out, hp.out_ready[slot], 0);
  if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, hp.out[slot], bytes, cudaMemcpyDeviceToHost, hp.copy_out);
  if (e == cudaSuccess) e = cudaEventRecord(hp.out_free[slot], hp.copy_out);
  if (e == cudaSuccess) {
    hp.used[slot] = true;
    ++hp.calls;
  }
  return cuda_status(e);
}

litevggt_status litevggt_host_drain(litevggt_ctx* ctx, void* stream) {
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  HostPipe& hp = ctx->pipe;
  if (!hp.created) return LITEVGGT_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LITEVGGT_ERR_CUDA;
  cudaError_t e = cudaSuccess;
  for (int slot = 0; slot < 2 && e == cudaSuccess; ++slot)
    if (hp.used[slot]) e = cudaStreamWaitEvent((cudaStream_t)stream, hp.out_free[slot], 0);
  return cuda_status(e);
}

litevggt_status litevggt_should_refresh(const litevggt_ctx* ctx, const litevggt_plan* plan, int32_t global_layer_idx,
                                        int32_t* yes) {
  if (!ctx_ok(ctx) || yes == nullptr) return LITEVGGT_ERR_NULL;
  if (global_layer_idx < 0) return LITEVGGT_ERR_SHAPE;
  if (plan != nullptr && (!plan_ok(plan) || plan->owner != ctx)) return LITEVGGT_ERR_STALE_PLAN;
  const bool never_built = plan == nullptr || !plan->built;
  *yes = (never_built || global_layer_idx % ctx->cfg.recompute_interval == 0) ? 1 : 0;
  return LITEVGGT_OK;
}

litevggt_status litevggt_plan_export(litevggt_ctx* ctx, const litevggt_plan* plan, int32_t* dst_of, int32_t* size,
                                     int32_t* kept_idx, uint8_t* cls, int32_t* best_dst, float* best_sim, float* var,
                                     float* ga, void* stream) {
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  if (!plan_ok(plan) || plan->owner != ctx || !plan->built) return LITEVGGT_ERR_STALE_PLAN;
  const Sizes& z = ctx->sz;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return cuda_status(cudaGetLastError());
  cudaError_t e = cudaSuccess;
  auto pull = [&](void* dst, const void* src, size_t bytes) {
    if (dst != nullptr && bytes > 0 && e == cudaSuccess) e = cudaMemcpy(dst, src, bytes, cudaMemcpyDeviceToHost);
  };
  pull(dst_of, plan->dst_of, (size_t)z.n_tokens * 4);
  pull(size, plan->size, (size_t)z.n_merged * 4);
  pull(kept_idx, plan->kept_idx, (size_t)z.n_merged * 4);
  pull(cls, ctx->ws.cls, (size_t)z.n_tokens);
  pull(best_dst, plan->best_dst, (size_t)z.n_src * 4);
  pull(best_sim, plan->best_sim, (size_t)z.n_src * 4);
  const size_t map_bytes = (size_t)z.frames * z.patches * 4;
  if (plan->has_maps) {
    pull(var, ctx->ws.var_map, map_bytes);
    pull(ga, ctx->ws.ga_score, map_bytes);
  } else {
    if (var != nullptr) memset(var, 0, map_bytes);
    if (ga != nullptr) memset(ga, 0, map_bytes);
  }
  return cuda_status(e);
}

litevggt_status litevggt_plan_import(litevggt_ctx* ctx, const int32_t* dst_of, litevggt_plan** out) {
  if (!ctx_ok(ctx) || dst_of == nullptr || out == nullptr) return LITEVGGT_ERR_NULL;
  *out = nullptr;
  const Sizes& z = ctx->sz;
  const long long n = z.n_tokens, m = z.n_merged, r = z.n_remove;
  // kept tokens are exactly those mapped to the next unused row, in ascending order
  std::vector<int> kept_idx((size_t)m), size((size_t)m, 0), seg_off((size_t)m + 1, 0), seg_src((size_t)(r > 0 ? r : 1));
  std::vector<char> kept((size_t)n, 0);
  long long rows = 0;
  for (long long i = 0; i < n; ++i) {
    const int d = dst_of[i];
    if (d < 0 || d >= m) return LITEVGGT_ERR_SHAPE;
    if (d == rows) {
      kept[(size_t)i] = 1;
      kept_idx[(size_t)rows++] = (int)i;
    }
    ++size[(size_t)d];
  }
  if (rows != m) return LITEVGGT_ERR_SHAPE;
  for (long long j = 0; j < m; ++j) {
    if (size[(size_t)j] < 1) return LITEVGGT_ERR_SHAPE;
    seg_off[(size_t)j + 1] = seg_off[(size_t)j] + size[(size_t)j] - 1;
  }
  if (seg_off[(size_t)m] != r) return LITEVGGT_ERR_SHAPE;
  {
    std::vector<int> fill(seg_off.begin(), seg_off.end() - 1);
    for (long long i = 0; i < n; ++i)
      if (!kept[(size_t)i]) {
        // a merged token must point at a row whose own token is not itself
        seg_src[(size_t)fill[(size_t)dst_of[i]]++] = (int)i;
      }
  }
  litevggt_plan* p = nullptr;
  litevggt_status st = alloc_plan(ctx, &p);
  if (st != LITEVGGT_OK) return st;
  cudaError_t e = cudaMemcpy(p->dst_of, dst_of, (size_t)n * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(p->size, size.data(), (size_t)m * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(p->kept_idx, kept_idx.data(), (size_t)m * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(p->seg_off, seg_off.data(), (size_t)(m + 1) * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && r > 0) e = cudaMemcpy(p->seg_src, seg_src.data(), (size_t)r * 4, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    litevggt_plan_destroy(p);
    return cuda_status(e);
  }
  p->built = 1;
  p->has_maps = false;
  *out = p;
  return LITEVGGT_OK;
}

litevggt_status litevggt_plan_destroy(litevggt_plan* plan) {
  if (plan == nullptr) return LITEVGGT_OK;
  if (!plan_ok(plan)) return LITEVGGT_ERR_STALE_PLAN;
  if (plan->base != nullptr) {
    cudaDeviceSynchronize();
    cudaFree(plan->base);
    (void)cudaGetLastError();
  }
  plan->magic = 0;
  delete plan;
  return LITEVGGT_OK;
}

litevggt_status litevggt_debug_buffer(litevggt_ctx* ctx, int which, void** dev_ptr, size_t* bytes) {
  if (!ctx_ok(ctx) || dev_ptr == nullptr) return LITEVGGT_ERR_NULL;
  const Sizes& z = ctx->sz;
  if (which == 0) {
    *dev_ptr = ctx->ws.qkv;
    if (bytes) *bytes = (size_t)z.n_merged * 3 * z.dim * 2;
  } else if (which == 1) {
    *dev_ptr = ctx->ws.attn_o;
    if (bytes) *bytes = (size_t)z.n_merged * z.dim * 2;
  } else if (which >= 2 && which <= 5 && ctx->cfg.qkv_dtype == 1) {
    const size_t mp = (size_t)round_up(z.n_merged, 128);
    void* ptrs[4] = {ctx->ws.q8, ctx->ws.k8, ctx->ws.v8t, ctx->ws.qkv_amax};
    const size_t sizes[4] = {(size_t)z.n_merged * z.dim, (size_t)z.n_merged * z.dim, mp * z.dim, 48 * sizeof(float)};
    *dev_ptr = ptrs[which - 2];
    if (bytes) *bytes = sizes[which - 2];
  } else {
    return LITEVGGT_ERR_SHAPE;
  }
  return LITEVGGT_OK;
}

litevggt_status litevggt_poll_device_status(litevggt_ctx* ctx, void* stream) {
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  cudaStream_t s = (cudaStream_t)stream;
  uint32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, ctx->ws.status, sizeof(word), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws.status, 0, sizeof(word), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_status(e);
  if (word & kStatusTimeout) return LITEVGGT_ERR_DEVICE_TIMEOUT;
  if (word & kStatusBounds) return LITEVGGT_ERR_DEVICE_BOUNDS;
  return LITEVGGT_OK;
}

litevggt_status litevggt_selftest_bounded_wait(litevggt_ctx* ctx, int64_t limit_cycles, uint32_t* outcome, void* stream) {
  if (!ctx_ok(ctx)) return LITEVGGT_ERR_NULL;
  if (limit_cycles < 1000 || limit_cycles > (1ll << 32)) return LITEVGGT_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)stream;
  uint32_t* dev_outcome = ctx->ws.status + 1;  // second word of the status block
  int n = 0;
  cudaError_t e = launch_bounded_wait_selftest(ctx, limit_cycles, dev_outcome, s, &n);
  bump(ctx, n);
  if (e != cudaSuccess) return cuda_status(e);
  if (outcome != nullptr) {
    e = cudaMemcpyAsync(outcome, dev_outcome, sizeof(uint32_t), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  }
  return cuda_status(e);
}

litevggt_status litevggt_launch_count(const litevggt_ctx* ctx, int64_t* launches) {
  if (!ctx_ok(ctx) || launches == nullptr) return LITEVGGT_ERR_NULL;
  *launches = ctx->launches;
  return LITEVGGT_OK;
}

const char* litevggt_status_string(litevggt_status s) {
  switch (s) {
    case LITEVGGT_OK: return "ok";
    case LITEVGGT_ERR_NULL: return "null or invalid handle/pointer";
    case LITEVGGT_ERR_BAD_CONFIG: return "bad or unsupported config";
    case LITEVGGT_ERR_SHAPE: return "shape mismatch";
    case LITEVGGT_ERR_ALIGN: return "tensor not 16-byte aligned";
    case LITEVGGT_ERR_ALLOC: return "allocation failed";
    case LITEVGGT_ERR_CUDA: return "CUDA call failed";
    case LITEVGGT_ERR_ARCH: return "device is not sm_100";
    case LITEVGGT_ERR_STALE_PLAN: return "stale or foreign plan";
    case LITEVGGT_ERR_DEVICE_TIMEOUT: return "device-side bounded wait timed out";
    case LITEVGGT_ERR_DEVICE_BOUNDS: return "device-side index out of range";
  }
  return "unknown status";
}

}  // extern "C"
