// Geometric-importance scoring and anchor selection (Sec. 3.4, "Geometry-aware Feature
// Map" and "GA Token Partitioning"): Grad map, Var map, GA map, token classes and the
// ascending src / anchor token lists.  All of this is bandwidth- or latency-bound work;
// no tensor cores are involved.
#include "common.cuh"
#include "runtime.h"

namespace lv {

// ----------------------------------------------------------------------------------------
// Grad map.  One CTA per (frame, patch row).  Phase 1: the 16 grey rows it needs (14 + one halo
// row above and below, replicate padding) are staged in shared memory, one warp per image row,
// two pixels per load when the width is even.  Phase 2: one thread per pixel column walks down
// the 16 rows with the separable form of the Sobel pair - per row the horizontal difference
// r - l and the horizontal smoothing l + 2c + r, kept for the last three rows - and adds up the
// 14 magnitudes of its column.  Phase 3: one thread per patch adds its 14 column sums.  All sums
// run in a fixed order.
constexpr int kGradThreads = 256;

__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kGradThreads)
grad_map_kernel(const float* __restrict__ images, float* __restrict__ grad, int grid_h, int grid_w, int patch) {
  extern __shared__ float grey[];  // [(patch+2)][w+2], then [w] column sums
  const int f = blockIdx.y;
  const int py = blockIdx.x;
  const int h = grid_h * patch, w = grid_w * patch;
  const int pitch = w + 2;
  const int rows = patch + 2;
  float* colsum = grey + rows * pitch;
  const size_t plane = (size_t)h * w;
  const float* img = images + (size_t)f * 3 * plane;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = warp; r < rows; r += kGradThreads / 32) {
    int y = py * patch - 1 + r;
    y = y < 0 ? 0 : (y >= h ? h - 1 : y);
    const float* p0 = img + (size_t)y * w;
    float* g = grey + r * pitch + 1;
    if ((w & 1) == 0) {  // rows are 8-byte aligned
      const float2* q0 = reinterpret_cast<const float2*>(p0);
      const float2* q1 = reinterpret_cast<const float2*>(p0 + plane);
      const float2* q2 = reinterpret_cast<const float2*>(p0 + 2 * plane);
      const int half_w = w >> 1;
#pragma unroll 4
      for (int xh = lane; xh < half_w; xh += 32) {
        const float2 a = __ldg(q0 + xh), b = __ldg(q1 + xh), c = __ldg(q2 + xh);
        g[2 * xh] = (a.x + b.x + c.x) / 3.0f;
        g[2 * xh + 1] = (a.y + b.y + c.y) / 3.0f;
      }
    } else {
#pragma unroll 4
      for (int x = lane; x < w; x += 32) g[x] = (__ldg(p0 + x) + __ldg(p0 + plane + x) + __ldg(p0 + 2 * plane + x)) / 3.0f;
    }
    __syncwarp();
    if (lane == 0) {
      g[-1] = g[0];
      g[w] = g[w - 1];
    }
  }
  __syncthreads();
  for (int col = threadIdx.x; col < w; col += kGradThreads) {
    const float* p = grey + col;  // p[0], p[1], p[2] = left, centre, right of this column in row 0
    float d0 = p[2] - p[0], s0 = fmaf(2.0f, p[1], p[0] + p[2]);
    p += pitch;
    float d1 = p[2] - p[0], s1 = fmaf(2.0f, p[1], p[0] + p[2]);
    float acc = 0.0f;
    for (int r = 0; r < patch; ++r) {
      p += pitch;
      const float d2 = p[2] - p[0], s2 = fmaf(2.0f, p[1], p[0] + p[2]);
      const float gx = fmaf(2.0f, d1, d0 + d2);
      const float gy = s2 - s0;
      acc += sqrt_approx(fmaf(gx, gx, gy * gy));
      d0 = d1; s0 = s1; d1 = d2; s1 = s2;
    }
    colsum[col] = acc;
  }
  __syncthreads();
  for (int px = threadIdx.x; px < grid_w; px += kGradThreads) {
    float acc = 0.0f;
    for (int c = 0; c < patch; ++c) acc += colsum[px * patch + c];
    grad[((size_t)f * grid_h + py) * grid_w + px] = acc / (float)(patch * patch);
  }
}

cudaError_t launch_grad_map(const litevggt_ctx* ctx, const float* images, float* grad, cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const int patch = ctx->cfg.patch_px;
  const size_t smem = ((size_t)(patch + 2) * (z.grid_w * patch + 2) + (size_t)z.grid_w * patch) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(grad_map_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  grad_map_kernel<<<dim3(z.grid_h, z.frames), kGradThreads, smem, s>>>(images, grad, z.grid_h, z.grid_w, patch);
  ++*launches;
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------
// Var map.  One CTA per (frame, grid row, quarter of the channels).  A single thread issues
// two or three TMA loads - the 256-channel slices of the (clipped) 3 grid rows around the
// CTA's row - so the whole 57 KB working set of the CTA is in flight at once; with several
// CTAs per SM that is what keeps HBM busy.  Thread t then owns channels 2(t%128), 2(t%128)+1
// and slides along its quarter of the row: per column it forms the sums of x - x0 and (x - x0)^2 over the window rows
// (x0 = the row's first token, per channel, which removes a common offset before squaring),
// a window is the sum of up to three columns, and the population variance follows as
// E[d^2] - E[d]^2 in fp32.  The per-position sums over the CTA's 256 channels are reduced in
// a fixed order and written to this quarter's plane; a second tiny kernel adds the four
// planes in a fixed order, so the map is deterministic.
constexpr int kVarThreads = 512;   // 128 channel pairs x 4 segments of the row
constexpr int kVarSegments = kVarThreads / 128;
constexpr int kVarChannels = 256;  // per CTA
constexpr int kVarMaxW = 64;

struct VarControl {
  uint64_t bar;
  uint32_t abort_flag;
  uint32_t landed;
};
// dynamic shared memory: [control, 128 B][tile: nr x grid_w x 256 bf16][partial: grid_w x 32 fp32]
__host__ __device__ inline size_t var_smem_bytes(int grid_w) {
  return 128 + (size_t)3 * grid_w * kVarChannels * 2 + (size_t)grid_w * 32 * sizeof(float) + 128;
}

__global__ void __launch_bounds__(kVarThreads)
var_map_kernel(const __grid_constant__ CUtensorMap tmap_x, float* __restrict__ var_parts, int frames, int grid_h,
               int grid_w, int n_special, uint32_t* status) {
  extern __shared__ uint8_t var_smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(var_smem_raw) + 127) & ~uintptr_t(127));
  VarControl* ctrl = reinterpret_cast<VarControl*>(base);
  uint8_t* tile = base + 128;
  const uint32_t row_bytes = (uint32_t)grid_w * kVarChannels * 2;  // one grid row of 256-channel slices
  float* partial = reinterpret_cast<float*>(tile + 3 * (size_t)row_bytes);  // [grid_w][32]
  const int quarter = blockIdx.x, py = blockIdx.y, f = blockIdx.z;
  const int tokens_frame = grid_h * grid_w + n_special;
  const int r0 = py > 0 ? py - 1 : 0;
  const int r1 = py < grid_h - 1 ? py + 1 : grid_h - 1;
  const int nr = r1 - r0 + 1;
  if (threadIdx.x == 0) {
    mbar_init(&ctrl->bar, 1);
    ctrl->abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    mbar_expect_tx(&ctrl->bar, row_bytes * nr);
    for (int r = 0; r < nr; ++r) {
      const int token = f * tokens_frame + n_special + (r0 + r) * grid_w;
      tma_load_2d(tile + (size_t)r * row_bytes, &tmap_x, &ctrl->bar, quarter * kVarChannels, token);
    }
  }
  // Only the issuing thread polls the barrier; everyone else parks at the CTA barrier, which costs
  // no issue slots (hundreds of polling threads would starve the CTAs that are computing).
  if (threadIdx.x == 0) {
    const WaitCtl ctl{&ctrl->abort_flag, status};
    bool ok = mbar_wait(&ctrl->bar, 0, ctl);
    if (!ok) {
      // the copies are still in flight: they must finish before the shared memory is given up
      const long long t0 = clock64();
      while (!mbar_try_wait(&ctrl->bar, 0)) {
        if (clock64() - t0 > kTimeoutCycles) break;
      }
    }
    ctrl->landed = ok ? 1u : 0u;
  }
  __syncthreads();
  const bool landed = ctrl->landed != 0u;
  const int lane = threadIdx.x & 31;
  if (landed) {
    const int pair = threadIdx.x & 127, seg = threadIdx.x >> 7;
    const int seg_len = (grid_w + kVarSegments - 1) / kVarSegments;
    const int px_begin = seg * seg_len, px_end = min(grid_w, px_begin + seg_len);
    const uint32_t* words = reinterpret_cast<const uint32_t*>(tile) + pair;  // this thread's channel pair
    const int pitch = kVarChannels / 2;   // 32-bit words per token slice
    const int row_words = grid_w * pitch; // per grid row
    const uint32_t w0 = words[(py - r0) * row_words];
    const float2 x0 = make_float2(bf16_lo(w0), bf16_hi(w0));
    const bool three = nr == 3;  // CTA-uniform
    // column sums of d and d^2 over the window rows, for the two channels of this thread (packed)
    auto column = [&](int px, float2& s1, float2& s2) {
      if (px < 0 || px >= grid_w) {
        s1 = s2 = make_float2(0.0f, 0.0f);
        return;
      }
      const uint32_t* p = words + px * pitch;
      const uint32_t wa = p[0], wb = p[row_words];
      const float2 da = make_float2(bf16_lo(wa) - x0.x, bf16_hi(wa) - x0.y);
      const float2 db = make_float2(bf16_lo(wb) - x0.x, bf16_hi(wb) - x0.y);
      s1 = __fadd2_rn(da, db);
      s2 = __ffma2_rn(db, db, __fmul2_rn(da, da));
      if (three) {
        const uint32_t wc = p[2 * row_words];
        const float2 dc = make_float2(bf16_lo(wc) - x0.x, bf16_hi(wc) - x0.y);
        s1 = __fadd2_rn(s1, dc);
        s2 = __ffma2_rn(dc, dc, s2);
      }
    };
    const float inv_edge = 1.0f / (float)(nr * (grid_w > 1 ? 2 : 1)), inv_mid = 1.0f / (float)(nr * 3);
    // one output position from the three column sums around it
    auto emit = [&](int px, const float2& a1, const float2& a2, const float2& b1, const float2& b2, const float2& c1,
                    const float2& c2) {
      const float inv_n = (px == 0 || px == grid_w - 1) ? inv_edge : inv_mid;
      const float2 inv2 = make_float2(inv_n, inv_n);
      const float2 mean = __fmul2_rn(__fadd2_rn(__fadd2_rn(a1, b1), c1), inv2);
      const float2 msq = __fmul2_rn(__fadd2_rn(__fadd2_rn(a2, b2), c2), inv2);
      const float2 v = __ffma2_rn(make_float2(-mean.x, -mean.y), mean, msq);
      float tot = fmaxf(v.x, 0.0f) + fmaxf(v.y, 0.0f);
      // fixed-order partial reduction over groups of four lanes
      tot += __shfl_xor_sync(0xffffffffu, tot, 1);
      tot += __shfl_xor_sync(0xffffffffu, tot, 2);
      if ((lane & 3) == 0) partial[px * 32 + (pair >> 2)] = tot;
    };
    float2 a1, a2, b1, b2, c1, c2;
    column(px_begin - 1, a1, a2);
    column(px_begin, b1, b2);
    // three positions per trip, so the column sums rotate through fixed registers
    for (int px = px_begin; px < px_end; px += 3) {
      column(px + 1, c1, c2);
      emit(px, a1, a2, b1, b2, c1, c2);
      if (px + 1 < px_end) {
        column(px + 2, a1, a2);
        emit(px + 1, b1, b2, c1, c2, a1, a2);
      }
      if (px + 2 < px_end) {
        column(px + 3, b1, b2);
        emit(px + 2, c1, c2, a1, a2, b1, b2);
      }
    }
  }
  __syncthreads();
  if (!landed) return;
  const int warp = threadIdx.x >> 5;
  float* out = var_parts + ((size_t)quarter * frames + f) * grid_h * grid_w + (size_t)py * grid_w;
  for (int px = warp; px < grid_w; px += kVarThreads / 32) {
    float acc = partial[px * 32 + lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) out[px] = acc;
  }
}

__global__ void var_sum_kernel(const float* __restrict__ parts, float* __restrict__ var, long long count) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) var[i] = (((parts[i] + parts[count + i]) + parts[2 * count + i]) + parts[3 * count + i]) / 1024.0f;
}

cudaError_t launch_var_map(const litevggt_ctx* ctx, const __nv_bfloat16* x, float* var_parts, float* var,
                           cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  CUtensorMap tmap;
  if (!make_tmap_bf16_2d_linear(ctx->encode_tiled, &tmap, x, 1024, (uint64_t)z.n_tokens, 1024, kVarChannels,
                                (uint32_t)z.grid_w))
    return cudaErrorInvalidValue;
  const int smem = (int)var_smem_bytes(z.grid_w);
  cudaError_t e = cudaFuncSetAttribute(var_map_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  var_map_kernel<<<dim3(4, z.grid_h, z.frames), kVarThreads, smem, s>>>(tmap, var_parts, z.frames, z.grid_h, z.grid_w,
                                                                        z.n_special, ctx->ws.status);
  ++*launches;
  const long long count = (long long)z.frames * z.patches;
  var_sum_kernel<<<(unsigned)((count + 255) / 256), 256, 0, s>>>(var_parts, var, count);
  ++*launches;
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------
// GA map + partition.  One CTA per frame.  Per-frame min-max normalisation of both maps,
// weighted sum, segmented (per cell) argmin for the anchors, then an exact top-k of the
// remaining patches by rank counting (rank = number of candidates that beat this one,
// ties towards the lower index); P <= a few thousand, so all of it lives in shared memory.
constexpr int kPartThreads = 512;

__device__ __forceinline__ float block_reduce_minmax(float v, bool is_max, float* scratch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, other) : fminf(v, other);
  }
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float r = scratch[0];
  for (int i = 1; i < kPartThreads / 32; ++i) r = is_max ? fmaxf(r, scratch[i]) : fminf(r, scratch[i]);
  return r;
}

__global__ void __launch_bounds__(kPartThreads)
partition_kernel(const float* __restrict__ grad, const float* __restrict__ var, float* __restrict__ ga,
                 uint8_t* __restrict__ cls, int grid_h, int grid_w, int n_special, int n_ga, int cell_h, int cell_w,
                 float alpha, float beta) {
  extern __shared__ float part_smem[];
  const int p_count = grid_h * grid_w;
  float* score = part_smem;                                        // [P]
  uint8_t* is_dst = reinterpret_cast<uint8_t*>(score + p_count);   // [P]
  __shared__ float scratch[kPartThreads / 32];
  const int f = blockIdx.x;
  const float* g = grad + (size_t)f * p_count;
  const float* v = var + (size_t)f * p_count;
  float gmin = INFINITY, gmax = -INFINITY, vmin = INFINITY, vmax = -INFINITY;
  for (int p = threadIdx.x; p < p_count; p += kPartThreads) {
    gmin = fminf(gmin, g[p]); gmax = fmaxf(gmax, g[p]);
    vmin = fminf(vmin, v[p]); vmax = fmaxf(vmax, v[p]);
  }
  gmin = block_reduce_minmax(gmin, false, scratch);
  gmax = block_reduce_minmax(gmax, true, scratch);
  vmin = block_reduce_minmax(vmin, false, scratch);
  vmax = block_reduce_minmax(vmax, true, scratch);
  const float gden = gmax - gmin + 1e-6f, vden = vmax - vmin + 1e-6f;
  for (int p = threadIdx.x; p < p_count; p += kPartThreads) {
    const float sc = alpha * ((g[p] - gmin) / gden) + beta * ((v[p] - vmin) / vden);
    score[p] = sc;
    is_dst[p] = 0;
    ga[(size_t)f * p_count + p] = sc;
  }
  uint8_t* out = cls + (size_t)f * (p_count + n_special);
  for (int t = threadIdx.x; t < n_special; t += kPartThreads) out[t] = LITEVGGT_CLS_PROTECTED;
  out += n_special;
  if (f == 0) {  // the first frame's patches are all anchors
    for (int p = threadIdx.x; p < p_count; p += kPartThreads) out[p] = LITEVGGT_CLS_DST;
    return;
  }
  __syncthreads();
  const int cells_w = (grid_w + cell_w - 1) / cell_w, cells_h = (grid_h + cell_h - 1) / cell_h;
  for (int c = threadIdx.x; c < cells_w * cells_h; c += kPartThreads) {
    const int cy = (c / cells_w) * cell_h, cx = (c % cells_w) * cell_w;
    int best = -1;
    float best_v = INFINITY;
    for (int yy = cy; yy < min(grid_h, cy + cell_h); ++yy)
      for (int xx = cx; xx < min(grid_w, cx + cell_w); ++xx) {
        const float sv = score[yy * grid_w + xx];
        if (best < 0 || sv < best_v) { best = yy * grid_w + xx; best_v = sv; }
      }
    is_dst[best] = 1;
  }
  __syncthreads();
  for (int p = threadIdx.x; p < p_count; p += kPartThreads) {
    uint8_t c = LITEVGGT_CLS_DST;
    if (!is_dst[p]) {
      const float sp = score[p];
      int rank = 0;
      for (int q = 0; q < p_count; ++q) {
        const float sq = score[q];
        rank += (!is_dst[q] && (sq > sp || (sq == sp && q < p))) ? 1 : 0;
      }
      c = rank < n_ga ? LITEVGGT_CLS_GA : LITEVGGT_CLS_SRC;
    }
    out[p] = c;
  }
}

cudaError_t launch_partition(const litevggt_ctx* ctx, const float* grad, const float* var, float* ga, uint8_t* cls,
                             cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const size_t smem = (size_t)z.patches * (sizeof(float) + 1) + 16;
  cudaError_t e = cudaFuncSetAttribute(partition_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  partition_kernel<<<z.frames, kPartThreads, smem, s>>>(grad, var, ga, cls, z.grid_h, z.grid_w, z.n_special,
                                                        z.n_ga_frame, ctx->cfg.cell_h, ctx->cfg.cell_w,
                                                        ctx->cfg.alpha, ctx->cfg.beta);
  ++*launches;
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------
// Token lists.  One CTA per frame: src / anchor tokens of the frame in ascending token
// order, written at the offsets the per-frame class counts imply.  A frame whose counts
// differ from the expected ones (possible only with a caller-supplied partition) is
// flagged in the status word; writes never leave the frame's slot.
constexpr int kListThreads = 256;

__global__ void __launch_bounds__(kListThreads)
build_lists_kernel(const uint8_t* __restrict__ cls, int* __restrict__ src_list, int* __restrict__ dst_list,
                   int p_count, int n_special, int n_src_frame, int n_dst_frame, uint32_t* status) {
  __shared__ int warp_src[kListThreads / 32], warp_dst[kListThreads / 32];
  const int f = blockIdx.x;
  const int tokens_frame = p_count + n_special;
  const int token0 = f * tokens_frame;
  const int exp_src = f == 0 ? 0 : n_src_frame;
  const int exp_dst = f == 0 ? p_count : n_dst_frame;
  const long long src_base = f == 0 ? 0 : (long long)(f - 1) * n_src_frame;
  const long long dst_base = f == 0 ? 0 : (long long)p_count + (long long)(f - 1) * n_dst_frame;
  const int per = (tokens_frame + kListThreads - 1) / kListThreads;
  const int t0 = threadIdx.x * per, t1 = min(tokens_frame, t0 + per);
  int ns = 0, nd = 0;
  for (int t = t0; t < t1; ++t) {
    const uint8_t c = cls[token0 + t];
    ns += c == LITEVGGT_CLS_SRC;
    nd += c == LITEVGGT_CLS_DST;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int xs = ns, xd = nd;  // inclusive warp scans
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, xs, o), b = __shfl_up_sync(0xffffffffu, xd, o);
    if (lane >= o) { xs += a; xd += b; }
  }
  if (lane == 31) { warp_src[warp] = xs; warp_dst[warp] = xd; }
  __syncthreads();
  int off_s = xs - ns, off_d = xd - nd, tot_s = 0, tot_d = 0;
  for (int i = 0; i < kListThreads / 32; ++i) {
    if (i < warp) { off_s += warp_src[i]; off_d += warp_dst[i]; }
    tot_s += warp_src[i];
    tot_d += warp_dst[i];
  }
  if (tot_s != exp_src || tot_d != exp_dst) {
    if (threadIdx.x == 0) atomicOr(status, kStatusBounds);
  }
  for (int t = t0; t < t1; ++t) {
    const uint8_t c = cls[token0 + t];
    if (c == LITEVGGT_CLS_SRC) {
      if (off_s < exp_src) src_list[src_base + off_s] = token0 + t;
      ++off_s;
    } else if (c == LITEVGGT_CLS_DST) {
      if (off_d < exp_dst) dst_list[dst_base + off_d] = token0 + t;
      ++off_d;
    }
  }
  // a short frame (flagged above) still gets valid token indices in its unused slots
  for (int i = tot_s + (int)threadIdx.x; i < exp_src; i += kListThreads) src_list[src_base + i] = token0;
  for (int i = tot_d + (int)threadIdx.x; i < exp_dst; i += kListThreads) dst_list[dst_base + i] = token0;
}

cudaError_t launch_build_lists(const litevggt_ctx* ctx, const uint8_t* cls, int* src_list, int* dst_list,
                               cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  build_lists_kernel<<<z.frames, kListThreads, 0, s>>>(cls, src_list, dst_list, z.patches, z.n_special,
                                                       z.n_src_frame, z.n_dst_frame, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
