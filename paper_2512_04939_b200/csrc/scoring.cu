// Geometric-importance scoring and anchor selection (Sec. 3.4, "Geometry-aware Feature
// Map" and "GA Token Partitioning"): Grad map, Var map, GA map, token classes and the
// ascending src / anchor token lists.  All of this is bandwidth- or latency-bound work;
// no tensor cores are involved.
#include "common.cuh"
#include "runtime.h"

namespace lv {

// ----------------------------------------------------------------------------------------
// Grad map.  A warp owns a vertical strip of the image - as many whole patches as fit into 30 pixel
// columns, plus one halo column on either side (lane = pixel column, replicate padding by clamping
// the coordinate) - over a block of 7 patch rows, and walks down it one image row per step: three
// coalesced 4-byte loads per lane (R, G, B), the grey value, its left and right neighbours by
// shuffle, the separable Sobel pair (per row the horizontal difference r - l and the horizontal
// smoothing l + 2c + r, kept for the last three rows), the magnitude, a running sum per column.  At
// the bottom of a patch row the columns of a patch are added by a shuffle tree and one lane writes
// the patch mean.  Rows are loaded three steps ahead (deeper measured slower); there is no shared
// memory and no barrier.
constexpr int kGradThreads = 128;
#ifndef LV_GRAD_PATCH_ROWS
#define LV_GRAD_PATCH_ROWS 7
#endif
#ifndef LV_GRAD_AHEAD
#define LV_GRAD_AHEAD 3
#endif
constexpr int kGradPatchRows = LV_GRAD_PATCH_ROWS;  // patch rows per warp
constexpr int kGradAhead = LV_GRAD_AHEAD;           // image rows in flight

__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kGradThreads)
grad_map_kernel(const float* __restrict__ images, float* __restrict__ grad, int grid_h, int grid_w, int patch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pps = 30 / patch;  // patches per strip (patch <= 30)
  const int strips = (grid_w + pps - 1) / pps;
  const int strip = blockIdx.x * (kGradThreads / 32) + warp;
  if (strip >= strips) return;  // whole warp; nothing below synchronises across warps
  const int f = blockIdx.z;
  const int pr0 = blockIdx.y * kGradPatchRows;
  const int pr1 = min(grid_h, pr0 + kGradPatchRows);
  const int h = grid_h * patch, w = grid_w * patch;
  const size_t plane = (size_t)h * w;
  int x = strip * pps * patch - 1 + lane;
  x = x < 0 ? 0 : (x >= w ? w - 1 : x);
  const float* col = images + (size_t)f * 3 * plane + x;
  // lanes 1 .. pps * patch carry the strip's own pixel columns
  const bool own = lane >= 1 && lane <= pps * patch;
  const int seg = own ? (lane - 1) / patch : 0;
  const int in_seg = own ? (lane - 1) - seg * patch : patch;
  const int patch_x = strip * pps + seg;
  const bool writer = own && in_seg == 0 && patch_x < grid_w;

  const float inv_area = 1.0f / (float)(patch * patch);
  const int y_first = pr0 * patch - 1;             // halo row above (clamped when it is outside)
  const int count = (pr1 - pr0) * patch + 2;       // rows visited, halo rows included
  float q[kGradAhead][3];
  auto load_row = [&](int i, float (&dst)[3]) {
    int y = y_first + i;
    y = y < 0 ? 0 : (y >= h ? h - 1 : y);
    const float* p = col + (size_t)y * w;
    dst[0] = __ldg(p);
    dst[1] = __ldg(p + plane);
    dst[2] = __ldg(p + 2 * plane);
  };
#pragma unroll
  for (int k = 0; k < kGradAhead; ++k)
    if (k < count) load_row(k, q[k]);
  float d0 = 0.0f, s0 = 0.0f, d1 = 0.0f, s1 = 0.0f, acc = 0.0f;
  int rows_done = 0, pr = pr0;
  for (int i0 = 0; i0 < count; i0 += kGradAhead) {
#pragma unroll
    for (int k = 0; k < kGradAhead; ++k) {
      const int i = i0 + k;
      if (i >= count) break;  // warp-uniform
      const float g = (q[k][0] + q[k][1] + q[k][2]) * (1.0f / 3.0f);
      if (i + kGradAhead < count) load_row(i + kGradAhead, q[k]);
      const float l = __shfl_up_sync(0xffffffffu, g, 1), r = __shfl_down_sync(0xffffffffu, g, 1);
      const float d = r - l, s = fmaf(2.0f, g, l + r);
      if (i >= 2) {  // rows i-2, i-1, i are in hand: the pixel of row i-1
        const float gx = fmaf(2.0f, d1, d0 + d);
        const float gy = s - s0;
        acc += sqrt_approx(fmaf(gx, gx, gy * gy));
        if (++rows_done == patch) {
          // bottom of a patch row: add the columns of each patch, lowest lane of the patch writes
          float v = own ? acc : 0.0f;
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
            const float t = __shfl_down_sync(0xffffffffu, v, off);
            if (in_seg + off < patch) v += t;
          }
          if (writer) grad[((size_t)f * grid_h + pr) * grid_w + patch_x] = v * inv_area;
          acc = 0.0f;
          rows_done = 0;
          ++pr;
        }
      }
      d0 = d1; s0 = s1; d1 = d; s1 = s;
    }
  }
}

cudaError_t launch_grad_map(const litevggt_ctx* ctx, const float* images, float* grad, cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const int patch = ctx->cfg.patch_px;
  const int pps = 30 / patch;
  const int strips = (z.grid_w + pps - 1) / pps;
  const dim3 grid((unsigned)((strips + kGradThreads / 32 - 1) / (kGradThreads / 32)),
                  (unsigned)((z.grid_h + kGradPatchRows - 1) / kGradPatchRows), (unsigned)z.frames);
  grad_map_kernel<<<grid, kGradThreads, 0, s>>>(images, grad, z.grid_h, z.grid_w, patch);
  ++*launches;
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------
// Var map.  Summed over the channels, the population variance of a window W of n tokens is
//     sum_c Var_c = (1/n) sum_{j in W} |d_j|^2  -  (1/n^2) sum_c (sum_{j in W} d_jc)^2,   d_j = x_j - x0,
// for any fixed x0 (here the frame's first patch token, which takes a common offset out before
// anything is squared).  So only the per-channel box sums of d are needed, plus a box sum of the
// scalar |d_j|^2 - not a second per-channel box filter.
//
// A warp owns 16 channels of a block of 30 grid rows (+ one halo row on either side) and walks along
// the rows, one grid column per step.  The column's 32 tokens (32 bytes each) arrive in the warp's own
// ring in shared memory by asynchronous copies, two lanes per token, kVarDepth columns ahead; rows
// outside the grid are filled with x0, so they contribute d = 0 and the clipped window needs no
// special case.  Lane = grid row: it reads its own token and the ones above and below from the ring
// (48-byte row pitch: conflict-free 16-byte reads), forms the vertical sums of d and of |d|^2, and
// keeps the last three columns in registers, from which the window sums of the column before follow.
// Scattered 16-byte global loads and two shuffles per channel cost this kernel's first version
// (lane loads its own token, neighbours by shuffle) three times the L1 wavefronts.  No barrier
// inside the walk; only __syncwarp around the ring.  A warp makes four such passes (64 channels),
// adding its results up in its own shared-memory rows; the four warps of a CTA cover a quarter of
// the channels and are added in a fixed order into that quarter's plane, and var_sum_kernel adds the
// four planes, so the map is deterministic.
#ifndef LV_VAR_OCC
#define LV_VAR_OCC 4
#endif
#ifndef LV_VAR_DEPTH
#define LV_VAR_DEPTH 4
#endif
constexpr int kVarThreads = 128;
constexpr int kVarWarps = kVarThreads / 32;
constexpr int kVarChannels = 256;     // per CTA
constexpr int kVarPassChannels = 16;  // per warp pass
constexpr int kVarRowsPerBlock = 30;
constexpr int kVarMaxW = 64;
constexpr int kVarDepth = LV_VAR_DEPTH;  // grid columns in flight
constexpr int kVarRowPitch = 48;         // bytes per token in the ring: 32 of data + 16 against bank conflicts
constexpr int kVarSlotBytes = 32 * kVarRowPitch;
// dynamic shared memory per warp: the ring [depth][32 rows][48 B], then this warp's results
// [32 lanes][grid_w + 1]
__host__ __device__ inline size_t var_warp_smem_bytes(int grid_w) {
  return (size_t)kVarDepth * kVarSlotBytes + (size_t)32 * (grid_w + 1) * sizeof(float);
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory");
}

struct VarColumn {
  float2 s[kVarPassChannels / 2];  // vertical 3-sum of d, per channel (pairs: packed fp32 arithmetic)
  float q;                         // vertical 3-sum of |d|^2
};

__global__ void __launch_bounds__(kVarThreads, LV_VAR_OCC)
var_map_kernel(const __nv_bfloat16* __restrict__ x, float* __restrict__ var_parts, int frames, int grid_h, int grid_w,
               int n_special) {
  extern __shared__ __align__(16) uint8_t var_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t warp_bytes = var_warp_smem_bytes(grid_w);
  uint8_t* ring = var_smem + warp * warp_bytes;
  const int acc_pitch = grid_w + 1;
  float* acc = reinterpret_cast<float*>(ring + kVarDepth * kVarSlotBytes) + lane * acc_pitch;  // this lane's results
  const int quarter = blockIdx.x, f = blockIdx.z;
  const int row0 = blockIdx.y * kVarRowsPerBlock - 1;  // grid row of lane 0 (a halo row)
  const int row = row0 + lane;
  const bool row_valid = row >= 0 && row < grid_h;
  const bool emits = row_valid && lane >= 1 && lane <= kVarRowsPerBlock;
  const int tokens_frame = grid_h * grid_w + n_special;
  const __nv_bfloat16* frame = x + ((size_t)f * tokens_frame + n_special) * 1024;
  const float inv_rows = 1.0f / (float)(1 + (row > 0 ? 1 : 0) + (row < grid_h - 1 ? 1 : 0));
  // as a copier, this lane moves 16 bytes of two tokens per column: rows row0 + lane/2 and + 16
  const int half = lane & 1;
  const int crow_a = row0 + (lane >> 1), crow_b = crow_a + 16;
  const bool cvalid_a = crow_a >= 0 && crow_a < grid_h, cvalid_b = crow_b >= 0 && crow_b < grid_h;
  // lanes 0 and 31 have no row above / below in the ring: they read their own row instead; what they
  // compute is never emitted
  const int up = lane > 0 ? lane - 1 : lane, dn = lane < 31 ? lane + 1 : lane;

  for (int pass = 0; pass < kVarChannels / kVarWarps / kVarPassChannels; ++pass) {
    // In one pass the four warps take the four 32-byte sectors of the same 128-byte lines, so a line
    // comes from HBM once and the other three warps find it in cache.
    const int ch = quarter * kVarChannels + (pass * kVarWarps + warp) * kVarPassChannels;
    const __nv_bfloat16* x0_ptr = frame + ch;  // first patch token of the frame, this pass's channels
    float2 x0[kVarPassChannels / 2], x0_3[kVarPassChannels / 2];
    {
      const uint4* p0 = reinterpret_cast<const uint4*>(x0_ptr);
      const uint4 a = __ldg(p0), b = __ldg(p0 + 1);
      const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        x0[i] = make_float2(bf16_lo(w[i]), bf16_hi(w[i]));
        x0_3[i] = make_float2(-3.0f * x0[i].x, -3.0f * x0[i].y);
      }
    }
    const __nv_bfloat16* src_a = cvalid_a ? frame + (size_t)crow_a * grid_w * 1024 + ch + half * 8 : nullptr;
    const __nv_bfloat16* src_b = cvalid_b ? frame + (size_t)crow_b * grid_w * 1024 + ch + half * 8 : nullptr;
    // column px into its slot of the ring; one copy group per column (empty past the last column), so
    // the number of groups still pending tells which columns have landed
    auto fetch = [&](int px) {
      if (px < grid_w) {
        uint8_t* slot = ring + (px % kVarDepth) * kVarSlotBytes + half * 16;
        cp_async16(slot + (lane >> 1) * kVarRowPitch, src_a != nullptr ? src_a + (size_t)px * 1024 : x0_ptr + half * 8);
        cp_async16(slot + ((lane >> 1) + 16) * kVarRowPitch,
                   src_b != nullptr ? src_b + (size_t)px * 1024 : x0_ptr + half * 8);
      }
      cp_async_commit();
    };
#pragma unroll
    for (int k = 0; k < kVarDepth; ++k) fetch(k);
    // the 16 channels of one token of the slot, as 8 pairs
    auto load_x = [&](const uint8_t* slot, int r, float2 (&v)[kVarPassChannels / 2]) {
      const uint4* p = reinterpret_cast<const uint4*>(slot + r * kVarRowPitch);
      const uint4 a = p[0], b = p[1];
      const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = make_float2(bf16_lo(w[i]), bf16_hi(w[i]));
    };
    // one grid column: vertical sums over this lane's row and the rows above and below, then the
    // slot goes back to the copiers.  Rows outside the grid hold x0, so the sum of d over the three
    // rows is always (sum of x) - 3 x0.
    auto take = [&](int c, VarColumn& out) {
      if (c < grid_w) {
        cp_async_wait<kVarDepth - 1>();  // all but the newest kVarDepth - 1 groups: column c has landed
        __syncwarp();                     // ... for every lane's copies
        const uint8_t* slot = ring + (c % kVarDepth) * kVarSlotBytes;
        float2 v[kVarPassChannels / 2];
        load_x(slot, lane, v);
        float2 q2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int i = 0; i < kVarPassChannels / 2; ++i) {
          const float2 d = __fadd2_rn(v[i], make_float2(-x0[i].x, -x0[i].y));
          q2 = __ffma2_rn(d, d, q2);
          out.s[i] = __fadd2_rn(v[i], x0_3[i]);
        }
        load_x(slot, up, v);
#pragma unroll
        for (int i = 0; i < kVarPassChannels / 2; ++i) out.s[i] = __fadd2_rn(out.s[i], v[i]);
        load_x(slot, dn, v);
#pragma unroll
        for (int i = 0; i < kVarPassChannels / 2; ++i) out.s[i] = __fadd2_rn(out.s[i], v[i]);
        const float q = q2.x + q2.y;
        const float q_up = __shfl_up_sync(0xffffffffu, q, 1), q_dn = __shfl_down_sync(0xffffffffu, q, 1);
        out.q = q + (lane > 0 ? q_up : 0.0f) + (lane < 31 ? q_dn : 0.0f);
        __syncwarp();  // every lane has read the slot
      } else {
#pragma unroll
        for (int i = 0; i < kVarPassChannels / 2; ++i) out.s[i] = make_float2(0.0f, 0.0f);
        out.q = 0.0f;
      }
      fetch(c + kVarDepth);
    };
    // window of grid column px = columns l, m, r (absent ones are all-zero)
    auto emit = [&](int px, const VarColumn& l, const VarColumn& m, const VarColumn& r) {
      float2 m2 = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int i = 0; i < kVarPassChannels / 2; ++i) {
        const float2 t = __fadd2_rn(__fadd2_rn(l.s[i], m.s[i]), r.s[i]);
        m2 = __ffma2_rn(t, t, m2);
      }
      const float inv_n = inv_rows * ((px > 0 && px < grid_w - 1) ? (1.0f / 3.0f) : (grid_w > 1 ? 0.5f : 1.0f));
      const float v = (l.q + m.q + r.q) * inv_n - (m2.x + m2.y) * inv_n * inv_n;
      if (emits) acc[px] = pass == 0 ? v : acc[px] + v;
    };
    VarColumn ca, cb, cc;
#pragma unroll
    for (int i = 0; i < kVarPassChannels / 2; ++i) ca.s[i] = make_float2(0.0f, 0.0f);
    ca.q = 0.0f;
    take(0, cb);
    // three columns per trip, so the column sums rotate through fixed registers
    for (int px = 0; px < grid_w; px += 3) {
      take(px + 1, cc);
      emit(px, ca, cb, cc);
      if (px + 1 < grid_w) {
        take(px + 2, ca);
        emit(px + 1, cb, cc, ca);
      }
      if (px + 2 < grid_w) {
        take(px + 3, cb);
        emit(px + 2, cc, ca, cb);
      }
    }
    cp_async_wait<0>();
    __syncwarp();
  }
  __syncthreads();
  // rows of this block, all columns: the four warps' partial sums in a fixed order
  const int r0 = blockIdx.y * kVarRowsPerBlock;
  const int n_rows = min(kVarRowsPerBlock, grid_h - r0);
  float* out = var_parts + ((size_t)quarter * frames + f) * grid_h * grid_w + (size_t)r0 * grid_w;
  auto warp_acc = [&](int w, int lane_row, int px) {
    return reinterpret_cast<const float*>(var_smem + w * warp_bytes + kVarDepth * kVarSlotBytes)[lane_row * acc_pitch + px];
  };
  for (int i = threadIdx.x; i < n_rows * grid_w; i += kVarThreads) {
    const int r = i / grid_w, px = i - r * grid_w;
    out[i] = ((warp_acc(0, r + 1, px) + warp_acc(1, r + 1, px)) + warp_acc(2, r + 1, px)) + warp_acc(3, r + 1, px);
  }
}

__global__ void var_sum_kernel(const float* __restrict__ parts, float* __restrict__ var, long long count) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) var[i] = (((parts[i] + parts[count + i]) + parts[2 * count + i]) + parts[3 * count + i]) / 1024.0f;
}

cudaError_t launch_var_map(const litevggt_ctx* ctx, const __nv_bfloat16* x, float* var_parts, float* var,
                           cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const unsigned row_blocks = (unsigned)((z.grid_h + kVarRowsPerBlock - 1) / kVarRowsPerBlock);
  const int smem = (int)(kVarWarps * var_warp_smem_bytes(z.grid_w));
  cudaError_t e = cudaFuncSetAttribute(var_map_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  var_map_kernel<<<dim3(4, row_blocks, z.frames), kVarThreads, smem, s>>>(x, var_parts, z.frames, z.grid_h, z.grid_w,
                                                                         z.n_special);
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
