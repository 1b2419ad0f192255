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
// the patch mean.  Rows are loaded a few steps ahead; there is no shared memory and no barrier.
// grad_map_kernel takes any patch size up to 30; grad_map_patch_kernel is the same walk for the
// 14-pixel patches of the model, with a patch's rows unrolled and seven rows in flight.
constexpr int kGradThreads = 128;
#ifndef LV_GRAD_PATCH_ROWS
#define LV_GRAD_PATCH_ROWS 7
#endif
#ifndef LV_GRAD_AHEAD
#define LV_GRAD_AHEAD 3
#endif
#ifndef LV_GRAD_AHEAD14
#define LV_GRAD_AHEAD14 7
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

// The same walk with the patch size known at compile time: the rows of a patch are unrolled, so the
// row in hand, its place in the load queue and the bottom of the patch are all static and the
// per-row bookkeeping (row counters, queue index, end-of-patch test) is gone.  kAhead divides kPatch.
template <int kPatch, int kAhead>
__global__ void __launch_bounds__(kGradThreads)
grad_map_patch_kernel(const float* __restrict__ images, float* __restrict__ grad, int grid_h, int grid_w) {
  static_assert(kPatch % kAhead == 0 && kPatch <= 30 && kAhead >= 2, "queue slots must be static");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int pps = 30 / kPatch;
  const int strips = (grid_w + pps - 1) / pps;
  const int strip = blockIdx.x * (kGradThreads / 32) + warp;
  if (strip >= strips) return;  // whole warp; nothing below synchronises across warps
  const int f = blockIdx.z;
  const int pr0 = blockIdx.y * kGradPatchRows;
  const int pr1 = min(grid_h, pr0 + kGradPatchRows);
  const int h = grid_h * kPatch, w = grid_w * kPatch;
  const size_t plane = (size_t)h * w;
  int x = strip * pps * kPatch - 1 + lane;
  x = x < 0 ? 0 : (x >= w ? w - 1 : x);
  const float* col = images + (size_t)f * 3 * plane + x;
  const bool own = lane >= 1 && lane <= pps * kPatch;
  const int seg = own ? (lane - 1) / kPatch : 0;
  const int in_seg = own ? (lane - 1) - seg * kPatch : kPatch;
  const int patch_x = strip * pps + seg;
  const bool writer = own && in_seg == 0 && patch_x < grid_w;
  constexpr float inv_area = 1.0f / (float)(kPatch * kPatch);

  const int y_first = pr0 * kPatch - 1;  // halo row above (clamped when it is outside)
  float q[kAhead][3];
  // row i of the walk (0 = halo row above the block); rows past the image repeat its last row
  auto load_row = [&](int i, float (&dst)[3]) {
    const int y = min(max(y_first + i, 0), h - 1);
    const float* p = col + (size_t)y * w;
    dst[0] = __ldg(p);
    dst[1] = __ldg(p + plane);
    dst[2] = __ldg(p + 2 * plane);
  };
  struct RowTerms { float d, s; };
  auto terms = [&](const float (&rgb)[3]) {
    const float g = (rgb[0] + rgb[1] + rgb[2]) * (1.0f / 3.0f);
    const float l = __shfl_up_sync(0xffffffffu, g, 1), r = __shfl_down_sync(0xffffffffu, g, 1);
    return RowTerms{r - l, fmaf(2.0f, g, l + r)};
  };
  // rows 0 and 1 come through registers of their own; the queue then holds rows 2 .. kAhead + 1,
  // so row 2 + k of a patch row sits in slot k % kAhead
  float first[2][3];
  load_row(0, first[0]);
  load_row(1, first[1]);
#pragma unroll
  for (int k = 0; k < kAhead; ++k) load_row(2 + k, q[k]);
  RowTerms t0 = terms(first[0]), t1 = terms(first[1]);
  int i = 2;  // next row of the walk
  for (int pr = pr0; pr < pr1; ++pr) {
    float acc = 0.0f;
#pragma unroll
    for (int k = 0; k < kPatch; ++k) {
      const RowTerms t2 = terms(q[k % kAhead]);
      load_row(i + k + kAhead, q[k % kAhead]);
      const float gx = fmaf(2.0f, t1.d, t0.d + t2.d);
      const float gy = t2.s - t0.s;
      acc += sqrt_approx(fmaf(gx, gx, gy * gy));
      t0 = t1;
      t1 = t2;
    }
    i += kPatch;
    // bottom of a patch row: add the columns of each patch, lowest lane of the patch writes
    float v = own ? acc : 0.0f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float t = __shfl_down_sync(0xffffffffu, v, off);
      if (in_seg + off < kPatch) v += t;
    }
    if (writer) grad[((size_t)f * grid_h + pr) * grid_w + patch_x] = v * inv_area;
  }
}

cudaError_t launch_grad_map(const litevggt_ctx* ctx, const float* images, float* grad, cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const int patch = ctx->cfg.patch_px;
  const int pps = 30 / patch;
  const int strips = (z.grid_w + pps - 1) / pps;
  const dim3 grid((unsigned)((strips + kGradThreads / 32 - 1) / (kGradThreads / 32)),
                  (unsigned)((z.grid_h + kGradPatchRows - 1) / kGradPatchRows), (unsigned)z.frames);
  if (patch == 14)
    grad_map_patch_kernel<14, LV_GRAD_AHEAD14><<<grid, kGradThreads, 0, s>>>(images, grad, z.grid_h, z.grid_w);
  else
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
// The step costs about nine fp32 operations per channel of a token (difference, square, two adds
// down the rows, two along them, square of the window sum, with the halo rows on top), which at the
// rate of the FMA pipes is as long as reading the token from HBM: the kernel has to be lean in
// instructions, not only in bytes.  A CTA owns a strip of kVarRows grid rows of one frame, its four
// warps a quarter of the channels each; lane = 8 consecutive channels, so a token's quarter is one
// fully coalesced 512-byte load straight into registers, with no shared-memory stage and no
// barrier.  The warp walks along the strip one grid column per step: the column's kVarRows + 2
// tokens (one halo row above and below; outside the grid the lane's own x0 stands in, so d = 0)
// are read once (the difference to x0 comes from a mixed-precision add that takes the bf16 value
// as it is, so there is no separate conversion) and give the column's vertical sums of d and of
// |d|^2; the sums of the two columns before stay in registers; the loads of the next column are
// issued as soon as this column's registers are free, and the column after it is asked into L2.
// A window's value, (1/n) sum |d|^2 - (1/n^2) |sum d|^2, is linear in
// the per-lane partial sums over the channels, so each lane forms it for its 8 channels, a
// butterfly over the warp adds the 32 lanes for all rows of the strip at once, the four warps'
// sums meet in shared memory and are added in a fixed order: the map is deterministic.
#ifndef LV_VAR_OCC
#define LV_VAR_OCC 3
#endif
constexpr int kVarThreads = 128;
constexpr int kVarWarps = kVarThreads / 32;
constexpr int kVarRows = 4;  // grid rows per CTA
constexpr int kVarMaxW = 64;
constexpr int kVarTokenVec = 128;  // 16-byte vectors per token
#ifndef LV_VAR_PREFETCH
#define LV_VAR_PREFETCH 2
#endif
constexpr int kVarPrefetch = LV_VAR_PREFETCH;  // grid columns between the L2 prefetch and the load

// (bf16 pair) + (fp32 pair): the mixed-precision add converts its 16-bit operand exactly, so the
// result is the fp32 sum rounded once, as with a separate conversion
__device__ __forceinline__ float2 bf16x2_plus_f32x2(uint32_t w, float2 c) {
  float2 r;
  asm("{\n .reg .b16 lo, hi;\n mov.b32 {lo, hi}, %2;\n add.rn.f32.bf16 %0, lo, %3;\n add.rn.f32.bf16 %1, hi, %4;\n}"
      : "=f"(r.x), "=f"(r.y)
      : "r"(w), "f"(c.x), "f"(c.y));
  return r;
}

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

struct VarColumn {
  float2 s[kVarRows][4];  // vertical 3-sums of d, this lane's 8 channels as pairs (packed fp32 arithmetic)
  float q[kVarRows];      // vertical 3-sums of this lane's share of |d|^2
};

__device__ __forceinline__ void var_zero(VarColumn& c) {
#pragma unroll
  for (int r = 0; r < kVarRows; ++r) {
#pragma unroll
    for (int i = 0; i < 4; ++i) c.s[r][i] = make_float2(0.0f, 0.0f);
    c.q[r] = 0.0f;
  }
}

// Vertical sums of the column held in raw[] (kVarRows + 2 tokens, top halo first) into `out`.
__device__ __forceinline__ void var_column(const uint4 (&raw)[kVarRows + 2], const float2 (&neg_x0)[4], VarColumn& out) {
  float2 d[kVarRows + 2][4];
  float q[kVarRows + 2];
#pragma unroll
  for (int r = 0; r < kVarRows + 2; ++r) {
    const uint32_t w[4] = {raw[r].x, raw[r].y, raw[r].z, raw[r].w};
    float2 q2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      d[r][i] = bf16x2_plus_f32x2(w[i], neg_x0[i]);
      q2 = __ffma2_rn(d[r][i], d[r][i], q2);
    }
    q[r] = q2.x + q2.y;
  }
  // rows r and r + 1 of the strip share the sum of the two tokens between them
#pragma unroll
  for (int r = 0; r < kVarRows; r += 2) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 mid = __fadd2_rn(d[r + 1][i], d[r + 2][i]);
      out.s[r][i] = __fadd2_rn(mid, d[r][i]);
      out.s[r + 1][i] = __fadd2_rn(mid, d[r + 3][i]);
    }
    const float qm = q[r + 1] + q[r + 2];
    out.q[r] = qm + q[r];
    out.q[r + 1] = qm + q[r + 3];
  }
}

// The 32 lanes' values of all four rows added up: afterwards every lane holds the sum for row lane >> 3.
__device__ __forceinline__ float var_reduce_rows(const float (&v)[kVarRows], int lane) {
  static_assert(kVarRows == 4, "the butterfly below is written for four rows");
  const bool hi = (lane & 16) != 0;
  const float a0 = (hi ? v[2] : v[0]) + __shfl_xor_sync(0xffffffffu, hi ? v[0] : v[2], 16);
  const float a1 = (hi ? v[3] : v[1]) + __shfl_xor_sync(0xffffffffu, hi ? v[1] : v[3], 16);
  const bool hi2 = (lane & 8) != 0;
  float b = (hi2 ? a1 : a0) + __shfl_xor_sync(0xffffffffu, hi2 ? a0 : a1, 8);
  b += __shfl_xor_sync(0xffffffffu, b, 4);
  b += __shfl_xor_sync(0xffffffffu, b, 2);
  b += __shfl_xor_sync(0xffffffffu, b, 1);
  return b;
}

__global__ void __launch_bounds__(kVarThreads, LV_VAR_OCC)
var_map_kernel(const __nv_bfloat16* __restrict__ x, float* __restrict__ var, int grid_h, int grid_w, int n_special) {
  __shared__ float part[kVarWarps][kVarRows][kVarMaxW];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int f = blockIdx.y, row_base = blockIdx.x * kVarRows;
  const int tokens_frame = grid_h * grid_w + n_special;
  // this lane's 8 channels of the frame's first patch token
  const uint4* frame = reinterpret_cast<const uint4*>(x + ((size_t)f * tokens_frame + n_special) * 1024) + warp * 32 + lane;
  const uint4 x0_raw = __ldg(frame);
  float2 neg_x0[4];
  {
    const uint32_t w[4] = {x0_raw.x, x0_raw.y, x0_raw.z, x0_raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) neg_x0[i] = make_float2(-bf16_lo(w[i]), -bf16_hi(w[i]));
  }
  // rows of the column: r = 0 is the halo row above the strip
  bool row_ok[kVarRows + 2];
  float inv_rows[kVarRows];
#pragma unroll
  for (int r = 0; r < kVarRows + 2; ++r) {
    const int row = row_base - 1 + r;
    row_ok[r] = row >= 0 && row < grid_h;
  }
#pragma unroll
  for (int r = 0; r < kVarRows; ++r)
    inv_rows[r] = 1.0f / (float)(1 + (row_ok[r] ? 1 : 0) + (row_ok[r + 2] ? 1 : 0));
  const int row_stride = grid_w * kVarTokenVec;
  const uint4* col_ptr = frame + (ptrdiff_t)(row_base - 1) * row_stride;  // only dereferenced where row_ok

  uint4 raw[kVarRows + 2];
#pragma unroll
  for (int r = 0; r < kVarRows + 2; ++r) raw[r] = row_ok[r] ? __ldg(col_ptr + (ptrdiff_t)r * row_stride) : x0_raw;
  // rows outside the grid keep x0 in their registers for the whole walk
  auto load_next = [&](int c) {
    if (c < grid_w) {
      col_ptr += kVarTokenVec;
#pragma unroll
      for (int r = 0; r < kVarRows + 2; ++r)
        if (row_ok[r]) raw[r] = __ldg(col_ptr + (ptrdiff_t)r * row_stride);
    }
    // the registers hold one column ahead; the columns after it are asked into L2 meanwhile, so
    // the loads above find them there instead of waiting for HBM
    if (c + kVarPrefetch < grid_w) {
#pragma unroll
      for (int r = 0; r < kVarRows + 2; ++r)
        if (row_ok[r]) prefetch_l2(col_ptr + (ptrdiff_t)r * row_stride + kVarPrefetch * kVarTokenVec);
    }
  };
  // window of grid column px = columns a, b, c (an absent one is all-zero); `ab` = a + b
  auto emit = [&](int px, const VarColumn& ab, const VarColumn& c) {
    const float inv_cols = (px > 0 && px < grid_w - 1) ? (1.0f / 3.0f) : (grid_w > 1 ? 0.5f : 1.0f);
    float v[kVarRows];
#pragma unroll
    for (int r = 0; r < kVarRows; ++r) {
      float2 m2 = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 t = __fadd2_rn(ab.s[r][i], c.s[r][i]);
        m2 = __ffma2_rn(t, t, m2);
      }
      const float inv_n = inv_rows[r] * inv_cols;
      v[r] = inv_n * ((ab.q[r] + c.q[r]) - inv_n * (m2.x + m2.y));
    }
    const float total = var_reduce_rows(v, lane);
    if ((lane & 7) == 0) part[warp][lane >> 3][px] = total;
  };
  // One step: `older` + `newer` are the columns cn - 2 and cn - 1; the column cn, in raw[], replaces
  // the older one, and the window of column cn - 1 is complete.
  auto step = [&](VarColumn& older, const VarColumn& newer, int cn) {
    VarColumn ab;
#pragma unroll
    for (int r = 0; r < kVarRows; ++r) {
#pragma unroll
      for (int i = 0; i < 4; ++i) ab.s[r][i] = __fadd2_rn(older.s[r][i], newer.s[r][i]);
      ab.q[r] = older.q[r] + newer.q[r];
    }
    var_column(raw, neg_x0, older);
    load_next(cn + 1);
    emit(cn - 1, ab, older);
  };

  VarColumn ca, cb;
  var_zero(ca);
  var_column(raw, neg_x0, cb);  // column 0
  load_next(1);
  for (int cn = 1; cn < grid_w; cn += 2) {
    step(ca, cb, cn);
    if (cn + 1 < grid_w) step(cb, ca, cn + 1);
  }
  {
    // last column: nothing to its right
    VarColumn zero;
    var_zero(zero);
    VarColumn ab;
#pragma unroll
    for (int r = 0; r < kVarRows; ++r) {
#pragma unroll
      for (int i = 0; i < 4; ++i) ab.s[r][i] = __fadd2_rn(ca.s[r][i], cb.s[r][i]);
      ab.q[r] = ca.q[r] + cb.q[r];
    }
    emit(grid_w - 1, ab, zero);
  }
  __syncthreads();
  // the four channel quarters in a fixed order; mean over the 1024 channels
  const int n_rows = min(kVarRows, grid_h - row_base);
  float* out = var + ((size_t)f * grid_h + row_base) * grid_w;
  for (int i = threadIdx.x; i < n_rows * grid_w; i += kVarThreads) {
    const int r = i / grid_w, px = i - r * grid_w;
    out[i] = (((part[0][r][px] + part[1][r][px]) + part[2][r][px]) + part[3][r][px]) / 1024.0f;
  }
}

cudaError_t launch_var_map(const litevggt_ctx* ctx, const __nv_bfloat16* x, float* var, cudaStream_t s,
                           int* launches) {
  const Sizes& z = ctx->sz;
  if (z.grid_w > kVarMaxW) return cudaErrorInvalidValue;
  const unsigned strips = (unsigned)((z.grid_h + kVarRows - 1) / kVarRows);
  var_map_kernel<<<dim3(strips, z.frames), kVarThreads, 0, s>>>(x, var, z.grid_h, z.grid_w, z.n_special);
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
