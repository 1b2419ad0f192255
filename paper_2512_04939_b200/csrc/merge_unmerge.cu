// Size-weighted merge and gather-unmerge (Sec. 3.4: merge equation and "Token Unmerging").
// Both are pure HBM streaming: one warp per 2 KB row, 16-byte vector accesses, 512
// contiguous bytes per warp instruction.
//
// Merge: row j of the merged sequence is the mean of its own token and the src tokens
// listed for it in the CSR, summed in fp32 in ascending token order (deterministic) and
// rounded once; rows that absorb nothing are copied bit-exactly.
// Unmerge: out_i = y'[dst_of[i]] (+ residual_i, added in fp32).
#include "common.cuh"
#include "runtime.h"

namespace lv {

constexpr int kRowThreads = 256;
constexpr int kRowsPerCta = kRowThreads / 32;

__device__ __forceinline__ void add_row(float (&acc)[32], const uint4 (&v)[4]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t w[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[q * 8 + 2 * i] += bf16_lo(w[i]);
      acc[q * 8 + 2 * i + 1] += bf16_hi(w[i]);
    }
  }
}

__device__ __forceinline__ void load_row(uint4 (&v)[4], const __nv_bfloat16* row, int lane) {
  const uint4* p = reinterpret_cast<const uint4*>(row);
#pragma unroll
  for (int q = 0; q < 4; ++q) v[q] = p[q * 32 + lane];
}

__global__ void __launch_bounds__(kRowThreads)
merge_kernel(const __nv_bfloat16* __restrict__ x, const int* __restrict__ kept_idx, const int* __restrict__ seg_off,
             const int* __restrict__ seg_src, __nv_bfloat16* __restrict__ xm, long long n_merged,
             long long n_tokens, long long n_remove, uint32_t* status) {
  const int lane = threadIdx.x & 31;
  const long long j = (long long)blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
  if (j >= n_merged) return;
  long long own = kept_idx[j];
  int s0 = seg_off[j], s1 = seg_off[j + 1];
  if (own < 0 || own >= n_tokens || s0 < 0 || s1 < s0 || s1 > n_remove) {
    if (lane == 0) atomicOr(status, kStatusBounds);
    own = own < 0 || own >= n_tokens ? 0 : own;
    s1 = s0;
  }
  uint4 v[4];
  load_row(v, x + own * 1024, lane);
  uint4* out = reinterpret_cast<uint4*>(xm + j * 1024);
  if (s1 == s0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) out[q * 32 + lane] = v[q];
    return;
  }
  float acc[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
  add_row(acc, v);
  int s = s0;
  for (; s + 1 < s1; s += 2) {  // two rows in flight
    long long t0 = seg_src[s], t1 = seg_src[s + 1];
    if (t0 < 0 || t0 >= n_tokens || t1 < 0 || t1 >= n_tokens) {
      if (lane == 0) atomicOr(status, kStatusBounds);
      continue;
    }
    uint4 a[4], b[4];
    load_row(a, x + t0 * 1024, lane);
    load_row(b, x + t1 * 1024, lane);
    add_row(acc, a);
    add_row(acc, b);
  }
  if (s < s1) {
    const long long t0 = seg_src[s];
    if (t0 < 0 || t0 >= n_tokens) {
      if (lane == 0) atomicOr(status, kStatusBounds);
    } else {
      uint4 a[4];
      load_row(a, x + t0 * 1024, lane);
      add_row(acc, a);
    }
  }
  const float denom = (float)(1 + s1 - s0);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 o;
    o.x = pack_bf16(acc[q * 8 + 0] / denom, acc[q * 8 + 1] / denom);
    o.y = pack_bf16(acc[q * 8 + 2] / denom, acc[q * 8 + 3] / denom);
    o.z = pack_bf16(acc[q * 8 + 4] / denom, acc[q * 8 + 5] / denom);
    o.w = pack_bf16(acc[q * 8 + 6] / denom, acc[q * 8 + 7] / denom);
    out[q * 32 + lane] = o;
  }
}

__global__ void __launch_bounds__(kRowThreads)
unmerge_kernel(const __nv_bfloat16* __restrict__ ym, const int* __restrict__ dst_of,
               const __nv_bfloat16* __restrict__ residual, __nv_bfloat16* __restrict__ out, long long n_tokens,
               long long n_merged, uint32_t* status) {
  const int lane = threadIdx.x & 31;
  const long long i = (long long)blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
  if (i >= n_tokens) return;
  long long row = dst_of[i];
  if (row < 0 || row >= n_merged) {
    if (lane == 0) atomicOr(status, kStatusBounds);
    row = 0;
  }
  uint4 v[4];
  load_row(v, ym + row * 1024, lane);
  uint4* o = reinterpret_cast<uint4*>(out + i * 1024);
  if (residual == nullptr) {
#pragma unroll
    for (int q = 0; q < 4; ++q) o[q * 32 + lane] = v[q];
    return;
  }
  uint4 r[4];
  load_row(r, residual + i * 1024, lane);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t a[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
    const uint32_t b[4] = {r[q].x, r[q].y, r[q].z, r[q].w};
    uint32_t c[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) c[k] = pack_bf16(bf16_lo(a[k]) + bf16_lo(b[k]), bf16_hi(a[k]) + bf16_hi(b[k]));
    o[q * 32 + lane] = make_uint4(c[0], c[1], c[2], c[3]);
  }
}

// LayerNorm over the 1024 channels of every row (the pre-norm of the transformer blocks, Sec. 3.1):
// y = (x - mean) / sqrt(var + eps) * gamma + beta, population variance, two passes over the row held
// in registers, fp32, one rounding.  One warp per row like the kernels above.
__global__ void __launch_bounds__(kRowThreads)
layernorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gamma,
                 const __nv_bfloat16* __restrict__ beta, __nv_bfloat16* __restrict__ out, long long rows, float eps) {
  const int lane = threadIdx.x & 31;
  const long long i = (long long)blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
  if (i >= rows) return;
  uint4 v[4];
  load_row(v, x + i * 1024, lane);
  float f[32];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t w[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      f[q * 8 + 2 * k] = bf16_lo(w[k]);
      f[q * 8 + 2 * k + 1] = bf16_hi(w[k]);
    }
  }
  float sum = 0.0f;
#pragma unroll
  for (int k = 0; k < 32; ++k) sum += f[k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum * (1.0f / 1024.0f);
  float ss = 0.0f;
#pragma unroll
  for (int k = 0; k < 32; ++k) {
    f[k] -= mean;
    ss = fmaf(f[k], f[k], ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float rstd = rsqrtf(ss * (1.0f / 1024.0f) + eps);
  uint4* op = reinterpret_cast<uint4*>(out + i * 1024);
  const uint4* gp = reinterpret_cast<const uint4*>(gamma);
  const uint4* bp = reinterpret_cast<const uint4*>(beta);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 g = gp[q * 32 + lane], b = bp[q * 32 + lane];
    const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, bw[4] = {b.x, b.y, b.z, b.w};
    uint32_t c[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      c[k] = pack_bf16(fmaf(f[q * 8 + 2 * k] * rstd, bf16_lo(gw[k]), bf16_lo(bw[k])),
                       fmaf(f[q * 8 + 2 * k + 1] * rstd, bf16_hi(gw[k]), bf16_hi(bw[k])));
    op[q * 32 + lane] = make_uint4(c[0], c[1], c[2], c[3]);
  }
}

cudaError_t launch_layernorm(const __nv_bfloat16* x, const __nv_bfloat16* gamma, const __nv_bfloat16* beta,
                             __nv_bfloat16* out, long long rows, float eps, cudaStream_t s, int* launches) {
  if (rows == 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((rows + kRowsPerCta - 1) / kRowsPerCta);
  layernorm_kernel<<<blocks, kRowThreads, 0, s>>>(x, gamma, beta, out, rows, eps);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_merge(const litevggt_ctx* ctx, const litevggt_plan* plan, const __nv_bfloat16* x,
                         __nv_bfloat16* xm, cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const unsigned blocks = (unsigned)((z.n_merged + kRowsPerCta - 1) / kRowsPerCta);
  merge_kernel<<<blocks, kRowThreads, 0, s>>>(x, plan->kept_idx, plan->seg_off, plan->seg_src, xm, z.n_merged,
                                              z.n_tokens, z.n_remove, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_unmerge(const litevggt_ctx* ctx, const litevggt_plan* plan, const __nv_bfloat16* ym,
                           const __nv_bfloat16* residual, __nv_bfloat16* out, cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  const unsigned blocks = (unsigned)((z.n_tokens + kRowsPerCta - 1) / kRowsPerCta);
  unmerge_kernel<<<blocks, kRowThreads, 0, s>>>(ym, plan->dst_of, residual, out, z.n_tokens, z.n_merged,
                                                ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
