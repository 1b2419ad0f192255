// FP8 variant of the attention operands (Sec. 3.5 "Fine-tuning and FP8 Quantization", supplementary
// "FP8 Quantization Details": E4M3).  Q, K and V leave the projection in bf16; here each of the
// 3 x 16 (tensor, head) slices gets one scale, amax / 448, from the tensor being quantised
// (current scaling: a single forward pass has no history of earlier iterations to take a delayed
// scale from), and is rounded to E4M3 (nearest even, saturating).  Q and K keep their row-major
// layout with one byte per element; V is written transposed, [head * 64 + channel][key], so that
// the attention kernel can feed it to the tensor core as a K-major operand like K.
#include "common.cuh"
#include "runtime.h"

namespace lv {

constexpr int kAmaxWarps = 8;

// Largest magnitude per (tensor, head).  Warp per row: the row's 384 16-byte pieces go to the lanes
// in 12 passes, 8 neighbouring lanes share a head.  Magnitudes are non-negative floats, which
// order like their bit patterns: integer atomicMax on a zeroed array.
__global__ void __launch_bounds__(kAmaxWarps * 32)
qkv_amax_kernel(const __nv_bfloat16* __restrict__ qkv, long long m, float* __restrict__ amax) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float best[12];
#pragma unroll
  for (int j = 0; j < 12; ++j) best[j] = 0.0f;
  for (long long r = (long long)blockIdx.x * kAmaxWarps + warp; r < m; r += (long long)gridDim.x * kAmaxWarps) {
    const uint4* src = reinterpret_cast<const uint4*>(qkv + (size_t)r * 3072);
#pragma unroll
    for (int j = 0; j < 12; ++j) {
      const uint4 v = __ldg(src + lane + 32 * j);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      float a = 0.0f;
#pragma unroll
      for (int e = 0; e < 4; ++e) a = fmaxf(a, fmaxf(fabsf(bf16_lo(w[e])), fabsf(bf16_hi(w[e]))));
      best[j] = fmaxf(best[j], a);
    }
  }
#pragma unroll
  for (int j = 0; j < 12; ++j) {
    float a = best[j];
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 4));
    // pass j covers elements [256 j, 256 j + 256) of the row = slices 4 j .. 4 j + 3 (tensor * 16 + head)
    if ((lane & 7) == 0) atomicMax(reinterpret_cast<unsigned int*>(amax) + 4 * j + (lane >> 3), __float_as_uint(a));
  }
}

// 1 / scale of a slice, with scale = amax / 448 (an all-zero slice counts as amax = 1); two
// correctly rounded fp32 divisions, which is also how the reference forms it.
__device__ __forceinline__ float e4m3_inv_scale(float amax) {
  const float scale = __fdiv_rn(amax > 0.0f ? amax : 1.0f, 448.0f);
  return __fdiv_rn(1.0f, scale);
}

// 32 bf16 values (64 bytes at src) times inv -> 32 E4M3 bytes
__device__ __forceinline__ void quantize32(const __nv_bfloat16* src, float inv, uint32_t (&out)[8]) {
  const uint4* p = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 v = __ldg(p + i);
    out[2 * i] = pack_e4m3x4(bf16_lo(v.x) * inv, bf16_hi(v.x) * inv, bf16_lo(v.y) * inv, bf16_hi(v.y) * inv);
    out[2 * i + 1] = pack_e4m3x4(bf16_lo(v.z) * inv, bf16_hi(v.z) * inv, bf16_lo(v.w) * inv, bf16_hi(v.w) * inv);
  }
}

// Block = 128 rows of one head, 256 threads: thread (row, half) converts 32 channels of Q, of K and
// of V.  Q and K go straight out; V goes through shared memory as [channel][row] and leaves as 64
// rows of 128 bytes.  Rows past m are written as zeros (V's rows are padded to a multiple of 128
// keys, and a padded key must not carry anything that is not finite).
__global__ void __launch_bounds__(256)
qkv_quantize_kernel(const __nv_bfloat16* __restrict__ qkv, long long m, long long m_pad, const float* __restrict__ amax,
                    uint8_t* __restrict__ q8, uint8_t* __restrict__ k8, uint8_t* __restrict__ v8t) {
  __shared__ __align__(16) uint8_t v_tile[64][128 + 16];
  const int head = blockIdx.y;
  const long long row0 = (long long)blockIdx.x * 128;
  const int r = threadIdx.x >> 1, half = threadIdx.x & 1;
  const long long row = row0 + r;
  const bool live = row < m;
  uint32_t bytes[8];
  const __nv_bfloat16* src = qkv + (size_t)(live ? row : 0) * 3072 + head * 64 + half * 32;
  if (live) {
    quantize32(src, e4m3_inv_scale(amax[head]), bytes);
    uint4* dq = reinterpret_cast<uint4*>(q8 + (size_t)row * 1024 + head * 64 + half * 32);
    dq[0] = make_uint4(bytes[0], bytes[1], bytes[2], bytes[3]);
    dq[1] = make_uint4(bytes[4], bytes[5], bytes[6], bytes[7]);
    quantize32(src + 1024, e4m3_inv_scale(amax[16 + head]), bytes);
    uint4* dk = reinterpret_cast<uint4*>(k8 + (size_t)row * 1024 + head * 64 + half * 32);
    dk[0] = make_uint4(bytes[0], bytes[1], bytes[2], bytes[3]);
    dk[1] = make_uint4(bytes[4], bytes[5], bytes[6], bytes[7]);
    quantize32(src + 2048, e4m3_inv_scale(amax[32 + head]), bytes);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) bytes[i] = 0u;
  }
#pragma unroll
  for (int i = 0; i < 32; ++i) v_tile[half * 32 + i][r] = (uint8_t)(bytes[i >> 2] >> (8 * (i & 3)));
  __syncthreads();
  // thread -> (channel, 32-byte piece of the channel's 128 keys)
  const int ch = threadIdx.x >> 2, piece = threadIdx.x & 3;
  const uint4* sv = reinterpret_cast<const uint4*>(&v_tile[ch][piece * 32]);
  uint4* dv = reinterpret_cast<uint4*>(v8t + ((size_t)head * 64 + ch) * m_pad + row0 + piece * 32);
  dv[0] = sv[0];
  dv[1] = sv[1];
}

cudaError_t launch_qkv_quantize(litevggt_ctx* ctx, const __nv_bfloat16* qkv, long long m, cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  Workspace& ws = ctx->ws;
  if (ws.q8 == nullptr || ctx->sz.dim != 1024 || ctx->sz.heads != 16) return cudaErrorInvalidValue;
  cudaError_t e = cudaMemsetAsync(ws.qkv_amax, 0, 48 * sizeof(float), s);
  if (e != cudaSuccess) return e;
  long long blocks = (m + kAmaxWarps - 1) / kAmaxWarps;
  if (blocks > 4096) blocks = 4096;
  qkv_amax_kernel<<<(unsigned)blocks, kAmaxWarps * 32, 0, s>>>(qkv, m, ws.qkv_amax);
  ++*launches;
  const long long m_pad = round_up(m, 128);
  qkv_quantize_kernel<<<dim3((unsigned)(m_pad / 128), 16), 256, 0, s>>>(qkv, m, m_pad, ws.qkv_amax, ws.q8, ws.k8, ws.v8t);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
