// Src -> anchor cosine matching with a fused row argmax (Sec. 3.4, "Cached Token Merging":
// every src token is matched to its most similar dst token by cosine similarity).
//
// Step 1 (pack): the src and anchor rows, interleaved inside each frame of x, are copied
// into two contiguous panels so that plain 2-D TMA tiles can feed the tensor cores, and
// 1/max(||row||, 1e-12) is computed in fp32 on the way.
// Step 2 (match): persistent tcgen05 GEMM panel_src x panel_dst^T on the raw bf16 rows
// (exact products, fp32 accumulation); the epilogue scales each column by the anchor's
// inverse norm and keeps a running (max, argmax) per src row, so the |Src| x |Dst| score
// matrix is never written.  Scaling by the src row's own inverse norm cannot change the
// argmax and is applied once to the reported similarity.
#include "gemm_tc.cuh"
#include "runtime.h"

namespace lv {

constexpr int kPackThreads = 256;

__global__ void __launch_bounds__(kPackThreads)
pack_rows_kernel(const __nv_bfloat16* __restrict__ x, const int* __restrict__ src_list,
                 const int* __restrict__ dst_list, long long n_src, long long n_dst, long long n_dst_padded,
                 long long n_tokens, __nv_bfloat16* __restrict__ panel_src, __nv_bfloat16* __restrict__ panel_dst,
                 float* __restrict__ inv_norm_src, float* __restrict__ inv_norm_dst, uint32_t* status) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * (kPackThreads / 32) + (threadIdx.x >> 5);
  if (row >= n_src + n_dst_padded) return;
  if (row >= n_src + n_dst) {  // padding of the anchor norm vector
    if (lane == 0) inv_norm_dst[row - n_src] = 0.0f;
    return;
  }
  const bool is_src = row < n_src;
  const long long r = is_src ? row : row - n_src;
  long long token = is_src ? src_list[r] : dst_list[r];
  if (token < 0 || token >= n_tokens) {
    if (lane == 0) atomicOr(status, kStatusBounds);
    token = 0;
  }
  const uint4* in = reinterpret_cast<const uint4*>(x + token * 1024);
  uint4* out = reinterpret_cast<uint4*>((is_src ? panel_src : panel_dst) + r * 1024);
  float ss = 0.0f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 v = in[q * 32 + lane];
    out[q * 32 + lane] = v;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = bf16_lo(w[i]), b = bf16_hi(w[i]);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) {
    const float inv = 1.0f / fmaxf(sqrtf(ss), 1e-12f);
    (is_src ? inv_norm_src : inv_norm_dst)[r] = inv;
  }
}

cudaError_t launch_match(litevggt_ctx* ctx, const __nv_bfloat16* x, int* best_dst, float* best_sim, cudaStream_t s,
                         int* launches) {
  const Sizes& z = ctx->sz;
  Workspace& ws = ctx->ws;
  if (z.n_src == 0) return cudaSuccess;
  const long long n_dst_padded = round_up(z.n_dst, 256);
  const long long rows = z.n_src + n_dst_padded;
  const int warps = kPackThreads / 32;
  pack_rows_kernel<<<(unsigned)((rows + warps - 1) / warps), kPackThreads, 0, s>>>(
      x, ws.src_list, ws.dst_list, z.n_src, z.n_dst, n_dst_padded, z.n_tokens, ws.panel_src, ws.panel_dst,
      ws.inv_norm_src, ws.inv_norm_dst, ws.status);
  ++*launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  CUtensorMap tmap_a, tmap_b;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap_a, ws.panel_src, 1024, (uint64_t)z.n_src, 1024, kGemmBK, kGemmBM) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_b, ws.panel_dst, 1024, (uint64_t)z.n_dst, 1024, kGemmBK, kGemmBN))
    return cudaErrorInvalidValue;
  ArgmaxEpilogue epi;
  epi.inv_norm_a = ws.inv_norm_src;
  epi.inv_norm_b = ws.inv_norm_dst;
  epi.col_ids = ws.dst_list;
  epi.best_idx = best_dst;
  epi.best_val = best_sim;
  epi.m_rows = (int)z.n_src;
  epi.n_cols = (int)z.n_dst;
  static std::atomic<unsigned long long> smem_set{0};
  e = set_max_dynamic_smem_once(reinterpret_cast<const void*>(gemm_tc_kernel<ArgmaxEpilogue>), kGemmSmemBytes, smem_set);
  if (e != cudaSuccess) return e;
  const int m_blocks = (int)((z.n_src + kGemmBM - 1) / kGemmBM);
  const int grid = m_blocks < ctx->num_sms ? m_blocks : ctx->num_sms;
  // the argmax epilogue writes no matrix: the store map is never read, any valid map fills the slot
  gemm_tc_kernel<ArgmaxEpilogue><<<grid, gemm_threads<ArgmaxEpilogue>(), kGemmSmemBytes, s>>>(tmap_a, tmap_b, tmap_a, (int)z.n_src,
                                                                            (int)z.n_dst, 1024, epi, ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
