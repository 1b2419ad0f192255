// bf16 linear layer out = a w^T + bias on the tcgen05 GEMM mainloop (the QKV and output
// projections of the attention block, Sec. 3.1).  The output leaves the SM through TMA stores of
// 32-row x 64-column blocks, so `out` needs a 16-byte aligned base and a row pitch (n) that is a
// multiple of 8 elements.
#include "gemm_tc.cuh"
#include "runtime.h"

namespace lv {

cudaError_t launch_linear(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k, const __nv_bfloat16* w,
                          long long n, const __nv_bfloat16* bias, __nv_bfloat16* out, cudaStream_t s, int* launches) {
  return launch_linear_scaled(ctx, a, m, k, w, n, bias, 0, 0, 1.0f, out, s, launches);
}

cudaError_t launch_linear_scaled(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k,
                                 const __nv_bfloat16* w, long long n, const __nv_bfloat16* bias, int scale_begin,
                                 int scale_end, float scale, __nv_bfloat16* out, cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  if (scale_begin % 64 != 0 || scale_end % 64 != 0) return cudaErrorInvalidValue;
  CUtensorMap tmap_a, tmap_b, tmap_out;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap_a, a, (uint64_t)k, (uint64_t)m, (uint64_t)k, kGemmBK, kGemmBM) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_b, w, (uint64_t)k, (uint64_t)n, (uint64_t)k, kGemmBK, kGemmBN) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_out, out, (uint64_t)n, (uint64_t)m, (uint64_t)n, kGemmOutChunkCols,
                         32))
    return cudaErrorInvalidValue;
  LinearEpilogue epi;
  epi.bias = bias;
  epi.m_rows = (int)m;
  epi.n_cols = (int)n;
  epi.scale_begin = scale_begin;
  epi.scale_end = scale_end;
  epi.scale = scale;
  static std::atomic<unsigned long long> smem_set{0};
  cudaError_t e = set_max_dynamic_smem_once(reinterpret_cast<const void*>(gemm_tc_kernel<LinearEpilogue>), kGemmSmemBytes,
                                            smem_set);
  if (e != cudaSuccess) return e;
  const long long tiles = ((m + kGemmBM - 1) / kGemmBM) * ((n + kGemmBN - 1) / kGemmBN);
  const int grid = tiles < ctx->num_sms ? (int)tiles : ctx->num_sms;
  gemm_tc_kernel<LinearEpilogue><<<grid, gemm_threads<LinearEpilogue>(), kGemmSmemBytes, s>>>(tmap_a, tmap_b, tmap_out, (int)m, (int)n,
                                                                            (int)k, epi, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

// out = act(a w^T + bias) + residual, the two layers of the transformer MLP (fc1: GELU, no residual;
// fc2: identity, residual = the block's input).
cudaError_t launch_linear_mlp(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k,
                              const __nv_bfloat16* w, long long n, const __nv_bfloat16* bias, int gelu,
                              const __nv_bfloat16* residual, __nv_bfloat16* out, cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  CUtensorMap tmap_a, tmap_b, tmap_out;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap_a, a, (uint64_t)k, (uint64_t)m, (uint64_t)k, kGemmBK, kGemmBM) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_b, w, (uint64_t)k, (uint64_t)n, (uint64_t)k, kGemmBK, kGemmBN) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_out, out, (uint64_t)n, (uint64_t)m, (uint64_t)n, kGemmOutChunkCols,
                         32))
    return cudaErrorInvalidValue;
  MlpEpilogue epi;
  epi.bias = bias;
  epi.residual = residual;
  epi.m_rows = (int)m;
  epi.n_cols = (int)n;
  epi.ld_res = n;
  epi.gelu = gelu;
  static std::atomic<unsigned long long> smem_set{0};
  cudaError_t e = set_max_dynamic_smem_once(reinterpret_cast<const void*>(gemm_tc_kernel<MlpEpilogue>), kGemmSmemBytes,
                                            smem_set);
  if (e != cudaSuccess) return e;
  const long long tiles = ((m + kGemmBM - 1) / kGemmBM) * ((n + kGemmBN - 1) / kGemmBN);
  const int grid = tiles < ctx->num_sms ? (int)tiles : ctx->num_sms;
  gemm_tc_kernel<MlpEpilogue><<<grid, gemm_threads<MlpEpilogue>(), kGemmSmemBytes, s>>>(tmap_a, tmap_b, tmap_out, (int)m, (int)n,
                                                                         (int)k, epi, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
