// bf16 linear layer out = a w^T + bias on the tcgen05 GEMM mainloop (the QKV and output
// projections of the attention block, Sec. 3.1).
#include "gemm_tc.cuh"
#include "runtime.h"

namespace lv {

cudaError_t launch_linear(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k, const __nv_bfloat16* w,
                          long long n, const __nv_bfloat16* bias, __nv_bfloat16* out, cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  CUtensorMap tmap_a, tmap_b;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap_a, a, (uint64_t)k, (uint64_t)m, (uint64_t)k, kGemmBK, kGemmBM) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_b, w, (uint64_t)k, (uint64_t)n, (uint64_t)k, kGemmBK, kGemmBN))
    return cudaErrorInvalidValue;
  LinearEpilogue epi;
  epi.out = out;
  epi.bias = bias;
  epi.m_rows = (int)m;
  epi.n_cols = (int)n;
  epi.ld_out = n;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<LinearEpilogue>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kGemmSmemBytes);
  if (e != cudaSuccess) return e;
  const int m_blocks = (int)((m + kGemmBM - 1) / kGemmBM);
  const int grid = m_blocks < ctx->num_sms ? m_blocks : ctx->num_sms;
  gemm_tc_kernel<LinearEpilogue><<<grid, kGemmThreads, kGemmSmemBytes, s>>>(tmap_a, tmap_b, (int)m, (int)n, (int)k,
                                                                            epi, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

// out = act(a w^T + bias) + residual, the two layers of the transformer MLP (fc1: GELU, no residual;
// fc2: identity, residual = the block's input).
cudaError_t launch_linear_mlp(litevggt_ctx* ctx, const __nv_bfloat16* a, long long m, long long k,
                              const __nv_bfloat16* w, long long n, const __nv_bfloat16* bias, int gelu,
                              const __nv_bfloat16* residual, __nv_bfloat16* out, cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  CUtensorMap tmap_a, tmap_b;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap_a, a, (uint64_t)k, (uint64_t)m, (uint64_t)k, kGemmBK, kGemmBM) ||
      !make_tmap_bf16_2d(ctx->encode_tiled, &tmap_b, w, (uint64_t)k, (uint64_t)n, (uint64_t)k, kGemmBK, kGemmBN))
    return cudaErrorInvalidValue;
  MlpEpilogue epi;
  epi.out = out;
  epi.bias = bias;
  epi.residual = residual;
  epi.m_rows = (int)m;
  epi.n_cols = (int)n;
  epi.ld_out = n;
  epi.gelu = gelu;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<MlpEpilogue>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kGemmSmemBytes);
  if (e != cudaSuccess) return e;
  const int m_blocks = (int)((m + kGemmBM - 1) / kGemmBM);
  const int grid = m_blocks < ctx->num_sms ? m_blocks : ctx->num_sms;
  gemm_tc_kernel<MlpEpilogue><<<grid, kGemmThreads, kGemmSmemBytes, s>>>(tmap_a, tmap_b, (int)m, (int)n, (int)k, epi,
                                                                         ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
