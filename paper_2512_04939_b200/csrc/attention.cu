// Global self-attention over the merged token sequence (Sec. 3.1: the frame-global
// attention layer; after merging it runs over M instead of N tokens).  Per head
//   O = softmax(Q K^T / sqrt(64)) V,      non-causal, no mask,
// computed flash-style: scores never leave the SM.
//
// One CTA = 256 query rows (two tiles of 128) of one head, sweeping all keys in tiles of
// 128.  Warp roles (12 warps):
//   warps 0-3   softmax of query tile 0 (thread = one query row = one TMEM lane)
//   warps 4-7   softmax of query tile 1
//   warp  8     MMA issuer (one elected lane):  S_t = Q_t K_j^T  and  O_t += P_t V_j
//   warp  9     TMA producer (one elected lane): Q once, then K_j / V_j through two
//               4-stage shared-memory rings
//   warps 10-11 idle; they only complete the third warpgroup so that the register file can
//               be re-split (softmax warps take 216 registers, the rest 64)
// Tensor memory (512 columns): S_0 S_1 (fp32, 128 columns each) | O_0 O_1 (fp32, 64 each)
// | P_0 P_1 (bf16 pairs, 64 each).  P is fed to the second MMA straight from tensor
// memory; V tiles are consumed as an MN-major B operand, K tiles as a K-major one, so
// neither needs a transpose.  While the softmax warps of one tile work, the tensor core
// runs the other tile's MMAs.
//
// Softmax arithmetic.  At head dim 64 every score costs 256 tensor flops and one
// exponential, and the special-function unit issues only 16 ex2 per clock per SM, half of
// what the tensor cores would need.  So a fixed share of the exponentials of every row is
// evaluated on the FMA pipes instead: round-to-nearest split x = n + f, |f| <= 1/2, a cubic
// for 2^f (relative error 7.5e-5, far below the bf16 rounding of P) and n added into the
// exponent field.  Scale, subtraction of the reference maximum, the polynomial and the row
// sums use packed two-wide fp32 instructions.
//
// Online softmax in base 2 with a lazily updated reference maximum: the running output
// is rescaled only when a row maximum grows by more than 2^8 over the reference, and the
// final division by the row sum removes the reference again, so the result equals the
// plain softmax up to rounding.
#include "common.cuh"
#include "runtime.h"

namespace lv {

constexpr int kFaStages = 4;
constexpr int kFaThreads = 384;
constexpr int kFaTileBytes = 128 * 64 * 2;
constexpr int kFaSmemBytes = (2 + 2 * kFaStages) * kFaTileBytes + 512 + 1024;
constexpr uint32_t kFaColS = 0, kFaColO = 256, kFaColP = 384;
constexpr float kFaRescaleThreshold = 8.0f;
// Of every 8 consecutive pairs of scores, this many take the polynomial exponential.
#ifndef LV_FA_POLY_PAIRS
#define LV_FA_POLY_PAIRS 2
#endif
constexpr int kFaPolyPairsPer8 = LV_FA_POLY_PAIRS;

struct FaBarriers {
  uint64_t q_full;
  uint64_t k_full[kFaStages], k_empty[kFaStages];
  uint64_t v_full[kFaStages], v_empty[kFaStages];
  uint64_t s_full[2], p_ready[2], o_done[2];
  uint64_t teardown;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x for a pair of arguments on the FMA pipes.  Adding 1.5 * 2^23 rounds x to the nearest
// integer n in the low mantissa bits; 2^(x - n) comes from a cubic fitted on [-1/2, 1/2] and
// n is added to the exponent field.  Arguments are clamped at -120 (2^-120 stands in for
// zero); the callers keep them below 2^8.
__device__ __forceinline__ float2 poly_exp2_pair(float2 x) {
  x.x = fmaxf(x.x, -120.0f);
  x.y = fmaxf(x.y, -120.0f);
  const float2 magic = make_float2(12582912.0f, 12582912.0f);
  const float2 t = __fadd2_rn(x, magic);
  const float2 n = __fadd2_rn(t, make_float2(-12582912.0f, -12582912.0f));
  const float2 f = __ffma2_rn(n, make_float2(-1.0f, -1.0f), x);
  float2 p = __ffma2_rn(make_float2(0.0551716648f, 0.0551716648f), f, make_float2(0.2426111251f, 0.2426111251f));
  p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
  p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
  float2 r;
  r.x = __uint_as_float(__float_as_uint(p.x) + (__float_as_uint(t.x) << 23));
  r.y = __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(t.y) << 23));
  return r;
}

// Wait until the most recent loads into a ring (up to one per stage) have landed.
// `issued` counts the loads issued into the ring so far; load i uses stage i % kFaStages and
// completes the phase with parity (i / kFaStages) & 1.  Not sensitive to the abort flag: the
// copies are in flight and must finish before the shared memory can be given up.
__device__ __forceinline__ void drain_ring(uint64_t* full, uint32_t issued, uint32_t* status) {
  const uint32_t n_drain = issued < (uint32_t)kFaStages ? issued : (uint32_t)kFaStages;
  for (uint32_t i = 0; i < n_drain; ++i) {
    const uint32_t idx = issued - 1 - i;
    const long long t0 = clock64();
    while (!mbar_try_wait(&full[idx % kFaStages], (idx / kFaStages) & 1u)) {
      if (clock64() - t0 > kTimeoutCycles) { atomicOr(status, kStatusTimeout); break; }
    }
  }
}

// Exponentials of one 32-score chunk of a row: p = 2^(s * scale - m_ref), packed to bf16
// pairs; the fp32 values are added to the row's packed partial sums.
__device__ __forceinline__ void softmax_chunk(const uint32_t (&s)[32], float2 scale2, float2 neg_m2,
                                              float2 (&sum2)[2], uint32_t (&packed)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), scale2, neg_m2);
    float2 p;
    if ((i & 7) < kFaPolyPairsPer8) {
      p = poly_exp2_pair(x);
    } else {
      p.x = fast_exp2(x.x);
      p.y = fast_exp2(x.y);
    }
    sum2[i & 1] = __fadd2_rn(sum2[i & 1], p);
    packed[i] = pack_bf16(p.x, p.y);
  }
}

__global__ void __launch_bounds__(kFaThreads, 1)
flash_attention_kernel(const __grid_constant__ CUtensorMap tmap_qkv, __nv_bfloat16* __restrict__ o, int m_rows,
                       int dim, float scale_log2e, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_q = smem;
  uint8_t* smem_k = smem + 2 * kFaTileBytes;
  uint8_t* smem_v = smem_k + kFaStages * kFaTileBytes;
  FaBarriers* bars = reinterpret_cast<FaBarriers*>(smem_v + kFaStages * kFaTileBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * 256;
  const int head = blockIdx.y;
  const int n_kv = (m_rows + 127) / 128;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    for (int s = 0; s < kFaStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(&bars->s_full[t], 1);
      mbar_init(&bars->p_ready[t], 4);
      mbar_init(&bars->o_done[t], 1);
    }
    mbar_init(&bars->teardown, 1);
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_qkv);
  }
  if (warp == 8) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const WaitCtl ctl{&bars->abort_flag, status};

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    if (warp == 9) {
      // ---------------------------------------------------------------- TMA producer
      if (elect_one()) {
        mbar_expect_tx(&bars->q_full, 2 * kFaTileBytes);
        tma_load_2d(smem_q, &tmap_qkv, &bars->q_full, head * 64, q0);
        tma_load_2d(smem_q + kFaTileBytes, &tmap_qkv, &bars->q_full, head * 64, q0 + 128);
        uint32_t k_issued = 0, v_issued = 0;
        for (int j = 0; j < n_kv; ++j) {
          const int stage = j % kFaStages;
          const uint32_t phase = (uint32_t)(j / kFaStages) & 1u;
          if (!mbar_wait(&bars->k_empty[stage], phase ^ 1u, ctl)) break;
          mbar_expect_tx(&bars->k_full[stage], kFaTileBytes);
          tma_load_2d(smem_k + stage * kFaTileBytes, &tmap_qkv, &bars->k_full[stage], dim + head * 64, j * 128);
          ++k_issued;
          if (!mbar_wait(&bars->v_empty[stage], phase ^ 1u, ctl)) break;
          mbar_expect_tx(&bars->v_full[stage], kFaTileBytes);
          tma_load_2d(smem_v + stage * kFaTileBytes, &tmap_qkv, &bars->v_full[stage], 2 * dim + head * 64, j * 128);
          ++v_issued;
        }
        // every load issued by this thread must have landed before the CTA may exit
        {
          const long long t0 = clock64();
          while (!mbar_try_wait(&bars->q_full, 0)) {
            if (clock64() - t0 > kTimeoutCycles) { atomicOr(status, kStatusTimeout); break; }
          }
        }
        drain_ring(bars->k_full, k_issued, status);
        drain_ring(bars->v_full, v_issued, status);
      }
    } else if (warp == 8) {
      // ---------------------------------------------------------------- MMA issuer
      if (elect_one()) {
        constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 128, false, false);
        constexpr uint32_t idesc_pv = umma_idesc_bf16(128, 64, false, true);
        bool ok = mbar_wait(&bars->q_full, 0, ctl);
        auto issue_qk = [&](int t, int stage) {
          const uint64_t a_desc = smem_desc_sw128(smem_u32(smem_q + t * kFaTileBytes), 16, 1024);
          const uint64_t b_desc = smem_desc_sw128(smem_u32(smem_k + stage * kFaTileBytes), 16, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss(tmem_base + kFaColS + t * 128, a_desc + 2 * k, b_desc + 2 * k, idesc_qk, k != 0 ? 1u : 0u);
          umma_commit(&bars->s_full[t]);
        };
        if (ok) ok = mbar_wait(&bars->k_full[0], 0, ctl);
        if (ok) {
          tc_fence_after();
          issue_qk(0, 0);
          issue_qk(1, 0);
          umma_commit(&bars->k_empty[0]);
        }
        int stage = 0;
        uint32_t phase = 0;
        for (int j = 0; j < n_kv && ok; ++j) {
          int next_stage = stage + 1;
          uint32_t next_phase = phase;
          if (next_stage == kFaStages) { next_stage = 0; next_phase ^= 1u; }
          const bool last = j + 1 == n_kv;
          if (!mbar_wait(&bars->v_full[stage], phase, ctl)) { ok = false; break; }
          const uint64_t v_desc = smem_desc_sw128(smem_u32(smem_v + stage * kFaTileBytes), 1024, 1024);
          for (int t = 0; t < 2; ++t) {
            if (!mbar_wait(&bars->p_ready[t], j & 1, ctl)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < 8; ++k)  // 16 keys per instruction: 8 TMEM columns of P, 2048 bytes of V
              umma_ts(tmem_base + kFaColO + t * 64, tmem_base + kFaColP + t * 64 + k * 8, v_desc + 128 * k, idesc_pv,
                      (j | k) != 0 ? 1u : 0u);
            if (last) {
              umma_commit(&bars->o_done[t]);
            } else {
              if (t == 0 && !mbar_wait(&bars->k_full[next_stage], next_phase, ctl)) { ok = false; break; }
              tc_fence_after();
              issue_qk(t, next_stage);
              if (t == 1) umma_commit(&bars->k_empty[next_stage]);
            }
          }
          if (!ok) break;
          umma_commit(&bars->v_empty[stage]);
          stage = next_stage;
          phase = next_phase;
        }
        if (!ok) {
          umma_commit(&bars->teardown);
          const long long t0 = clock64();
          while (!mbar_try_wait(&bars->teardown, 0)) {
            if (clock64() - t0 > kTimeoutCycles) break;
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int t = warp >> 2;
    const uint32_t quarter = warp & 3u;
    const uint32_t lane_base = (quarter * 32u) << 16;
    const int row = q0 + t * 128 + (int)quarter * 32 + lane;
    const uint32_t s_addr = tmem_base + lane_base + kFaColS + t * 128;
    const uint32_t o_addr = tmem_base + lane_base + kFaColO + t * 64;
    const uint32_t p_addr = tmem_base + lane_base + kFaColP + t * 64;
    const float2 scale2 = make_float2(scale_log2e, scale_log2e);
    float m_ref = -INFINITY;  // reference maximum, in log2 units (score * scale * log2 e)
    float2 l_sum2[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      if (!mbar_wait_warp(&bars->s_full[t], j & 1, ctl)) { ok = false; break; }
      tc_fence_after();
      uint32_t s[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, s[c]);
      tmem_ld_wait();
      const int valid = m_rows - j * 128;
      if (valid < 128) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c * 32 + i >= valid) s[c][i] = 0xff800000u;  // -inf
      }
      float mx[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        mx[c] = fmaxf(__uint_as_float(s[c][0]), __uint_as_float(s[c][1]));
#pragma unroll
        for (int i = 2; i < 32; i += 2) mx[c] = fmax3(mx[c], __uint_as_float(s[c][i]), __uint_as_float(s[c][i + 1]));
      }
      const float mx_scaled = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2e;
      if (j == 0) {
        m_ref = mx_scaled;
      } else {
        const bool grow = mx_scaled > m_ref + kFaRescaleThreshold;
        if (__any_sync(0xffffffffu, grow ? 1 : 0)) {
          const float m_new = grow ? mx_scaled : m_ref;
          const float alpha = fast_exp2(m_ref - m_new);
          const float2 alpha2 = make_float2(alpha, alpha);
          l_sum2[0] = __fmul2_rn(l_sum2[0], alpha2);
          l_sum2[1] = __fmul2_rn(l_sum2[1], alpha2);
          m_ref = m_new;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t acc[32];
            tmem_ld32(o_addr + c * 32, acc);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * alpha);
            tmem_st32(o_addr + c * 32, acc);
          }
        }
      }
      const float2 neg_m2 = make_float2(-m_ref, -m_ref);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t packed[16];
        softmax_chunk(s[c], scale2, neg_m2, l_sum2, packed);
        tmem_st16(p_addr + c * 16, packed);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_ready[t]);
    }
    if (ok && mbar_wait_warp(&bars->o_done[t], 0, ctl)) {
      tc_fence_after();
      const float inv = 1.0f / ((l_sum2[0].x + l_sum2[0].y) + (l_sum2[1].x + l_sum2[1].y));
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t acc[32];
        tmem_ld32(o_addr + c * 32, acc);
        tmem_ld_wait();
        if (row < m_rows) {
          uint4* dst = reinterpret_cast<uint4*>(o + (size_t)row * dim + head * 64 + c * 32);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(acc[q * 8 + 0]) * inv, __uint_as_float(acc[q * 8 + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(acc[q * 8 + 2]) * inv, __uint_as_float(acc[q * 8 + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(acc[q * 8 + 4]) * inv, __uint_as_float(acc[q * 8 + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(acc[q * 8 + 6]) * inv, __uint_as_float(acc[q * 8 + 7]) * inv);
            dst[q] = w;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

cudaError_t launch_flash_attention(litevggt_ctx* ctx, const __nv_bfloat16* qkv, long long m, __nv_bfloat16* o,
                                   cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  const int dim = ctx->sz.dim;
  CUtensorMap tmap;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap, qkv, (uint64_t)3 * dim, (uint64_t)m, (uint64_t)3 * dim, 64, 128))
    return cudaErrorInvalidValue;
  cudaError_t e =
      cudaFuncSetAttribute(flash_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFaSmemBytes);
  if (e != cudaSuccess) return e;
  const dim3 grid((unsigned)((m + 255) / 256), (unsigned)ctx->sz.heads);
  const float scale_log2e = 0.125f * 1.4426950408889634f;
  flash_attention_kernel<<<grid, kFaThreads, kFaSmemBytes, s>>>(tmap, o, (int)m, dim, scale_log2e, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
