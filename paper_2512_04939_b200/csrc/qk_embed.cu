// Per-head normalisation and 2-D rotary position embedding of the projected queries and keys, in
// place on the [M, 3D] Q/K/V buffer between the QKV projection and the attention core.  The paper
// prints neither; VGGT's attention, which the method keeps (Sec. 3.1), has both, so they are an
// option of the global attention layer.
//
//   normalisation  LayerNorm over the 64 channels of each head (population variance), affine with
//                  one gamma/beta pair for the queries and one for the keys
//   rotation       the head's channels split into two halves of 32: the first turns with the row
//                  position, the second with the column position; in a half, channel i (< 16) and
//                  channel i + 16 form a plane rotated by position * base^(-i/16)
//   positions      row r of the merged sequence carries the position of the token that owns it
//                  (kept_idx[r]); special tokens sit at (0, 0), the patch at grid row py, column
//                  px at (py + 1, px + 1)
//
// One warp per row, HBM-bound: a lane owns 8 consecutive channels (16 bytes), 8 lanes cover a head,
// one warp instruction moves four heads.  Statistics need three shuffles over the 8 lanes of a
// head; the rotation partner of a lane is two lanes away.  All arithmetic in fp32, one rounding.
#include "common.cuh"
#include "runtime.h"

namespace lv {

constexpr int kEmbedThreads = 256;
constexpr int kEmbedRowsPerCta = kEmbedThreads / 32;

struct EmbedParams {
  const __nv_bfloat16* q_gamma;  // [64] or null: no normalisation
  const __nv_bfloat16* q_beta;
  const __nv_bfloat16* k_gamma;
  const __nv_bfloat16* k_beta;
  float eps;
  int rope;                      // 0: no rotation
  float log2_base;
  int tokens_frame, n_special, grid_w;
};

__global__ void __launch_bounds__(kEmbedThreads)
qk_embed_kernel(__nv_bfloat16* __restrict__ qkv, const int* __restrict__ kept_idx, long long m_rows,
                long long n_tokens, EmbedParams p, uint32_t* status) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kEmbedRowsPerCta + (threadIdx.x >> 5);
  if (row >= m_rows) return;
  const int j = lane & 7;  // which 8 channels of the head: 8j .. 8j+7

  // rotation of this lane's 8 channels: the same for every head and for queries and keys
  float cs[8], sn[8];
  const bool first = (j & 2) == 0;  // channels 0..15 of their half: out = v cos - partner sin
  if (p.rope) {
    long long token = kept_idx[row];
    if (token < 0 || token >= n_tokens) {
      if (lane == 0) atomicOr(status, kStatusBounds);
      token = 0;
    }
    const int t = (int)(token % p.tokens_frame);
    int pos = 0;
    if (t >= p.n_special) {
      const int patch = t - p.n_special;
      pos = (j < 4) ? patch / p.grid_w + 1 : patch % p.grid_w + 1;  // first half: row, second: column
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int plane = 8 * (j & 1) + e;  // i in 0..15
      const float theta = exp2f(-(float)plane * (1.0f / 16.0f) * p.log2_base);
      // angles stay below 2^8 rad (grids of at most 128 x 64), where the fast path is good to ~1e-5 absolute,
      // two orders under the rounding of the bf16 result
      __sincosf((float)pos * theta, &sn[e], &cs[e]);
      if (first) sn[e] = -sn[e];
    }
  }

  float gq[8], bq[8], gk[8], bk[8];
  const bool norm = p.q_gamma != nullptr;
  if (norm) {
    const uint4 a = reinterpret_cast<const uint4*>(p.q_gamma)[j], b = reinterpret_cast<const uint4*>(p.q_beta)[j];
    const uint4 c = reinterpret_cast<const uint4*>(p.k_gamma)[j], d = reinterpret_cast<const uint4*>(p.k_beta)[j];
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, dw[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      gq[2 * i] = bf16_lo(aw[i]); gq[2 * i + 1] = bf16_hi(aw[i]);
      bq[2 * i] = bf16_lo(bw[i]); bq[2 * i + 1] = bf16_hi(bw[i]);
      gk[2 * i] = bf16_lo(cw[i]); gk[2 * i + 1] = bf16_hi(cw[i]);
      bk[2 * i] = bf16_lo(dw[i]); bk[2 * i + 1] = bf16_hi(dw[i]);
    }
  }

  // Q occupies channels [0, 1024) of the row, K [1024, 2048): 8 steps of 4 heads each
  uint4* base = reinterpret_cast<uint4*>(qkv + row * 3072);
  uint4 raws[8];
#pragma unroll
  for (int step = 0; step < 8; ++step) raws[step] = base[step * 32 + lane];
#pragma unroll
  for (int step = 0; step < 8; ++step) {
    const bool is_k = step >= 4;
    const uint4 raw = raws[step];
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    float v[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = bf16_lo(w[i]);
      v[2 * i + 1] = bf16_hi(w[i]);
    }
    if (norm) {
      float sum = 0.0f;
#pragma unroll
      for (int e = 0; e < 8; ++e) sum += v[e];
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float mean = sum * (1.0f / 64.0f);
      float ss = 0.0f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        v[e] -= mean;
        ss = fmaf(v[e], v[e], ss);
      }
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float rstd = rsqrtf(ss * (1.0f / 64.0f) + p.eps);
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e] * rstd, is_k ? gk[e] : gq[e], is_k ? bk[e] : bq[e]);
    }
    if (p.rope) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float partner = __shfl_xor_sync(0xffffffffu, v[e], 2);
        v[e] = fmaf(partner, sn[e], v[e] * cs[e]);
      }
    }
    if (is_k) {
      // the attention kernel expects K with the softmax scale folded in (the projection before this
      // pass left it out, so that the normalisation sees K itself)
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] *= kKeyScaleLog2e;
    }
    base[step * 32 + lane] = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]),
                                        pack_bf16(v[6], v[7]));
  }
}

cudaError_t launch_qk_embed(const litevggt_ctx* ctx, __nv_bfloat16* qkv, const int* kept_idx, long long m,
                            const __nv_bfloat16* q_gamma, const __nv_bfloat16* q_beta, const __nv_bfloat16* k_gamma,
                            const __nv_bfloat16* k_beta, float eps, int rope, float rope_base, cudaStream_t s,
                            int* launches) {
  if (m == 0 || (q_gamma == nullptr && !rope)) return cudaSuccess;
  const Sizes& z = ctx->sz;
  EmbedParams p;
  p.q_gamma = q_gamma;
  p.q_beta = q_beta;
  p.k_gamma = k_gamma;
  p.k_beta = k_beta;
  p.eps = eps;
  p.rope = rope;
  p.log2_base = log2f(rope_base);
  p.tokens_frame = z.tokens_frame;
  p.n_special = (int)z.n_special;
  p.grid_w = (int)z.grid_w;
  const unsigned blocks = (unsigned)((m + kEmbedRowsPerCta - 1) / kEmbedRowsPerCta);
  qk_embed_kernel<<<blocks, kEmbedThreads, 0, s>>>(qkv, kept_idx, m, z.n_tokens, p, ctx->ws.status);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
