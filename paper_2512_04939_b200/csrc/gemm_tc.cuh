// Persistent bf16 GEMM mainloop on the 5th-generation tensor cores:
//   C[m, n] = sum_k A[m, k] * B[n, k]        (both operands K-major, fp32 accumulate)
// with a pluggable epilogue that consumes the accumulator straight out of tensor memory.
//
// Used by (a) the projection layers of the attention block (plain epilogue: + bias,
// round to bf16, store) and (b) the src->anchor cosine matching (epilogue keeps a
// running row argmax, so the |Src| x |Dst| score matrix never exists in memory).
//
// Shape of one CTA:
//   warp 0      TMA producer (one elected lane): A tile 128 x 64 and B tile 256 x 64 per
//               k-block into a 4-stage shared-memory ring (128-byte swizzle)
//   warp 1      MMA issuer (one elected lane): 4 x tcgen05.mma M128 N256 K16 per k-block
//               into one of two 256-column fp32 accumulators in tensor memory
//   warps 2..   epilogue: each thread owns one accumulator row (one TMEM lane) and
//               walks its columns in chunks while the issuer already fills the other
//               accumulator.  An epilogue with per-row state (the argmax) runs on four
//               warps, one per 32-lane quarter, over all 256 columns.  An epilogue that
//               writes a matrix runs on eight (two per quarter, 128 columns each) and
//               hands every 64-column chunk back as bf16; the warp parks its 32 x 64
//               block in shared memory (128-byte swizzle) and one lane sends it to
//               global memory as a TMA store, so rows leave the SM as whole 128-byte
//               lines
// Tile order.  With a row-state epilogue each CTA owns a block of 128 rows at a time and
// sweeps all column tiles in ascending order (the state stays in registers); row blocks
// are handed out round-robin over a grid of at most one CTA per SM.  With a matrix
// epilogue tiles are numbered row block major and dealt round-robin, so the CTAs running
// at one moment share a few row blocks of A and the whole of B stays in L2 - with the
// row-block order and K = 4096 the 148 resident A panels (1 MB each) outgrew L2.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace lv {

constexpr int kGemmBM = 128;
constexpr int kGemmBN = 256;
constexpr int kGemmBK = 64;
constexpr int kGemmStages = 4;
constexpr int kGemmMaxThreads = 320;  // 2 + 8 warps
// Threads of a launch: TMA warp + MMA warp + 4 (row-state epilogue) or 8 (matrix epilogue) warps.
template <class Epi>
constexpr int gemm_threads() {
  return 64 + (Epi::kTileOut ? 256 : 128);
}
constexpr int kGemmTileABytes = kGemmBM * kGemmBK * 2;
constexpr int kGemmTileBBytes = kGemmBN * kGemmBK * 2;
constexpr int kGemmStageBytes = kGemmTileABytes + kGemmTileBBytes;
constexpr int kGemmOutChunkCols = 64;                                   // columns per staged output block
constexpr int kGemmOutBlockBytes = 32 * kGemmOutChunkCols * 2;          // one warp's 32 rows x 64 columns
constexpr int kGemmOutBytes = 8 * kGemmOutBlockBytes;                   // one block per epilogue warp
constexpr int kGemmSmemBytes = kGemmStages * kGemmStageBytes + kGemmOutBytes + 256 + 1024;  // + barriers + slack

struct GemmBarriers {
  uint64_t full[kGemmStages];
  uint64_t empty[kGemmStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t teardown;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

// The i-th tile of this CTA; false once the CTA has run out of tiles.
template <bool kRoundRobinTiles>
__device__ __forceinline__ bool gemm_tile_at(int i, int num_m_blocks, int num_n_tiles, int& mb, int& nt) {
  if constexpr (kRoundRobinTiles) {
    const long long t = (long long)blockIdx.x + (long long)i * gridDim.x;
    if (t >= (long long)num_m_blocks * num_n_tiles) return false;
    mb = (int)(t / num_n_tiles);
    nt = (int)(t % num_n_tiles);
    return true;
  } else {
    const long long b = (long long)blockIdx.x + (long long)(i / num_n_tiles) * gridDim.x;
    if (b >= num_m_blocks) return false;
    mb = (int)b;
    nt = i % num_n_tiles;
    return true;
  }
}

template <class Epi>
__global__ void __launch_bounds__(kGemmMaxThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_out, int m_rows, int n_cols, int k_dim, Epi epi,
               uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kGemmStages * kGemmTileABytes;
  uint8_t* smem_out = smem + kGemmStages * kGemmStageBytes;
  GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem_out + kGemmOutBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_m_blocks = (m_rows + kGemmBM - 1) / kGemmBM;
  const int num_n_tiles = (n_cols + kGemmBN - 1) / kGemmBN;
  const int num_kb = k_dim / kGemmBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGemmStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->tmem_full[b], 1);
      mbar_init(&bars->tmem_empty[b], Epi::kTileOut ? 8 : 4);
    }
    mbar_init(&bars->teardown, 1);
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_b);
    if constexpr (Epi::kTileOut) tma_prefetch_desc(&tmap_out);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const WaitCtl ctl{&bars->abort_flag, status};

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued = 0;
      bool ok = true;
      int mb, nt;
      for (int i = 0; ok && gemm_tile_at<Epi::kTileOut>(i, num_m_blocks, num_n_tiles, mb, nt); ++i) {
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&bars->empty[stage], phase ^ 1u, ctl)) { ok = false; break; }
          mbar_expect_tx(&bars->full[stage], kGemmStageBytes);
          tma_load_2d(smem_a + stage * kGemmTileABytes, &tmap_a, &bars->full[stage], kb * kGemmBK, mb * kGemmBM);
          tma_load_2d(smem_b + stage * kGemmTileBBytes, &tmap_b, &bars->full[stage], kb * kGemmBK, nt * kGemmBN);
          ++issued;
          if (++stage == kGemmStages) { stage = 0; phase ^= 1u; }
        }
      }
      // Drain: every load this thread issued must have landed before the CTA may exit.
      const uint32_t n_drain = issued < (uint32_t)kGemmStages ? issued : (uint32_t)kGemmStages;
      for (uint32_t i = 0; i < n_drain; ++i) {
        // walk back over the most recently used stages
        int s = stage - 1 - (int)i;
        uint32_t ph = phase;
        while (s < 0) { s += kGemmStages; ph ^= 1u; }
        const long long t0 = clock64();
        while (!mbar_try_wait(&bars->full[s], ph)) {
          if (clock64() - t0 > kTimeoutCycles) { atomicOr(status, kStatusTimeout); break; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc_bf16(kGemmBM, kGemmBN, false, false);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t tile_iter = 0;
      bool ok = true;
      int mb, nt;
      for (int i = 0; ok && gemm_tile_at<Epi::kTileOut>(i, num_m_blocks, num_n_tiles, mb, nt); ++i, ++tile_iter) {
        const uint32_t ab = tile_iter & 1u;
        const uint32_t ab_phase = (tile_iter >> 1) & 1u;
        if (!mbar_wait(&bars->tmem_empty[ab], ab_phase ^ 1u, ctl)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * kGemmBN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&bars->full[stage], phase, ctl)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = smem_desc_sw128(smem_u32(smem_a + stage * kGemmTileABytes), 16, 1024);
          const uint64_t b_desc = smem_desc_sw128(smem_u32(smem_b + stage * kGemmTileBBytes), 16, 1024);
#pragma unroll
          for (int k = 0; k < kGemmBK / 16; ++k) {
            // +32 bytes along K inside the swizzled row = +2 in descriptor units
            umma_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&bars->empty[stage]);
          if (++stage == kGemmStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&bars->tmem_full[ab]);
      }
      if (!ok) {
        // make sure no MMA is still in flight before tensor memory is released
        umma_commit(&bars->teardown);
        const long long t0 = clock64();
        while (!mbar_try_wait(&bars->teardown, 0)) {
          if (clock64() - t0 > kTimeoutCycles) break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const uint32_t quarter = warp & 3u;  // TMEM lanes 32*quarter .. 32*quarter+31
    const uint32_t half = (uint32_t)(warp - 2) >> 2;  // which 128 columns (matrix epilogue only)
    const int row_in_tile = quarter * 32 + lane;
    uint32_t tile_iter = 0;
    uint32_t chunk_iter = 0;
    typename Epi::State st;
    int mb, nt;
    for (int i = 0; gemm_tile_at<Epi::kTileOut>(i, num_m_blocks, num_n_tiles, mb, nt); ++i, ++tile_iter) {
      const int row = mb * kGemmBM + row_in_tile;
      if (nt == 0) epi.begin(st, row);
      const uint32_t ab = tile_iter & 1u;
      const uint32_t ab_phase = (tile_iter >> 1) & 1u;
      if (!mbar_wait_warp(&bars->tmem_full[ab], ab_phase, ctl)) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((quarter * 32u) << 16) + ab * kGemmBN;
      if constexpr (Epi::kTileOut) {
        const int warp_row0 = mb * kGemmBM + (int)quarter * 32;
        uint8_t* block = smem_out + (warp - 2) * kGemmOutBlockBytes;
#pragma unroll 1
        for (int c = (int)half * 2; c < (int)half * 2 + 2; ++c) {
          const int col0 = nt * kGemmBN + c * kGemmOutChunkCols;
          if (col0 >= n_cols || warp_row0 >= m_rows) break;  // nothing of this block exists (warp-uniform)
          uint32_t acc[64];
          tmem_ld32(t_addr + c * 64, reinterpret_cast<uint32_t(&)[32]>(acc[0]));
          tmem_ld32(t_addr + c * 64 + 32, reinterpret_cast<uint32_t(&)[32]>(acc[32]));
          tmem_ld_wait();
          uint32_t packed[32];
          epi.transform(row, col0, acc, packed);
          // The previous store out of this warp's staging block must be done reading it.
          if (chunk_iter != 0) {
            if (lane == 0) bulk_wait_group_read<0>();
            __syncwarp();
          }
          // Row `lane` of the block, its eight 16-byte units permuted the way the 128-byte swizzle
          // of the store's tensor map expects (unit u of row r sits at u ^ (r mod 8)).
          uint8_t* my_row = block + lane * 128;
#pragma unroll
          for (int u = 0; u < 8; ++u)
            *reinterpret_cast<uint4*>(my_row + ((u ^ (lane & 7)) << 4)) =
                make_uint4(packed[4 * u], packed[4 * u + 1], packed[4 * u + 2], packed[4 * u + 3]);
          fence_proxy_async_shared();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tmap_out, block, col0, warp_row0);
            bulk_commit_group();
          }
          ++chunk_iter;
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < kGemmBN / 32; ++c) {
          uint32_t acc[32];
          tmem_ld32(t_addr + c * 32, acc);
          tmem_ld_wait();
          epi.consume(st, row, nt * kGemmBN + c * 32, acc);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->tmem_empty[ab]);
      if (nt == num_n_tiles - 1) epi.finish(st, row);
    }
    // Shared memory must outlive every store that still reads it.
    if constexpr (Epi::kTileOut) {
      if (lane == 0) bulk_wait_group_all();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ----------------------------------------------------------------------------------------
// Epilogue: out[row, col] = bf16(acc + bias[col])
struct LinearEpilogue {
  static constexpr bool kTileOut = true;
  struct State {};
  const __nv_bfloat16* bias;  // may be null
  int m_rows;
  int n_cols;
  int scale_begin, scale_end;  // output columns [scale_begin, scale_end) are multiplied by `scale`
  float scale;

  __device__ __forceinline__ void begin(State&, int) const {}
  __device__ __forceinline__ void finish(State&, int) const {}
  // 64 accumulator columns of one row -> 32 bf16 pairs
  __device__ __forceinline__ void transform(int, int col0, const uint32_t (&acc)[64], uint32_t (&packed)[32]) const {
    const float sc = (col0 >= scale_begin && col0 < scale_end) ? scale : 1.0f;
    if (bias != nullptr) {
      const uint4* bp = reinterpret_cast<const uint4*>(bias + col0);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const uint4 b = __ldg(bp + q);
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float lo = (__uint_as_float(acc[q * 8 + 2 * i]) + bf16_lo(bw[i])) * sc;
          const float hi = (__uint_as_float(acc[q * 8 + 2 * i + 1]) + bf16_hi(bw[i])) * sc;
          packed[q * 4 + i] = pack_bf16(lo, hi);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        packed[i] = pack_bf16(__uint_as_float(acc[2 * i]) * sc, __uint_as_float(acc[2 * i + 1]) * sc);
    }
  }
};

// GELU with the error function, x Phi(x) = 0.5 x (1 + erf(x / sqrt 2)).  erf comes from the five-term
// rational approximation of Abramowitz & Stegun (7.1.26): for z >= 0, 1 - erf(z) = P(t) exp(-z^2) with
// t = 1 / (1 + p z), absolute error below 1.5e-7 - three orders of magnitude under the bf16 rounding
// of the result.  With e = P(t) exp(-z^2), z = |x| / sqrt 2: the result is x (1 - e/2) for x >= 0 and
// x e/2 for x < 0, so the negative side has no cancellation.
__device__ __forceinline__ float gelu_erf(float x) {
  const float z = fabsf(x) * 0.70710678118654752f;
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, z, 1.0f)));
  float p = fmaf(1.061405429f, t, -1.453152027f);
  p = fmaf(p, t, 1.421413741f);
  p = fmaf(p, t, -0.284496736f);
  p = fmaf(p, t, 0.254829592f);
  p *= t;
  float ex;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(ex) : "f"(z * z * -1.4426950408889634f));
  const float h = 0.5f * p * ex;
  return x * (x >= 0.0f ? 1.0f - h : h);
}

// Epilogue of the MLP layers: out[row, col] = bf16(act(acc + bias[col]) + residual[row, col]) with
// act = erf-GELU (0.5 x (1 + erf(x / sqrt 2))) or the identity, residual optional.
struct MlpEpilogue {
  static constexpr bool kTileOut = true;
  struct State {};
  const __nv_bfloat16* bias;      // may be null
  const __nv_bfloat16* residual;  // may be null, same shape as the output with pitch ld_res
  int m_rows;
  int n_cols;
  long long ld_res;
  int gelu;

  __device__ __forceinline__ void begin(State&, int) const {}
  __device__ __forceinline__ void finish(State&, int) const {}
  __device__ __forceinline__ void transform(int row, int col0, const uint32_t (&acc)[64],
                                            uint32_t (&packed)[32]) const {
    const bool has_res = residual != nullptr && row < m_rows;
    const uint4* bp = reinterpret_cast<const uint4*>(bias + col0);
    const uint4* rp = reinterpret_cast<const uint4*>(residual + (long long)row * ld_res + col0);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      float v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(acc[q * 8 + i]);
      if (bias != nullptr) {
        const uint4 b = __ldg(bp + q);
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[2 * i] += bf16_lo(bw[i]);
          v[2 * i + 1] += bf16_hi(bw[i]);
        }
      }
      if (gelu) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = gelu_erf(v[i]);
      }
      if (has_res) {
        const uint4 r = rp[q];
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[2 * i] += bf16_lo(rw[i]);
          v[2 * i + 1] += bf16_hi(rw[i]);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) packed[q * 4 + i] = pack_bf16(v[2 * i], v[2 * i + 1]);
    }
  }
};

// Epilogue: running argmax over columns of acc[row, col] * inv_norm_b[col]; at the end
// best_idx[row] = col_ids[argmax], best_val[row] = max * inv_norm_a[row].
// Columns are visited in ascending order and only a strictly larger value replaces the
// current best, so exact ties resolve to the lowest column.
struct ArgmaxEpilogue {
  static constexpr bool kTileOut = false;
  struct State {
    float best;
    int best_col;
  };
  const float* inv_norm_a;  // [m_rows]
  const float* inv_norm_b;  // [n_cols rounded up to 256], padding = 0
  const int* col_ids;       // [n_cols]
  int* best_idx;            // [m_rows]
  float* best_val;          // [m_rows]
  int m_rows;
  int n_cols;

  __device__ __forceinline__ void begin(State& st, int) const {
    st.best = -INFINITY;
    st.best_col = 0;
  }
  __device__ __forceinline__ void consume(State& st, int, int col0, const uint32_t (&acc)[32]) const {
    const int valid = n_cols - col0;  // columns of this chunk that exist
    if (valid <= 0) return;
    const float4* np = reinterpret_cast<const float4*>(inv_norm_b + col0);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 w = __ldg(np + q);
      const float wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = q * 4 + i;
        const float v = __uint_as_float(acc[c]) * wv[i];
        if (c < valid && v > st.best) {
          st.best = v;
          st.best_col = col0 + c;
        }
      }
    }
  }
  __device__ __forceinline__ void finish(State& st, int row) const {
    if (row >= m_rows) return;
    best_idx[row] = col_ids[st.best_col];
    best_val[row] = st.best * inv_norm_a[row];
  }
};

}  // namespace lv
