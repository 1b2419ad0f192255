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
//   warps 2..5  epilogue: each thread owns one accumulator row (one TMEM lane) and
//               walks its 256 columns in chunks of 32 while the issuer already fills
//               the other accumulator
// Each CTA owns a block of 128 rows at a time and sweeps all column tiles in ascending
// order (so an epilogue can keep per-row state in registers); row blocks are handed
// out round-robin over a grid of at most one CTA per SM.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace lv {

constexpr int kGemmBM = 128;
constexpr int kGemmBN = 256;
constexpr int kGemmBK = 64;
constexpr int kGemmStages = 4;
constexpr int kGemmThreads = 192;
constexpr int kGemmTileABytes = kGemmBM * kGemmBK * 2;
constexpr int kGemmTileBBytes = kGemmBN * kGemmBK * 2;
constexpr int kGemmStageBytes = kGemmTileABytes + kGemmTileBBytes;
constexpr int kGemmSmemBytes = kGemmStages * kGemmStageBytes + 256 + 1024;  // + barriers + alignment slack

struct GemmBarriers {
  uint64_t full[kGemmStages];
  uint64_t empty[kGemmStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t teardown;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

template <class Epi>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               int m_rows, int n_cols, int k_dim, Epi epi, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kGemmStages * kGemmTileABytes;
  GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem + kGemmStages * kGemmStageBytes);

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
      mbar_init(&bars->tmem_empty[b], 4);
    }
    mbar_init(&bars->teardown, 1);
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_b);
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
      for (int mb = blockIdx.x; mb < num_m_blocks && ok; mb += gridDim.x) {
        for (int nt = 0; nt < num_n_tiles && ok; ++nt) {
          for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait(&bars->empty[stage], phase ^ 1u, ctl)) { ok = false; break; }
            mbar_expect_tx(&bars->full[stage], kGemmStageBytes);
            tma_load_2d(smem_a + stage * kGemmTileABytes, &tmap_a, &bars->full[stage], kb * kGemmBK, mb * kGemmBM);
            tma_load_2d(smem_b + stage * kGemmTileBBytes, &tmap_b, &bars->full[stage], kb * kGemmBK, nt * kGemmBN);
            ++issued;
            if (++stage == kGemmStages) { stage = 0; phase ^= 1u; }
          }
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
      for (int mb = blockIdx.x; mb < num_m_blocks && ok; mb += gridDim.x) {
        for (int nt = 0; nt < num_n_tiles && ok; ++nt, ++tile_iter) {
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
    const int row_in_tile = quarter * 32 + lane;
    uint32_t tile_iter = 0;
    bool ok = true;
    for (int mb = blockIdx.x; mb < num_m_blocks && ok; mb += gridDim.x) {
      const int row = mb * kGemmBM + row_in_tile;
      typename Epi::State st;
      epi.begin(st, row);
      for (int nt = 0; nt < num_n_tiles; ++nt, ++tile_iter) {
        const uint32_t ab = tile_iter & 1u;
        const uint32_t ab_phase = (tile_iter >> 1) & 1u;
        if (!mbar_wait_warp(&bars->tmem_full[ab], ab_phase, ctl)) { ok = false; break; }
        tc_fence_after();
        const uint32_t t_addr = tmem_base + ((quarter * 32u) << 16) + ab * kGemmBN;
#pragma unroll 1
        for (int c = 0; c < kGemmBN / 32; ++c) {
          uint32_t acc[32];
          tmem_ld32(t_addr + c * 32, acc);
          tmem_ld_wait();
          epi.consume(st, row, nt * kGemmBN + c * 32, acc);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->tmem_empty[ab]);
      }
      if (ok) epi.finish(st, row);
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
  struct State {};
  __nv_bfloat16* out;
  const __nv_bfloat16* bias;  // may be null
  int m_rows;
  int n_cols;
  long long ld_out;

  __device__ __forceinline__ void begin(State&, int) const {}
  __device__ __forceinline__ void finish(State&, int) const {}
  __device__ __forceinline__ void consume(State&, int row, int col0, const uint32_t (&acc)[32]) const {
    if (row >= m_rows || col0 >= n_cols) return;
    uint32_t packed[16];
    if (bias != nullptr) {
      const uint4* bp = reinterpret_cast<const uint4*>(bias + col0);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 b = bp[q];
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float lo = __uint_as_float(acc[q * 8 + 2 * i]) + bf16_lo(bw[i]);
          const float hi = __uint_as_float(acc[q * 8 + 2 * i + 1]) + bf16_hi(bw[i]);
          packed[q * 4 + i] = pack_bf16(lo, hi);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) packed[i] = pack_bf16(__uint_as_float(acc[2 * i]), __uint_as_float(acc[2 * i + 1]));
    }
    uint4* op = reinterpret_cast<uint4*>(out + (long long)row * ld_out + col0);
#pragma unroll
    for (int q = 0; q < 4; ++q) op[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
  }
};

// Epilogue of the MLP layers: out[row, col] = bf16(act(acc + bias[col]) + residual[row, col]) with
// act = exact GELU (0.5 x (1 + erf(x / sqrt 2))) or the identity, residual optional.
struct MlpEpilogue {
  struct State {};
  __nv_bfloat16* out;
  const __nv_bfloat16* bias;      // may be null
  const __nv_bfloat16* residual;  // may be null, same shape and pitch as out
  int m_rows;
  int n_cols;
  long long ld_out;
  int gelu;

  __device__ __forceinline__ void begin(State&, int) const {}
  __device__ __forceinline__ void finish(State&, int) const {}
  __device__ __forceinline__ void consume(State&, int row, int col0, const uint32_t (&acc)[32]) const {
    if (row >= m_rows || col0 >= n_cols) return;
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(acc[i]);
    if (bias != nullptr) {
      const uint4* bp = reinterpret_cast<const uint4*>(bias + col0);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 b = bp[q];
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[q * 8 + 2 * i] += bf16_lo(bw[i]);
          v[q * 8 + 2 * i + 1] += bf16_hi(bw[i]);
        }
      }
    }
    if (gelu) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = 0.5f * v[i] * (1.0f + erff(v[i] * 0.70710678118654752f));
    }
    if (residual != nullptr) {
      const uint4* rp = reinterpret_cast<const uint4*>(residual + (long long)row * ld_out + col0);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 r = rp[q];
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[q * 8 + 2 * i] += bf16_lo(rw[i]);
          v[q * 8 + 2 * i + 1] += bf16_hi(rw[i]);
        }
      }
    }
    uint4* op = reinterpret_cast<uint4*>(out + (long long)row * ld_out + col0);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      op[q] = make_uint4(pack_bf16(v[q * 8], v[q * 8 + 1]), pack_bf16(v[q * 8 + 2], v[q * 8 + 3]),
                         pack_bf16(v[q * 8 + 4], v[q * 8 + 5]), pack_bf16(v[q * 8 + 6], v[q * 8 + 7]));
  }
};

// Epilogue: running argmax over columns of acc[row, col] * inv_norm_b[col]; at the end
// best_idx[row] = col_ids[argmax], best_val[row] = max * inv_norm_a[row].
// Columns are visited in ascending order and only a strictly larger value replaces the
// current best, so exact ties resolve to the lowest column.
struct ArgmaxEpilogue {
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
