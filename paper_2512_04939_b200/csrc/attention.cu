// Global self-attention over the merged token sequence (Sec. 3.1: the frame-global
// attention layer; after merging it runs over M instead of N tokens).  Per head
//   O = softmax(Q K^T / sqrt(64)) V,      non-causal, no mask,
// computed flash-style: scores never leave the SM.
//
// One CTA = 256 query rows (two tiles of 128) of one head, sweeping all keys in tiles of
// 128 that are consumed as two halves of 64 ("steps").  Warp roles (20 warps):
//   warps 0-15  softmax.  Warp w works on query tile t = w / 8, TMEM lane quarter w % 4 (one
//               thread = one query row) and the column half c = (w / 4) % 2 of every step:
//               32 of the step's 64 scores per row.  The two threads of a row swap their
//               partial row maxima through shared memory once per step.  Four softmax warps
//               per scheduler keep the special-function unit busy while others wait.
//   warp  16    MMA issuer of tile 0 (one elected lane):  S_h = Q K_jh^T  and  O += P_h V_jh
//   warp  17    TMA producer (one elected lane): K_j / V_j through two 4-stage shared-memory rings
//   warp  18    MMA issuer of tile 1 (issuing costs tens of cycles per instruction, so one
//               thread cannot feed both tiles)
//   warp  19    idle
// Tensor memory (512 columns allocated, 480 used):
//   [0,256)    S/P: tile t, half h at column t*128 + h*64.  S_th is 128 x 64 fp32.  A softmax
//              thread reads its 32 columns and writes its 32 probabilities (16 columns of bf16
//              pairs) over the start of the same 32 columns, so P_th sits in columns [0,16) and
//              [32,48) of the half and no thread writes where another one reads; the second MMA
//              takes its A operand from there, 8 columns (16 keys) per instruction.
//   [256,416)  O_0, O_1 (fp32, 80 columns each: 64 output channels, then the row sum - the second
//              MMA's B operand carries a column of ones next to V, so the tensor core adds up
//              exactly the bf16 probabilities that it multiplies with V - and 15 unused columns)
//   [416,480)  Q_0, Q_1 (bf16 pairs, 32 columns each), written once by the softmax threads
//              straight from global memory: Q is the A operand of the first MMA from tensor
//              memory, so only K and V tiles travel through shared memory.
// The two halves of a tile double-buffer the scores: while the softmax threads work on
// half h the tensor core already runs O += P V of the other half and the next Q K^T into
// it.  The MMAs are issued in order, which is what makes the S/P aliasing safe: Q K^T for
// step n+2 is issued after the P V that reads the same columns.
// V tiles are consumed as an MN-major B operand, K tiles as a K-major one, so neither
// needs a transpose.
//
// Softmax arithmetic.  At head dim 64 every score costs 256 tensor flops and one
// exponential, and the special-function unit issues only 16 ex2 per clock per SM (the packed
// bf16x2 / f16x2 forms issue at half the rate, so they give the same 16 results per clock), half of
// what the tensor cores would need.  A fixed share of the exponentials of every row is therefore
// evaluated on the FMA pipes instead: round-to-nearest split x = n + f, |f| <= 1/2, a cubic
// for 2^f (relative error 7.5e-5, far below the bf16 rounding of P) and n added into the
// exponent field.  The share is a build-time constant, kFaPolyPairs of the 16 pairs of scores a
// thread handles per step; 7 measured best in the kernel (on register data alone, 4 warps per
// scheduler: 6 pairs take 182 clocks per 32 scores against 257 with the special-function unit only,
// 8 pairs 220).
// Shared memory: K ring, V ring, and behind the V ring a block of the same size that holds the
// ones column of the P V operand for every ring position (see the kernel).
//
// Key chunks.  All CTAs of a head stream the same K/V, but they drift apart, so their combined
// working set is the head's whole K/V; beyond about a quarter of the L2 that no longer stays
// resident and every CTA would pull its tiles from HBM (measured: 2.4 TB per launch at 520 K
// keys).  Long sequences are therefore swept in chunks of at most kFaChunkTiles key tiles, one
// launch per chunk: a chunk's K/V of one head (16 MiB) stays in L2 while all query blocks pass
// over it.  Every launch starts its accumulators from zero and, at its end, adds its partial
// output rows, row sums and reference to what the earlier chunks left in global memory (fp32,
// round to nearest; a few GB of traffic per launch).  That also bounds the chain of additions
// into one tensor-memory accumulator: carried through all 4067 key tiles of a 520 K-key sweep,
// the accumulator picked up an error that grew in proportion to the number of keys (2.9e-3 of
// the output's RMS at 252 K keys, 5.0e-3 at 520 K, against 2e-4 at 1.5 K).
//
// Softmax reference.  Any per-row constant m may be subtracted from the scores before the
// exponential: the division by the row sum removes it again.  It only has to keep 2^(s - m)
// inside the range of bf16 / fp32, it does not have to be the row maximum.  By Cauchy-Schwarz
// every score of a row is at most B = |q| max_k |k| (K carrying the softmax scale: base-2 units), so
// with m = B all exponents lie in [-2B, 0]; while 2B stays well inside the exponent range of
// fp32 nothing underflows, every probability keeps its 8 significant bits and the fp32
// accumulators their 24.  A small pass over K finds max_k |k|^2 per head before the sweep, each
// softmax thread takes |q|^2 of its row while loading Q, and a warp pair whose rows all have
// B <= kFaFixedRefLimit runs the sweep with a constant reference (in fact with none: the constant
// cancels, see the kernel): no row maximum, no exchange between the two threads of a row, no
// rescaling, and - the softmax scale 1/sqrt(64) log2(e) arriving folded into K - no arithmetic
// between the tensor core's scores and the exponential.  Rows with larger B (scores that could span more than
// the exponent range allows) take the online form: base-2 softmax with a lazily updated reference
// maximum, the running output rescaled only when a row maximum grows by more than 2^8 over the
// reference (the threads then first wait until the tile's last P V has retired).  Both forms equal
// the plain softmax up to rounding.
#include "common.cuh"
#include "runtime.h"

namespace lv {

constexpr int kFaStages = 4;
constexpr int kFaSoftmaxWarps = 16;
constexpr int kFaThreads = (kFaSoftmaxWarps + 4) * 32;
constexpr int kFaTileBytes = 128 * 64 * 2;
constexpr uint32_t kFaColS = 0, kFaColO = 256, kFaColQ = 416;
constexpr uint32_t kFaOCols = 80;  // 64 output channels, the row sum, 15 unused columns
constexpr float kFaRescaleThreshold = 8.0f;
// Largest Cauchy-Schwarz bound B on the base-2 scores of a row for which the fixed reference is
// used.  With the reference left out the probabilities lie in [2^-B, 2^B]: at B = 80 their products
// with |v| >= 2^-20 are normal fp32 numbers (>= 2^-100), and a row sum over 2^20 keys times
// |v| <= 2^20 stays below 2^120, inside fp32; the polynomial exponential is valid to +-120.
#ifndef LV_FA_FIXED_REF_LIMIT
#define LV_FA_FIXED_REF_LIMIT 80.0f
#endif
constexpr float kFaFixedRefLimit = LV_FA_FIXED_REF_LIMIT;
#ifndef LV_FA_CHUNK_TILES
#define LV_FA_CHUNK_TILES 512
#endif
constexpr int kFaChunkTiles = LV_FA_CHUNK_TILES;  // 65536 keys: K and V of one head = 16 MiB
// Of the 16 pairs of scores a thread handles per step, this many take the polynomial exponential
// (fixed-reference form only, where every argument lies in [-kFaFixedRefLimit, kFaFixedRefLimit]).
#ifndef LV_FA_POLY_PAIRS
#define LV_FA_POLY_PAIRS 7
#endif
constexpr int kFaPolyPairs = LV_FA_POLY_PAIRS;

struct FaBarriers {
  uint64_t q_ready;
  uint64_t k_full[kFaStages], k_empty[kFaStages];
  uint64_t v_full[kFaStages], v_empty[kFaStages];
  uint64_t s_full[2][2], p_ready[2][2], pv_done[2], o_done[2];
  uint64_t teardown[2];
  uint32_t tmem_base;
  uint32_t abort_flag;
};
// partial row maxima swapped between the two threads of a row: [step parity][tile][column half][row]
struct FaExchange {
  float row_max[2][2][2][128];
};
constexpr int kFaSmemBytes = 3 * kFaStages * kFaTileBytes + (int)sizeof(FaExchange) + 512 + 1024;

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x for a pair of arguments on the FMA pipes.  Adding 1.5 * 2^23 rounds x to the nearest
// integer n in the low mantissa bits; 2^(x - n) comes from a cubic fitted on [-1/2, 1/2] and
// n is added to the exponent field.  Valid for arguments in [-120, 120].
__device__ __forceinline__ float2 poly_exp2_pair(float2 x) {
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

// Exponentials of 32 scores of a row: p = 2^(s * scale - m_ref), packed to bf16 pairs (the row sum
// is formed by the tensor core from these rounded values).  The first kPoly of the 16 pairs take the
// polynomial on the FMA pipes (callers guarantee arguments above -120 for them), the others the
// special-function unit.
template <int kPoly>
__device__ __forceinline__ void softmax_chunk(const uint32_t (&s)[32], float2 scale2, float2 neg_m2,
                                              uint32_t (&packed)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), scale2, neg_m2);
    float2 p;
    if (i < kPoly) {
      p = poly_exp2_pair(x);
    } else {
      p.x = fast_exp2(x.x);
      p.y = fast_exp2(x.y);
    }
    packed[i] = pack_bf16(p.x, p.y);
  }
}

// The same for scores that arrive already scaled, with no reference to subtract: p = 2^s.
template <int kPoly>
__device__ __forceinline__ void exp2_chunk(const uint32_t (&s)[32], uint32_t (&packed)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 x = make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1]));
    float2 p;
    if (i < kPoly) {
      p = poly_exp2_pair(x);
    } else {
      p.x = fast_exp2(x.x);
      p.y = fast_exp2(x.y);
    }
    packed[i] = pack_bf16(p.x, p.y);
  }
}

__device__ __forceinline__ void pair_barrier(int id) {  // the two warps of one (tile, lane quarter)
  asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory");
}

// kFirst / kLast: this launch holds the first / the last key chunk of the sweep.
template <bool kFirst, bool kLast>
__global__ void __launch_bounds__(kFaThreads, 1)
flash_attention_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const __nv_bfloat16* __restrict__ qkv,
                       __nv_bfloat16* __restrict__ o, float* __restrict__ o_state, float* __restrict__ ml_state,
                       const float* __restrict__ k_norm2_max, int seq_len, int dim, int tile_begin, int tile_end,
                       uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_k = smem;
  uint8_t* smem_v = smem_k + kFaStages * kFaTileBytes;
  uint8_t* smem_ones = smem_v + kFaStages * kFaTileBytes;  // mirrors the V ring, see below
  FaExchange* xchg = reinterpret_cast<FaExchange*>(smem_ones + kFaStages * kFaTileBytes);
  FaBarriers* bars = reinterpret_cast<FaBarriers*>(xchg + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // blockIdx.z selects one of the independent sequences of seq_len rows laid back to back (the
  // global layer has one; a frame-local layer has one per frame)
  const int row_base = blockIdx.z * seq_len;
  const int q0 = blockIdx.x * 256;  // within the sequence
  const int head = blockIdx.y;
  // this launch covers key tiles [tile_begin, tile_end) of ceil(seq_len / 128); local tile j is
  // key tile tile_begin + j, step n = local tile n/2, half n%2
  const int n_kv = tile_end - tile_begin;
  const int n_steps = 2 * n_kv;
  constexpr bool first_chunk = kFirst;
  constexpr bool last_chunk = kLast;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_ready, kFaSoftmaxWarps);
    for (int s = 0; s < kFaStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 2);  // both MMA issuers release a stage
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 2);
    }
    for (int t = 0; t < 2; ++t) {
      for (int h = 0; h < 2; ++h) {
        mbar_init(&bars->s_full[t][h], 1);
        mbar_init(&bars->p_ready[t][h], 8);
      }
      mbar_init(&bars->pv_done[t], 1);
      mbar_init(&bars->o_done[t], 1);
    }
    mbar_init(&bars->teardown[0], 1);
    mbar_init(&bars->teardown[1], 1);
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_qkv);
  }
  // The row sums come out of the second MMA: its B operand is 80 columns wide, V's 64 channels and,
  // one descriptor stride (the size of the V ring) further on, a block whose first column is 1 and
  // whose other columns are 0, so accumulator column 64 collects sum_k P[row, k] of exactly the bf16
  // probabilities that multiply V.  The block is laid out like a V tile (128-byte rows, 16-byte
  // chunks XOR-swizzled with the row index modulo 8) and repeated for every ring position.
  for (int i = threadIdx.x; i < kFaStages * kFaTileBytes / 16; i += kFaThreads) {
    const int r = i >> 3, chunk = i & 7;  // 128-byte row, 16-byte chunk within it
    const uint32_t first = chunk == (r & 7) ? 0x00003f80u : 0u;  // bf16 1.0 in logical column 0
    reinterpret_cast<uint4*>(smem_ones)[i] = make_uint4(first, 0u, 0u, 0u);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes, read by the MMA
  if (warp == 16) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const WaitCtl ctl{&bars->abort_flag, status};

  if (warp == 17) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      uint32_t k_issued = 0, v_issued = 0;
      for (int j = 0; j < n_kv; ++j) {
        const int stage = j % kFaStages;
        const uint32_t phase = (uint32_t)(j / kFaStages) & 1u;
        if (!mbar_wait(&bars->k_empty[stage], phase ^ 1u, ctl)) break;
        mbar_expect_tx(&bars->k_full[stage], kFaTileBytes);
        tma_load_2d(smem_k + stage * kFaTileBytes, &tmap_qkv, &bars->k_full[stage], dim + head * 64,
                    row_base + (tile_begin + j) * 128);
        ++k_issued;
        if (!mbar_wait(&bars->v_empty[stage], phase ^ 1u, ctl)) break;
        mbar_expect_tx(&bars->v_full[stage], kFaTileBytes);
        tma_load_2d(smem_v + stage * kFaTileBytes, &tmap_qkv, &bars->v_full[stage], 2 * dim + head * 64,
                    row_base + (tile_begin + j) * 128);
        ++v_issued;
      }
      // every load issued by this thread must have landed before the CTA may exit
      drain_ring(bars->k_full, k_issued, status);
      drain_ring(bars->v_full, v_issued, status);
    }
  } else if (warp == 16 || warp == 18) {
    // ------------------------------------------------------------------ MMA issuer of tile t
    if (elect_one()) {
      const int t = warp == 16 ? 0 : 1;
      constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 64, false, false);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(128, kFaOCols, false, true);
      const uint32_t s_col = tmem_base + kFaColS + t * 128;
      const uint32_t o_col = tmem_base + kFaColO + t * kFaOCols;
      const uint32_t q_col = tmem_base + kFaColQ + t * 32;
      // S_h = Q (tensor memory) x K[64h .. 64h+63]^T (shared memory, K-major); 4 steps of 16 channels
      // the descriptors are linear in the shared-memory address (its 16-byte units sit in the low
      // bits and cannot carry out of their field), so a stage / half is one addition away
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem_k), 16, 1024);
      const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem_v), kFaStages * kFaTileBytes, 1024);
      auto issue_qk = [&](int h, int stage) {
        const uint64_t b_desc = k_desc0 + (uint64_t)((stage * kFaTileBytes + h * 8192) >> 4);
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_ts(s_col + h * 64, q_col + k * 8, b_desc + 2 * k, idesc_qk, k != 0 ? 1u : 0u);
        umma_commit(&bars->s_full[t][h]);
      };
      bool ok = mbar_wait(&bars->q_ready, 0, ctl);
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
        if (!last && !mbar_wait(&bars->k_full[next_stage], next_phase, ctl)) { ok = false; break; }
        for (int h = 0; h < 2; ++h) {
          if (!mbar_wait(&bars->p_ready[t][h], j & 1, ctl)) { ok = false; break; }
          tc_fence_after();
          // 64 keys of V_j (64 rows of 128 bytes = 8192 bytes per half), 16 keys per instruction:
          // 8 TMEM columns of P (keys 0-31 in columns [0,16) of the half, keys 32-63 in [32,48)),
          // 2048 bytes of V
          // second 64-column block of B = the ones block, one V ring further on
          const uint64_t v_desc = v_desc0 + (uint64_t)((stage * kFaTileBytes + h * 8192) >> 4);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ts(o_col, s_col + h * 64 + (k >> 1) * 32 + (k & 1) * 8, v_desc + 128 * k, idesc_pv,
                    (j | h | k) != 0 ? 1u : 0u);  // every launch starts its accumulators from zero
          if (last) {
            // no further Q K^T follows whose completion would tell the softmax threads that this
            // P V has retired
            umma_commit(&bars->pv_done[t]);
            if (h == 1) umma_commit(&bars->o_done[t]);
          } else {
            issue_qk(h, next_stage);
          }
        }
        if (!ok) break;
        umma_commit(&bars->v_empty[stage]);
        if (!last) umma_commit(&bars->k_empty[next_stage]);
        stage = next_stage;
        phase = next_phase;
      }
      if (!ok) {
        umma_commit(&bars->teardown[t]);
        const long long t0 = clock64();
        while (!mbar_try_wait(&bars->teardown[t], 0)) {
          if (clock64() - t0 > kTimeoutCycles) break;
        }
      }
    }
  } else if (warp < kFaSoftmaxWarps) {
    // ------------------------------------------------------------------ softmax warps
    const int t = warp >> 3;
    const int c = (warp >> 2) & 1;
    const uint32_t quarter = warp & 3u;
    const int barrier_id = 1 + t * 4 + (int)quarter;
    const int row_in_tile = (int)quarter * 32 + lane;
    const uint32_t lane_base = (quarter * 32u) << 16;
    const int row_local = q0 + t * 128 + row_in_tile;
    const bool row_live = row_local < seq_len;
    const int row = row_base + row_local;  // global row of qkv / o
    const uint32_t s_addr = tmem_base + lane_base + kFaColS + t * 128;
    const uint32_t o_addr = tmem_base + lane_base + kFaColO + t * kFaOCols + c * 32;
    const uint32_t l_addr = tmem_base + lane_base + kFaColO + t * kFaOCols + 64;  // row sum column (+15 unused)
    float q_norm2 = 0.0f;  // |q|^2 of the whole row, summed in the same order by both of its threads
    bool fixed_ref;
    {
      // this thread's half (32 channels) of its query row goes to tensor memory
      uint32_t qreg[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) qreg[i] = 0u;
      if (row_live) {
        const uint4* src = reinterpret_cast<const uint4*>(qkv + (size_t)row * 3 * dim + head * 64);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 v = __ldg(src + i);
          const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            q_norm2 = fmaf(bf16_lo(w[e]), bf16_lo(w[e]), q_norm2);
            q_norm2 = fmaf(bf16_hi(w[e]), bf16_hi(w[e]), q_norm2);
          }
          if ((i >> 2) == c) {
            qreg[4 * (i & 3)] = v.x; qreg[4 * (i & 3) + 1] = v.y; qreg[4 * (i & 3) + 2] = v.z; qreg[4 * (i & 3) + 3] = v.w;
          }
        }
      }
      // Cauchy-Schwarz bound on this row's scores (K carries the softmax scale, so the scores are in
      // base-2 units already); both threads of a row hold the same value, and both warps of a pair
      // vote over the same 32 rows, so they agree on the form they run
      const float score_bound = sqrtf(q_norm2 * k_norm2_max[blockIdx.z * gridDim.y + head]);
      fixed_ref = __all_sync(0xffffffffu, score_bound <= kFaFixedRefLimit ? 1 : 0) != 0;
      tmem_st16(tmem_base + lane_base + kFaColQ + t * 32 + c * 16, qreg);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->q_ready);
    }
    float m_ref = -INFINITY;  // reference, in the scores' own (base-2) units
    bool ok = true;
    int pair_syncs = 0;  // both warps of a pair must pass the same number of pair barriers
    if (fixed_ref) {
      // ---- fixed reference.  The scores all lie inside [-score_bound, score_bound]; the constant
      // 2^-score_bound that would bring the exponents to [-2 score_bound, 0] cancels between numerator
      // and row sum, so it is not applied: reference 0, and the scores go into the exponential as
      // they come out of the tensor core.
      m_ref = 0.0f;
      pair_syncs = n_steps;  // this form has no pair barriers
      // One step = this thread's 32 scores of one half of a key tile.  Only the last tile of a
      // launch can reach past the sequence, so the steps before it need no masking; the two halves
      // are written out so that barrier and tensor-memory addresses are constants of the loop.
      auto step = [&](int j, int h, bool may_mask) -> bool {
        if (!mbar_wait_warp(&bars->s_full[t][h], j & 1, ctl)) return false;
        tc_fence_after();
        uint32_t s[32];
        tmem_ld32(s_addr + h * 64 + c * 32, s);
        tmem_ld_wait();
        uint32_t packed[16];
        const int valid = may_mask ? seq_len - ((tile_begin + j) * 2 + h) * 64 - c * 32 : 32;
        if (may_mask && valid < 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i >= valid) s[i] = 0xff800000u;  // -inf: probability 0 (the polynomial cannot take it)
          exp2_chunk<0>(s, packed);
        } else {
          exp2_chunk<kFaPolyPairs>(s, packed);
        }
        tmem_st16(s_addr + h * 64 + c * 32, packed);  // over the start of the columns just read
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->p_ready[t][h]);
        return true;
      };
      for (int j = 0; j + 1 < n_kv && ok; ++j) ok = step(j, 0, false) && step(j, 1, false);
      if (ok && n_kv > 0) ok = step(n_kv - 1, 0, true) && step(n_kv - 1, 1, true);
    } else {
    // ---- online form; the same two written-out halves per key tile as above
    auto step = [&](int j, int h, bool may_mask) -> bool {
      if (!mbar_wait_warp(&bars->s_full[t][h], j & 1, ctl)) return false;
      tc_fence_after();
      uint32_t s[32];
      tmem_ld32(s_addr + h * 64 + c * 32, s);
      tmem_ld_wait();
      if (may_mask) {
        const int valid = seq_len - ((tile_begin + j) * 2 + h) * 64 - c * 32;
        if (valid < 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i >= valid) s[i] = 0xff800000u;  // -inf
        }
      }
      float mx[4];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t* sc = &s[g * 8];
        mx[g] = fmax3(__uint_as_float(sc[0]), __uint_as_float(sc[1]), __uint_as_float(sc[2]));
        mx[g] = fmax3(mx[g], __uint_as_float(sc[3]), __uint_as_float(sc[4]));
        mx[g] = fmax3(mx[g], __uint_as_float(sc[5]), __uint_as_float(sc[6]));
        mx[g] = fmaxf(mx[g], __uint_as_float(sc[7]));
      }
      const float mx_own = fmaxf(fmax3(mx[0], mx[1], mx[2]), mx[3]);
      // swap with the thread that holds the other 32 scores of this row
      xchg->row_max[h][t][c][row_in_tile] = mx_own;
      pair_barrier(barrier_id);
      ++pair_syncs;
      const float mx_scaled = fmaxf(mx_own, xchg->row_max[h][t][c ^ 1][row_in_tile]);
      if ((j | h) == 0) {
        m_ref = mx_scaled;
      } else {
        const bool grow = mx_scaled > m_ref + kFaRescaleThreshold;
        if (__any_sync(0xffffffffu, grow ? 1 : 0)) {
          // O_t may still be the target of the previous step's P V.  The issuer follows that P V
          // with the Q K^T that refills the other half's scores, so their arrival tells that it
          // has retired; after the last key tile, where nothing follows, pv_done does.
          const int jp = h == 1 ? j : j - 1;  // key tile of step n-1 (its half is h^1)
          const bool waited = jp + 1 < n_kv
                                  ? mbar_wait_warp(&bars->s_full[t][h ^ 1], (uint32_t)(jp + 1) & 1u, ctl)
                                  : mbar_wait_warp(&bars->pv_done[t], 0, ctl);
          if (!waited) return false;
          tc_fence_after();
          const float m_new = grow ? mx_scaled : m_ref;
          const float alpha = fast_exp2(m_ref - m_new);
          m_ref = m_new;
          uint32_t acc[32];  // this thread's 32 of the row's 64 output channels
          tmem_ld32(o_addr, acc);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * alpha);
          tmem_st32(o_addr, acc);
          if (c == 1) {  // and the row sum, which is one more accumulator column
            uint32_t sum[16];
            tmem_ld16(l_addr, sum);
            tmem_ld_wait();
            sum[0] = __float_as_uint(__uint_as_float(sum[0]) * alpha);
            tmem_st16(l_addr, sum);
          }
        }
      }
      const float2 neg_m2 = make_float2(-m_ref, -m_ref);
      uint32_t packed[16];
      softmax_chunk<0>(s, make_float2(1.0f, 1.0f), neg_m2, packed);
      tmem_st16(s_addr + h * 64 + c * 32, packed);  // over the start of the columns just read
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_ready[t][h]);
      return true;
    };
    for (int j = 0; j + 1 < n_kv && ok; ++j) ok = step(j, 0, false) && step(j, 1, false);
    if (ok && n_kv > 0) ok = step(n_kv - 1, 0, true) && step(n_kv - 1, 1, true);
    }
    // a warp that gave up early still meets its partner at every barrier the partner may be in
    for (; pair_syncs < n_steps; ++pair_syncs) pair_barrier(barrier_id);
    if (ok && mbar_wait_warp(&bars->o_done[t], 0, ctl)) {
      tc_fence_after();
      uint32_t acc[32], sum[16];
      tmem_ld32(o_addr, acc);
      tmem_ld16(l_addr, sum);
      tmem_ld_wait();
      if (row_live) {
        float row_sum = __uint_as_float(sum[0]);
        // each of the row's two threads keeps its own copy of {reference, row sum} in the state
        float* ml_mine = ml_state + ((size_t)row * (dim / 64) + head) * 4 + 2 * c;
        if (!first_chunk) {
          // add what the earlier chunks left for this row, in fp32 with round-to-nearest: partial
          // output, row sum, and - online form - their reference (the fixed form's is the same in
          // every launch, bit for bit)
          const float m_old = ml_mine[0], l_old = ml_mine[1];
          float a_old = 1.0f, a_new = 1.0f;
          if (m_old != m_ref) {
            const float m_tot = fmaxf(m_old, m_ref);
            a_old = fast_exp2(m_old - m_tot);
            a_new = fast_exp2(m_ref - m_tot);
            m_ref = m_tot;
          }
          const uint4* src = reinterpret_cast<const uint4*>(o_state + (size_t)row * dim + head * 64 + c * 32);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 v = src[i];
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
              acc[4 * i + e] = __float_as_uint(fmaf(__uint_as_float(acc[4 * i + e]), a_new, __uint_as_float(w[e]) * a_old));
          }
          row_sum = fmaf(row_sum, a_new, l_old * a_old);
        }
        if (last_chunk) {
          const float inv = 1.0f / row_sum;
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
        } else {
          // leave the sum over the chunks so far for the next launch
          uint4* dst = reinterpret_cast<uint4*>(o_state + (size_t)row * dim + head * 64 + c * 32);
#pragma unroll
          for (int i = 0; i < 8; ++i) dst[i] = make_uint4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
          ml_mine[0] = m_ref;
          ml_mine[1] = row_sum;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ------------------------------------------------------------------------------------------------
// E4M3 variant (qkv_dtype = 1).  Same CTA shape, warp roles, barriers and tensor-memory map as the
// bf16 kernel above; what differs:
//   * Q, K and V arrive as E4M3 bytes with one scale per (tensor, head); both products run as
//     kind::f8f6f4 (K = 32 per instruction: two instructions per step and product instead of four);
//   * K tiles are 128 keys x 64 bytes (64-byte swizzle); V comes transposed, 64 channel rows x 128
//     key bytes per tile, K-major like K, followed in shared memory by 16 rows of which the first
//     holds 1.0 in every byte: as rows 64..79 of the B operand they make accumulator column 64 the sum
//     of the very E4M3 probabilities that multiply V;
//   * the probabilities are rounded to E4M3, whose values reach from 2^-9 to 448 only, so they must
//     sit at the top of that range: every row runs the online form with the reference kept 8 below
//     the running row maximum (the largest probability of a row is 2^8 when the reference is set
//     and may grow to 2^8.75 before the row is rescaled), which leaves 17 binades below the row
//     maximum before a probability is rounded to zero;
//   * scores are multiplied by scale_q scale_k (K arrives with the softmax scale folded in, which its
//     per-head scale absorbs), the output by scale_v, in fp32.
constexpr int kFa8KTileBytes = 128 * 64;           // 128 keys x 64 channel bytes
constexpr int kFa8VTileBytes = 64 * 128;           // 64 channels x 128 key bytes
constexpr int kFa8VStageBytes = kFa8VTileBytes + 16 * 128;  // + the ones rows
constexpr uint32_t kFa8ColQ = 416;                 // Q_0, Q_1: 16 columns of 4 bytes each
constexpr float kFa8Headroom = 8.0f;               // the row maximum maps to 2^8 of E4M3's 448
constexpr int kFa8SmemBytes = kFaStages * (kFa8KTileBytes + kFa8VStageBytes) + (int)sizeof(FaExchange) + 512 + 1024;

template <bool kFirst, bool kLast>
__global__ void __launch_bounds__(kFaThreads, 1)
flash_attention_fp8_kernel(const __grid_constant__ CUtensorMap tmap_k8, const __grid_constant__ CUtensorMap tmap_v8t,
                           const uint8_t* __restrict__ q8, const float* __restrict__ amax, __nv_bfloat16* __restrict__ o,
                           float* __restrict__ o_state, float* __restrict__ ml_state, int seq_len, int dim, int tile_begin,
                           int tile_end, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_k = smem;
  uint8_t* smem_v = smem_k + kFaStages * kFa8KTileBytes;
  FaExchange* xchg = reinterpret_cast<FaExchange*>(smem_v + kFaStages * kFa8VStageBytes);
  FaBarriers* bars = reinterpret_cast<FaBarriers*>(xchg + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * 256;
  const int head = blockIdx.y;
  const int n_kv = tile_end - tile_begin;
  const int n_steps = 2 * n_kv;
  constexpr bool first_chunk = kFirst;
  constexpr bool last_chunk = kLast;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_ready, kFaSoftmaxWarps);
    for (int s = 0; s < kFaStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 2);
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 2);
    }
    for (int t = 0; t < 2; ++t) {
      for (int h = 0; h < 2; ++h) {
        mbar_init(&bars->s_full[t][h], 1);
        mbar_init(&bars->p_ready[t][h], 8);
      }
      mbar_init(&bars->pv_done[t], 1);
      mbar_init(&bars->o_done[t], 1);
    }
    mbar_init(&bars->teardown[0], 1);
    mbar_init(&bars->teardown[1], 1);
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_k8);
    tma_prefetch_desc(&tmap_v8t);
  }
  // the ones rows behind every V stage: 128 bytes of E4M3 1.0 (0x38), then 15 rows of zeros (a row
  // of equal bytes looks the same under the swizzle)
  for (int i = threadIdx.x; i < kFaStages * 16 * 128 / 16; i += kFaThreads) {
    const int stage = i / 128, piece = i % 128;  // 128 16-byte pieces per stage
    const uint32_t fill = piece < 8 ? 0x38383838u : 0u;
    reinterpret_cast<uint4*>(smem_v + stage * kFa8VStageBytes + kFa8VTileBytes)[piece] = make_uint4(fill, fill, fill, fill);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 16) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const WaitCtl ctl{&bars->abort_flag, status};

  if (warp == 17) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      uint32_t k_issued = 0, v_issued = 0;
      for (int j = 0; j < n_kv; ++j) {
        const int stage = j % kFaStages;
        const uint32_t phase = (uint32_t)(j / kFaStages) & 1u;
        if (!mbar_wait(&bars->k_empty[stage], phase ^ 1u, ctl)) break;
        mbar_expect_tx(&bars->k_full[stage], kFa8KTileBytes);
        tma_load_2d(smem_k + stage * kFa8KTileBytes, &tmap_k8, &bars->k_full[stage], head * 64, (tile_begin + j) * 128);
        ++k_issued;
        if (!mbar_wait(&bars->v_empty[stage], phase ^ 1u, ctl)) break;
        mbar_expect_tx(&bars->v_full[stage], kFa8VTileBytes);
        tma_load_2d(smem_v + stage * kFa8VStageBytes, &tmap_v8t, &bars->v_full[stage], (tile_begin + j) * 128, head * 64);
        ++v_issued;
      }
      drain_ring(bars->k_full, k_issued, status);
      drain_ring(bars->v_full, v_issued, status);
    }
  } else if (warp == 16 || warp == 18) {
    // ------------------------------------------------------------------ MMA issuer of tile t
    if (elect_one()) {
      const int t = warp == 16 ? 0 : 1;
      constexpr uint32_t idesc_qk = umma_idesc_e4m3(128, 64);
      constexpr uint32_t idesc_pv = umma_idesc_e4m3(128, kFaOCols);
      const uint32_t s_col = tmem_base + kFaColS + t * 128;
      const uint32_t o_col = tmem_base + kFaColO + t * kFaOCols;
      const uint32_t q_col = tmem_base + kFa8ColQ + t * 16;
      // S_h = Q x K[64h .. 64h+63]^T: 64 rows of 64 bytes = 4096 bytes per half, 32 channels per instruction
      auto issue_qk = [&](int h, int stage) {
        const uint64_t b_desc = smem_desc_sw64(smem_u32(smem_k + stage * kFa8KTileBytes + h * 4096), 16, 512);
#pragma unroll
        for (int k = 0; k < 2; ++k) umma_ts_f8(s_col + h * 64, q_col + k * 8, b_desc + 2 * k, idesc_qk, k != 0 ? 1u : 0u);
        umma_commit(&bars->s_full[t][h]);
      };
      bool ok = mbar_wait(&bars->q_ready, 0, ctl);
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
        if (!last && !mbar_wait(&bars->k_full[next_stage], next_phase, ctl)) { ok = false; break; }
        for (int h = 0; h < 2; ++h) {
          if (!mbar_wait(&bars->p_ready[t][h], j & 1, ctl)) { ok = false; break; }
          tc_fence_after();
          // 64 keys of the transposed V tile: bytes [64h, 64h + 64) of every channel row, 32 keys per
          // instruction; 8 tensor-memory columns of P each (keys 0-31 in columns [0,8) of the half,
          // keys 32-63 in [32,40)); rows 64..79 of B are the ones rows behind the tile
          const uint64_t v_desc = smem_desc_sw128(smem_u32(smem_v + stage * kFa8VStageBytes + h * 64), 16, 1024);
#pragma unroll
          for (int k = 0; k < 2; ++k)
            umma_ts_f8(o_col, s_col + h * 64 + k * 32, v_desc + 2 * k, idesc_pv, (j | h | k) != 0 ? 1u : 0u);
          if (last) {
            umma_commit(&bars->pv_done[t]);
            if (h == 1) umma_commit(&bars->o_done[t]);
          } else {
            issue_qk(h, next_stage);
          }
        }
        if (!ok) break;
        umma_commit(&bars->v_empty[stage]);
        if (!last) umma_commit(&bars->k_empty[next_stage]);
        stage = next_stage;
        phase = next_phase;
      }
      if (!ok) {
        umma_commit(&bars->teardown[t]);
        const long long t0 = clock64();
        while (!mbar_try_wait(&bars->teardown[t], 0)) {
          if (clock64() - t0 > kTimeoutCycles) break;
        }
      }
    }
  } else if (warp < kFaSoftmaxWarps) {
    // ------------------------------------------------------------------ softmax warps
    const int t = warp >> 3;
    const int c = (warp >> 2) & 1;
    const uint32_t quarter = warp & 3u;
    const int barrier_id = 1 + t * 4 + (int)quarter;
    const int row_in_tile = (int)quarter * 32 + lane;
    const uint32_t lane_base = (quarter * 32u) << 16;
    const int row_local = q0 + t * 128 + row_in_tile;
    const bool row_live = row_local < seq_len;
    const int row = row_local;
    const uint32_t s_addr = tmem_base + lane_base + kFaColS + t * 128;
    const uint32_t o_addr = tmem_base + lane_base + kFaColO + t * kFaOCols + c * 32;
    const uint32_t l_addr = tmem_base + lane_base + kFaColO + t * kFaOCols + 64;
    {
      // this thread's 32 channels (32 bytes) of its query row
      uint32_t qreg[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) qreg[i] = 0u;
      if (row_live) {
        const uint4* src = reinterpret_cast<const uint4*>(q8 + (size_t)row * dim + head * 64 + c * 32);
        const uint4 a = __ldg(src), b = __ldg(src + 1);
        qreg[0] = a.x; qreg[1] = a.y; qreg[2] = a.z; qreg[3] = a.w;
        qreg[4] = b.x; qreg[5] = b.y; qreg[6] = b.z; qreg[7] = b.w;
      }
      tmem_st8(tmem_base + lane_base + kFa8ColQ + t * 16 + c * 8, qreg);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->q_ready);
    }
    // dequantisation: score = (q8 . k8) scale_q scale_k / sqrt(64), output = (P v8) scale_v / sum P
    const float a_q = amax[head], a_k = amax[16 + head], a_v = amax[32 + head];
    const float scale_q = (a_q > 0.0f ? a_q : 1.0f) / 448.0f, scale_k = (a_k > 0.0f ? a_k : 1.0f) / 448.0f;
    const float scale_v = (a_v > 0.0f ? a_v : 1.0f) / 448.0f;
    const float scale_log2e = scale_q * scale_k;  // K was quantised with the softmax scale folded in
    const float2 scale2 = make_float2(scale_log2e, scale_log2e);
    float m_ref = -INFINITY;
    bool ok = true;
    int pair_syncs = 0;
    // the two halves of a key tile are written out (barrier and tensor-memory addresses constant);
    // only the last tile of a launch can reach past the sequence
    auto step = [&](int j, int h, bool may_mask) -> bool {
      if (!mbar_wait_warp(&bars->s_full[t][h], j & 1, ctl)) return false;
      tc_fence_after();
      uint32_t s[32];
      tmem_ld32(s_addr + h * 64 + c * 32, s);
      tmem_ld_wait();
      if (may_mask) {
        const int valid = seq_len - ((tile_begin + j) * 2 + h) * 64 - c * 32;
        if (valid < 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i >= valid) s[i] = 0xff800000u;  // -inf
        }
      }
      float mx[4];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t* sc = &s[g * 8];
        mx[g] = fmax3(__uint_as_float(sc[0]), __uint_as_float(sc[1]), __uint_as_float(sc[2]));
        mx[g] = fmax3(mx[g], __uint_as_float(sc[3]), __uint_as_float(sc[4]));
        mx[g] = fmax3(mx[g], __uint_as_float(sc[5]), __uint_as_float(sc[6]));
        mx[g] = fmaxf(mx[g], __uint_as_float(sc[7]));
      }
      const float mx_own = fmaxf(fmax3(mx[0], mx[1], mx[2]), mx[3]);
      xchg->row_max[h][t][c][row_in_tile] = mx_own;
      pair_barrier(barrier_id);
      ++pair_syncs;
      const float mx_scaled = fmaxf(mx_own, xchg->row_max[h][t][c ^ 1][row_in_tile]) * scale_log2e;
      if ((j | h) == 0) {
        m_ref = mx_scaled - kFa8Headroom;
      } else {
        const bool grow = mx_scaled > m_ref + kFa8Headroom + 0.75f;
        if (__any_sync(0xffffffffu, grow ? 1 : 0)) {
          const int jp = h == 1 ? j : j - 1;
          const bool waited = jp + 1 < n_kv
                                  ? mbar_wait_warp(&bars->s_full[t][h ^ 1], (uint32_t)(jp + 1) & 1u, ctl)
                                  : mbar_wait_warp(&bars->pv_done[t], 0, ctl);
          if (!waited) return false;
          tc_fence_after();
          const float m_new = grow ? mx_scaled - kFa8Headroom : m_ref;
          const float alpha = fast_exp2(m_ref - m_new);
          m_ref = m_new;
          uint32_t acc[32];
          tmem_ld32(o_addr, acc);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * alpha);
          tmem_st32(o_addr, acc);
          if (c == 1) {
            uint32_t sum[16];
            tmem_ld16(l_addr, sum);
            tmem_ld_wait();
            sum[0] = __float_as_uint(__uint_as_float(sum[0]) * alpha);
            tmem_st16(l_addr, sum);
          }
        }
      }
      const float2 neg_m2 = make_float2(-m_ref, -m_ref);
      uint32_t packed[8];  // 32 probabilities as E4M3 bytes
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(s[4 * i]), __uint_as_float(s[4 * i + 1])), scale2, neg_m2);
        const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(s[4 * i + 2]), __uint_as_float(s[4 * i + 3])), scale2, neg_m2);
        packed[i] = pack_e4m3x4(fast_exp2(x0.x), fast_exp2(x0.y), fast_exp2(x1.x), fast_exp2(x1.y));
      }
      tmem_st8(s_addr + h * 64 + c * 32, packed);  // over the start of the columns just read
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_ready[t][h]);
      return true;
    };
    for (int j = 0; j + 1 < n_kv && ok; ++j) ok = step(j, 0, false) && step(j, 1, false);
    if (ok && n_kv > 0) ok = step(n_kv - 1, 0, true) && step(n_kv - 1, 1, true);
    for (; pair_syncs < n_steps; ++pair_syncs) pair_barrier(barrier_id);
    if (ok && mbar_wait_warp(&bars->o_done[t], 0, ctl)) {
      tc_fence_after();
      uint32_t acc[32], sum[16];
      tmem_ld32(o_addr, acc);
      tmem_ld16(l_addr, sum);
      tmem_ld_wait();
      if (row_live) {
        float row_sum = __uint_as_float(sum[0]);
        float* ml_mine = ml_state + ((size_t)row * (dim / 64) + head) * 4 + 2 * c;
        if (!first_chunk) {
          const float m_old = ml_mine[0], l_old = ml_mine[1];
          float a_old = 1.0f, a_new = 1.0f;
          if (m_old != m_ref) {
            const float m_tot = fmaxf(m_old, m_ref);
            a_old = fast_exp2(m_old - m_tot);
            a_new = fast_exp2(m_ref - m_tot);
            m_ref = m_tot;
          }
          const uint4* src = reinterpret_cast<const uint4*>(o_state + (size_t)row * dim + head * 64 + c * 32);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 v = src[i];
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
              acc[4 * i + e] = __float_as_uint(fmaf(__uint_as_float(acc[4 * i + e]), a_new, __uint_as_float(w[e]) * a_old));
          }
          row_sum = fmaf(row_sum, a_new, l_old * a_old);
        }
        if (last_chunk) {
          const float inv = scale_v / row_sum;
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
        } else {
          uint4* dst = reinterpret_cast<uint4*>(o_state + (size_t)row * dim + head * 64 + c * 32);
#pragma unroll
          for (int i = 0; i < 8; ++i) dst[i] = make_uint4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
          ml_mine[0] = m_ref;
          ml_mine[1] = row_sum;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

cudaError_t launch_flash_attention_fp8(litevggt_ctx* ctx, long long m, __nv_bfloat16* o, cudaStream_t s, int* launches) {
  if (m == 0) return cudaSuccess;
  const int dim = ctx->sz.dim;
  Workspace& ws = ctx->ws;
  if (dim != 1024 || ws.q8 == nullptr) return cudaErrorInvalidValue;
  const long long m_pad = round_up(m, 128);
  CUtensorMap tmap_k, tmap_v;
  if (!make_tmap_u8_2d(ctx->encode_tiled, &tmap_k, ws.k8, (uint64_t)dim, (uint64_t)m, (uint64_t)dim, 64, 128) ||
      !make_tmap_u8_2d(ctx->encode_tiled, &tmap_v, ws.v8t, (uint64_t)m_pad, (uint64_t)dim, (uint64_t)m_pad, 128, 64))
    return cudaErrorInvalidValue;
  using Kernel = void (*)(const CUtensorMap, const CUtensorMap, const uint8_t*, const float*, __nv_bfloat16*, float*,
                          float*, int, int, int, int, uint32_t*);
  const Kernel kernels[2][2] = {{flash_attention_fp8_kernel<false, false>, flash_attention_fp8_kernel<false, true>},
                                {flash_attention_fp8_kernel<true, false>, flash_attention_fp8_kernel<true, true>}};
  static std::atomic<unsigned long long> smem_set[2][2];
  for (int a = 0; a < 2; ++a)
    for (int b = 0; b < 2; ++b) {
      cudaError_t e = set_max_dynamic_smem_once(reinterpret_cast<const void*>(kernels[a][b]), kFa8SmemBytes, smem_set[a][b]);
      if (e != cudaSuccess) return e;
    }
  const dim3 grid((unsigned)((m + 255) / 256), (unsigned)ctx->sz.heads, 1);
  const int n_tiles = (int)((m + 127) / 128);
  const int n_chunks = (n_tiles + kFaChunkTiles - 1) / kFaChunkTiles;
  const int per_chunk = (n_tiles + n_chunks - 1) / n_chunks;
  if (n_chunks > 1 && (ws.attn_o_state == nullptr || ws.attn_ml_state == nullptr)) return cudaErrorInvalidValue;
  for (int begin = 0; begin < n_tiles; begin += per_chunk) {
    const int end = begin + per_chunk < n_tiles ? begin + per_chunk : n_tiles;
    kernels[begin == 0][end == n_tiles]<<<grid, kFaThreads, kFa8SmemBytes, s>>>(
        tmap_k, tmap_v, ws.q8, ws.qkv_amax, o, ws.attn_o_state, ws.attn_ml_state, (int)m, dim, begin, end, ws.status);
    ++*launches;
  }
  return cudaGetLastError();
}

// max_k |k|^2 per (sequence, head), for the Cauchy-Schwarz bound on a row's scores.  Warp per key
// row: the 128 16-byte pieces of a K row go to the lanes in four passes, eight neighbouring lanes
// share a head.  Non-negative floats order like their bit patterns, so the maximum is an integer
// atomicMax on a zeroed array.
constexpr int kKnormWarps = 8;
__global__ void __launch_bounds__(kKnormWarps * 32)
key_norm_max_kernel(const __nv_bfloat16* __restrict__ qkv, int seq_len, int dim, float* __restrict__ k_norm2_max) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int seq = blockIdx.y, heads = dim / 64;
  float best[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int r = blockIdx.x * kKnormWarps + warp; r < seq_len; r += gridDim.x * kKnormWarps) {
    const uint4* src = reinterpret_cast<const uint4*>(qkv + ((size_t)seq * seq_len + r) * 3 * dim + dim);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint4 v = __ldg(src + lane + 32 * j);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      float sum = 0.0f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        sum = fmaf(bf16_lo(w[e]), bf16_lo(w[e]), sum);
        sum = fmaf(bf16_hi(w[e]), bf16_hi(w[e]), sum);
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sum += __shfl_xor_sync(0xffffffffu, sum, 4);
      best[j] = fmaxf(best[j], sum);
    }
  }
  if ((lane & 7) == 0) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      atomicMax(reinterpret_cast<unsigned int*>(k_norm2_max) + seq * heads + (lane >> 3) + 4 * j,
                __float_as_uint(best[j]));
  }
}

cudaError_t launch_flash_attention(litevggt_ctx* ctx, const __nv_bfloat16* qkv, long long seq_len, int n_seq,
                                   __nv_bfloat16* o, cudaStream_t s, int* launches) {
  if (seq_len == 0 || n_seq == 0) return cudaSuccess;
  const int dim = ctx->sz.dim;
  if (dim != 1024 || ctx->ws.attn_kmax == nullptr) return cudaErrorInvalidValue;
  {
    cudaError_t e = cudaMemsetAsync(ctx->ws.attn_kmax, 0, (size_t)n_seq * ctx->sz.heads * sizeof(float), s);
    if (e != cudaSuccess) return e;
    long long blocks = (seq_len + 63) / 64;
    if (blocks > 2048) blocks = 2048;
    key_norm_max_kernel<<<dim3((unsigned)blocks, (unsigned)n_seq), kKnormWarps * 32, 0, s>>>(qkv, (int)seq_len, dim,
                                                                                            ctx->ws.attn_kmax);
    ++*launches;
  }
  const long long rows = seq_len * n_seq;
  CUtensorMap tmap;
  if (!make_tmap_bf16_2d(ctx->encode_tiled, &tmap, qkv, (uint64_t)3 * dim, (uint64_t)rows, (uint64_t)3 * dim, 64, 128))
    return cudaErrorInvalidValue;
  using Kernel = void (*)(const CUtensorMap, const __nv_bfloat16*, __nv_bfloat16*, float*, float*, const float*, int,
                          int, int, int, uint32_t*);
  const Kernel kernels[2][2] = {{flash_attention_kernel<false, false>, flash_attention_kernel<false, true>},
                                {flash_attention_kernel<true, false>, flash_attention_kernel<true, true>}};
  static std::atomic<unsigned long long> smem_set[2][2];
  for (int a = 0; a < 2; ++a)
    for (int b = 0; b < 2; ++b) {
      cudaError_t e = set_max_dynamic_smem_once(reinterpret_cast<const void*>(kernels[a][b]), kFaSmemBytes, smem_set[a][b]);
      if (e != cudaSuccess) return e;
    }
  const dim3 grid((unsigned)((seq_len + 255) / 256), (unsigned)ctx->sz.heads, (unsigned)n_seq);
  // balanced chunks of at most kFaChunkTiles key tiles; more than one needs the state buffers (which
  // are sized for the single long sequence of the global layer)
  const int n_tiles = (int)((seq_len + 127) / 128);
  const int n_chunks = (n_tiles + kFaChunkTiles - 1) / kFaChunkTiles;
  const int per_chunk = (n_tiles + n_chunks - 1) / n_chunks;
  if (n_chunks > 1 && (n_seq != 1 || ctx->ws.attn_o_state == nullptr || ctx->ws.attn_ml_state == nullptr))
    return cudaErrorInvalidValue;
  for (int begin = 0; begin < n_tiles; begin += per_chunk) {
    const int end = begin + per_chunk < n_tiles ? begin + per_chunk : n_tiles;
    kernels[begin == 0][end == n_tiles]<<<grid, kFaThreads, kFaSmemBytes, s>>>(
        tmap, qkv, o, ctx->ws.attn_o_state, ctx->ws.attn_ml_state, ctx->ws.attn_kmax, (int)seq_len, dim, begin, end,
        ctx->ws.status);
    ++*launches;
  }
  return cudaGetLastError();
}

// Rows of fp32 partial output and of {reference, row sum} x 2 per head (one copy per thread of a row)
// that the chunked sweep sums up between launches; zero when m fits one chunk.
size_t attention_state_bytes(long long m, int dim, int heads, size_t* ml_offset) {
  const long long n_tiles = (m + 127) / 128;
  if (n_tiles <= kFaChunkTiles) {
    if (ml_offset) *ml_offset = 0;
    return 0;
  }
  const size_t o_bytes = (size_t)round_up(m * dim * 4, 256);
  if (ml_offset) *ml_offset = o_bytes;
  return o_bytes + (size_t)round_up(m * heads * 16, 256);
}

}  // namespace lv
