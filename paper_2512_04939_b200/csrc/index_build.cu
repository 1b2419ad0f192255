// Selection of the src tokens to merge and construction of the cached index arrays.
//
// Inputs: per src token (ascending token order) its best anchor and cosine.  The R most
// similar src tokens are merged (ties towards the lower token index); every other token
// keeps its own row, rows follow ascending token order.  Outputs: dst_of[N], size[M],
// kept_idx[M] and a CSR (seg_off[M+1], seg_src[R]) listing, per merged row, the absorbed
// src tokens in ascending token order - the order the merge kernel sums them in.
//
// Everything here is integer work on ~1 M elements: two bitonic sorts of unique 64-bit
// keys (so the result does not depend on scheduling), two exclusive scans and a few
// element-wise kernels.  No host synchronisation: all counts follow from the config.
#include "common.cuh"
#include "runtime.h"

namespace lv {

constexpr int kSortChunk = 2048;   // elements sorted per CTA in shared memory
constexpr int kSortThreads = 1024;
constexpr int kScanThreads = 1024;
constexpr int kScanItems = 4;
constexpr int kScanChunk = kScanThreads * kScanItems;

size_t sort_capacity(long long n) {
  size_t cap = kSortChunk;
  while ((long long)cap < n) cap <<= 1;
  return cap;
}

// ------------------------------------------------------------------------------ bitonic sort
__device__ __forceinline__ void cmp_swap(unsigned long long& a, unsigned long long& b, bool ascending) {
  if ((a > b) == ascending) {
    const unsigned long long t = a;
    a = b;
    b = t;
  }
}

// Runs the compare-exchange steps (k, j) for k in [k_first, k_last], j from min(k/2, 1024)
// down to 1, on one 2048-element chunk held in shared memory.
__global__ void __launch_bounds__(kSortThreads)
bitonic_local_kernel(unsigned long long* __restrict__ keys, unsigned k_first, unsigned k_last) {
  __shared__ unsigned long long s[kSortChunk];
  const unsigned base = blockIdx.x * kSortChunk;
  s[threadIdx.x] = keys[base + threadIdx.x];
  s[threadIdx.x + kSortThreads] = keys[base + threadIdx.x + kSortThreads];
  __syncthreads();
  for (unsigned k = k_first; k <= k_last; k <<= 1) {
    unsigned j = k >> 1;
    if (j > kSortChunk / 2) j = kSortChunk / 2;
    for (; j > 0; j >>= 1) {
      const unsigned t = threadIdx.x;
      const unsigned lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));  // index with bit j clear
      const unsigned hi = lo | j;
      const bool ascending = ((base + lo) & k) == 0;
      cmp_swap(s[lo], s[hi], ascending);
      __syncthreads();
    }
    if (k == 0x80000000u) break;
  }
  keys[base + threadIdx.x] = s[threadIdx.x];
  keys[base + threadIdx.x + kSortThreads] = s[threadIdx.x + kSortThreads];
}

__global__ void bitonic_global_kernel(unsigned long long* __restrict__ keys, unsigned n_half, unsigned k, unsigned j) {
  const unsigned t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_half) return;
  const unsigned lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
  const unsigned hi = lo | j;
  unsigned long long a = keys[lo], b = keys[hi];
  const bool ascending = (lo & k) == 0;
  if ((a > b) == ascending) {
    keys[lo] = b;
    keys[hi] = a;
  }
}

static cudaError_t bitonic_sort(unsigned long long* keys, size_t cap, cudaStream_t s, int* launches) {
  const unsigned n = (unsigned)cap;
  const unsigned chunks = n / kSortChunk;
  bitonic_local_kernel<<<chunks, kSortThreads, 0, s>>>(keys, 2, kSortChunk);
  ++*launches;
  for (unsigned k = kSortChunk * 2; k <= n && k != 0; k <<= 1) {
    for (unsigned j = k >> 1; j >= kSortChunk; j >>= 1) {
      bitonic_global_kernel<<<(n / 2 + 255) / 256, 256, 0, s>>>(keys, n / 2, k, j);
      ++*launches;
    }
    bitonic_local_kernel<<<chunks, kSortThreads, 0, s>>>(keys, k, k);
    ++*launches;
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------ exclusive scan
__global__ void __launch_bounds__(kScanThreads)
scan_block_kernel(const int* __restrict__ in, int* __restrict__ out, int* __restrict__ block_sums, long long n) {
  __shared__ int warp_tot[kScanThreads / 32];
  const long long base = (long long)blockIdx.x * kScanChunk + (long long)threadIdx.x * kScanItems;
  int v[kScanItems];
  int local = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    v[i] = (base + i < n) ? in[base + i] : 0;
    local += v[i];
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int offset = incl - local;
  int total = 0;
  for (int i = 0; i < kScanThreads / 32; ++i) {
    if (i < warp) offset += warp_tot[i];
    total += warp_tot[i];
  }
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    if (base + i < n) out[base + i] = offset;
    offset += v[i];
  }
  if (threadIdx.x == 0) block_sums[blockIdx.x] = total;
}

// exclusive scan of up to 1024 block sums in one CTA
__global__ void __launch_bounds__(kScanThreads) scan_sums_kernel(int* __restrict__ block_sums, int n_blocks) {
  __shared__ int warp_tot[kScanThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int v = (int)threadIdx.x < n_blocks ? block_sums[threadIdx.x] : 0;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int offset = incl - v;
  for (int i = 0; i < warp; ++i) offset += warp_tot[i];
  if ((int)threadIdx.x < n_blocks) block_sums[threadIdx.x] = offset;
}

__global__ void scan_add_kernel(int* __restrict__ out, const int* __restrict__ block_sums, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] += block_sums[i / kScanChunk];
}

static cudaError_t exclusive_scan(const int* in, int* out, int* block_sums, long long n, cudaStream_t s,
                                  int* launches) {
  const int blocks = (int)((n + kScanChunk - 1) / kScanChunk);
  scan_block_kernel<<<blocks, kScanThreads, 0, s>>>(in, out, block_sums, n);
  scan_sums_kernel<<<1, kScanThreads, 0, s>>>(block_sums, blocks);
  scan_add_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(out, block_sums, n);
  *launches += 3;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------ element-wise steps
__device__ __forceinline__ unsigned ordered_bits(float f) {  // monotone float -> unsigned
  const unsigned u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// key = (descending similarity, ascending position) ; padding sorts last
__global__ void make_sim_keys_kernel(const float* __restrict__ best_sim, unsigned long long* __restrict__ keys,
                                     long long n_src, long long cap) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= cap) return;
  keys[i] = i < n_src ? ((unsigned long long)(~ordered_bits(best_sim[i])) << 32) | (unsigned)i : ~0ull;
}

__global__ void fill_int_kernel(int* __restrict__ p, int v, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

__global__ void mark_removed_kernel(const unsigned long long* __restrict__ keys, const int* __restrict__ src_list,
                                    int* __restrict__ kept_flag, long long n_remove) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_remove) kept_flag[src_list[(unsigned)keys[i]]] = 0;
}

__global__ void rows_of_kept_kernel(const int* __restrict__ kept_flag, const int* __restrict__ row_of,
                                    int* __restrict__ dst_of, int* __restrict__ kept_idx, int* __restrict__ size,
                                    long long n_tokens, long long n_merged, uint32_t* status) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_tokens || !kept_flag[i]) return;
  const int row = row_of[i];
  if (row < 0 || row >= n_merged) {
    atomicOr(status, kStatusBounds);
    return;
  }
  dst_of[i] = row;
  kept_idx[row] = (int)i;
  size[row] = 1;
}

// merged src tokens: dst_of, anchor sizes, and the (row, token) keys of the CSR sort
__global__ void assign_removed_kernel(unsigned long long* __restrict__ keys, const int* __restrict__ src_list,
                                      const int* __restrict__ best_dst, const int* __restrict__ row_of,
                                      const int* __restrict__ kept_flag, int* __restrict__ dst_of,
                                      int* __restrict__ size, long long n_remove, long long cap, long long n_tokens,
                                      uint32_t* status) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= cap) return;
  unsigned long long out = ~0ull;
  if (i < n_remove) {
    const unsigned pos = (unsigned)keys[i];
    const int token = src_list[pos];
    const int anchor = best_dst[pos];
    if (anchor < 0 || anchor >= n_tokens || !kept_flag[anchor]) {
      atomicOr(status, kStatusBounds);
    } else {
      const int row = row_of[anchor];
      dst_of[token] = row;
      atomicAdd(&size[row], 1);
      out = ((unsigned long long)(unsigned)row << 32) | (unsigned)token;
    }
  }
  keys[i] = out;
}

__global__ void csr_counts_kernel(const int* __restrict__ size, int* __restrict__ cnt, long long n_merged) {
  const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (j <= n_merged) cnt[j] = j < n_merged ? size[j] - 1 : 0;
}

__global__ void csr_fill_kernel(const unsigned long long* __restrict__ keys, int* __restrict__ seg_src,
                                long long n_remove) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_remove) seg_src[i] = (int)(unsigned)keys[i];
}

static inline unsigned blocks_for(long long n, int threads = 256) { return (unsigned)((n + threads - 1) / threads); }

cudaError_t launch_index_build(litevggt_ctx* ctx, litevggt_plan* plan, cudaStream_t s, int* launches) {
  const Sizes& z = ctx->sz;
  Workspace& ws = ctx->ws;
  const long long n = z.n_tokens, m = z.n_merged, r = z.n_remove;
  const long long cap = (long long)sort_capacity(z.n_src);
  cudaError_t e;
  int* kept_flag = ws.scan_tmp;

  fill_int_kernel<<<blocks_for(n), 256, 0, s>>>(kept_flag, 1, n);
  ++*launches;
  if (r > 0) {
    make_sim_keys_kernel<<<blocks_for(cap), 256, 0, s>>>(plan->best_sim, ws.sort_keys, z.n_src, cap);
    ++*launches;
    if ((e = bitonic_sort(ws.sort_keys, (size_t)cap, s, launches)) != cudaSuccess) return e;
    mark_removed_kernel<<<blocks_for(r), 256, 0, s>>>(ws.sort_keys, ws.src_list, kept_flag, r);
    ++*launches;
  }
  if ((e = exclusive_scan(kept_flag, ws.row_of, ws.scan_blocks, n, s, launches)) != cudaSuccess) return e;
  rows_of_kept_kernel<<<blocks_for(n), 256, 0, s>>>(kept_flag, ws.row_of, plan->dst_of, plan->kept_idx, plan->size, n,
                                                    m, ws.status);
  ++*launches;
  if (r > 0) {
    assign_removed_kernel<<<blocks_for(cap), 256, 0, s>>>(ws.sort_keys, ws.src_list, plan->best_dst, ws.row_of,
                                                          kept_flag, plan->dst_of, plan->size, r, cap, n, ws.status);
    ++*launches;
    if ((e = bitonic_sort(ws.sort_keys, (size_t)cap, s, launches)) != cudaSuccess) return e;
    csr_fill_kernel<<<blocks_for(r), 256, 0, s>>>(ws.sort_keys, plan->seg_src, r);
    ++*launches;
  }
  // kept_flag is dead from here on: reuse it for the per-row counts
  csr_counts_kernel<<<blocks_for(m + 1), 256, 0, s>>>(plan->size, ws.scan_tmp, m);
  ++*launches;
  if ((e = exclusive_scan(ws.scan_tmp, plan->seg_off, ws.scan_blocks, m + 1, s, launches)) != cudaSuccess) return e;
  return cudaGetLastError();
}

}  // namespace lv
