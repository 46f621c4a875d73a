// Per-head top-B^l (Eq. 3; Algorithm 1's "topk(B^l)") under the total order
// (score descending, position ascending).  One CTA per (sample, KV head).
// Scores are non-negative floats, so their bit patterns order like unsigned integers.
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kSelThreads = 1024;

// Exclusive block scan of two counters at once; returns this thread's prefixes and the totals.
__device__ __forceinline__ void block_scan2(int a, int b, int& a_excl, int& b_excl, int& a_tot, int& b_tot,
                                            int* sm_a /*[33]*/, int* sm_b /*[33]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int ta = __shfl_up_sync(0xFFFFFFFFu, ia, o), tb = __shfl_up_sync(0xFFFFFFFFu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  __syncthreads();
  if (lane == 31) { sm_a[warp] = ia; sm_b[warp] = ib; }
  __syncthreads();
  if (warp == 0) {
    int wa = lane < nw ? sm_a[lane] : 0, wb = lane < nw ? sm_b[lane] : 0;
    int sa = wa, sb = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int ta = __shfl_up_sync(0xFFFFFFFFu, sa, o), tb = __shfl_up_sync(0xFFFFFFFFu, sb, o);
      if (lane >= o) { sa += ta; sb += tb; }
    }
    sm_a[lane] = sa - wa; sm_b[lane] = sb - wb;
    if (lane == 31) { sm_a[32] = sa; sm_b[32] = sb; }
  }
  __syncthreads();
  a_excl = sm_a[warp] + ia - a; b_excl = sm_b[warp] + ib - b;
  a_tot = sm_a[32]; b_tot = sm_b[32];
}

// scores: [Bt*Hkv][P] of one layer.  idx, rank: [Bt*Hkv][keep].  sort_n: power of two >= keep.
// Also records count[b][layer] = keep.
__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(const float* __restrict__ scores, int* __restrict__ idx, int* __restrict__ rank,
                   int* __restrict__ idx_out, int* __restrict__ rank_out, int P, int keep, int sort_n,
                   int* __restrict__ count, int Hkv, int L, int layer) {
  extern __shared__ __align__(16) unsigned long long skeys[];
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_bin, s_rem;
  __shared__ int sm_a[33], sm_b[33];
  const int tid = threadIdx.x;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + (size_t)blockIdx.x * P;
  if (tid == 0 && blockIdx.x % Hkv == 0) count[(blockIdx.x / Hkv) * L + layer] = keep;

  // Radix select, most significant byte first: T = bit pattern of the keep-th largest score.
  uint32_t prefix = 0, mask = 0;
  unsigned int remaining = (unsigned int)keep;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < P; i += kSelThreads) {
      const uint32_t u = v[i];
      if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned int cum = 0;
      int bin = 255;
      for (; bin > 0; --bin) {
        const unsigned int c = hist[bin];
        if (cum + c >= remaining) break;
        cum += c;
      }
      s_bin = (unsigned int)bin;
      s_rem = remaining - cum;
    }
    __syncthreads();
    prefix |= s_bin << shift;
    mask |= 255u << shift;
    remaining = s_rem;
    __syncthreads();
  }
  const uint32_t T = prefix;
  const int need_eq = (int)remaining;     // how many of the entries equal to T are kept (lowest positions)

  // Ordered compaction: each thread owns a contiguous run of positions.
  const int chunk = (P + kSelThreads - 1) / kSelThreads;
  const int p0 = min(P, tid * chunk), p1 = min(P, p0 + chunk);
  int gt = 0, eq = 0;
  for (int i = p0; i < p1; ++i) { const uint32_t u = v[i]; gt += (u > T); eq += (u == T); }
  int gt_before, eq_before, gt_tot, eq_tot;
  block_scan2(gt, eq, gt_before, eq_before, gt_tot, eq_tot, sm_a, sm_b);
  for (int i = tid + keep; i < sort_n; i += kSelThreads) skeys[i] = ~0ull;
  int* my_idx = idx + (size_t)blockIdx.x * keep;
  int* my_rank = rank + (size_t)blockIdx.x * keep;
  {
    int g = gt_before, e = eq_before;
    for (int i = p0; i < p1; ++i) {
      const uint32_t u = v[i];
      const bool is_eq = (u == T);
      if (u > T || (is_eq && e < need_eq)) {
        const int out = g + min(e, need_eq);
        my_idx[out] = i;
        if (idx_out) idx_out[(size_t)blockIdx.x * keep + out] = i;
        skeys[out] = ((unsigned long long)(~u) << 32) | (unsigned int)out;
      }
      g += (u > T); e += is_eq;
    }
  }
  __syncthreads();

  // Rank = place in (score descending, position ascending): bitonic sort of (~bits, list slot).
  for (int size = 2; size <= sort_n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = tid; t < (sort_n >> 1); t += kSelThreads) {
        const int lo = ((t / stride) * stride * 2) + (t % stride);
        const int hi = lo + stride;
        const bool up = ((lo & size) == 0);
        const unsigned long long a = skeys[lo], b = skeys[hi];
        if ((a > b) == up) { skeys[lo] = b; skeys[hi] = a; }
      }
      __syncthreads();
    }
  }
  for (int i = tid; i < keep; i += kSelThreads) {
    const int slot = (int)(skeys[i] & 0xFFFFFFFFull);
    my_rank[slot] = i;
    if (rank_out) rank_out[(size_t)blockIdx.x * keep + slot] = i;
  }
}

}  // namespace dkv
