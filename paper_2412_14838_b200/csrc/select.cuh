// Per-head top-B^l (Eq. 3; Algorithm 1's "topk(B^l)") under the total order
// (score descending, position ascending), plus what the later global top-K (Eq. 4) needs from
// this layer.  One CTA per (sample, KV head).
//
// Scores are non-negative floats, so their bit patterns order like unsigned integers.  The
// threshold T (bit pattern of the B^l-th largest score) is found by a 3-pass radix select,
// most significant digit first (11 + 11 + 10 bits), with a shared-memory histogram per pass.
// The first pass's histogram (top 11 bits: sign, exponent, 2 mantissa bits) is also kept per head
// in global memory, together with a copy of the head's scores grouped by that digit, so that
// Update_Buffer_Length can locate the global K-th value from histograms and then look only at
// the one bucket that contains it, instead of re-reading every layer's scores at every update.
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kSelThreads = 1024;
constexpr int kBins = 2048;               // 11-bit digits
constexpr int kRegChunk = 32;             // positions per thread held in registers

__device__ __forceinline__ int digit_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ uint32_t digit_mask(int pass) { return pass == 2 ? 1023u : 2047u; }

// Exclusive prefix sum of one int per thread over the block; *total gets the block sum.
// sm must hold 33 ints.  Ends with a barrier.
__device__ __forceinline__ int block_excl_scan(int v, int* sm, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
  __syncthreads();
  if (lane == 31) sm[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < nw ? sm[lane] : 0;
    int s = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, s, o); if (lane >= o) s += t; }
    sm[lane] = s - w;
    if (lane == 31) sm[32] = s;
  }
  __syncthreads();
  const int r = sm[warp] + inc - v;
  *total = sm[32];
  __syncthreads();
  return r;
}

// Given hist[nbins] in shared memory (counts per digit, `total` entries in all), find the digit d
// holding the need-th largest entry: (#entries with digit > d) < need <= that + hist[d].
// Results go to out[0] = d, out[1] = need - (#entries with digit > d).  Every thread owns
// nbins / blockDim.x consecutive digits.  If offs != nullptr, the ascending exclusive offsets of all
// digits are written there (global).  Ends with a barrier; hist is unchanged.
__device__ __forceinline__ void find_digit(const unsigned int* hist, int nbins, int total, int need, int* sm_scan,
                                           volatile int* out, unsigned int* offs) {
  const int per = nbins / (int)blockDim.x;
  const int b0 = threadIdx.x * per;
  int mine = 0;
  for (int j = 0; j < per; ++j) mine += (int)hist[b0 + j];
  int tot;
  int off = block_excl_scan(mine, sm_scan, &tot);
  for (int j = 0; j < per; ++j) {
    const int c = (int)hist[b0 + j];
    if (offs) offs[b0 + j] = (unsigned int)off;
    const int above = total - off - c;
    if (c > 0 && above < need && need <= above + c) { out[0] = b0 + j; out[1] = need - above; }
    off += c;
  }
  __syncthreads();
}

// scores: [Bt*Hkv][P] of one layer.  idx: [Bt*Hkv][keep] kept positions, ascending.
// head_hist, head_offs: [Bt*Hkv][2048] first-digit counts of the head and their ascending exclusive offsets.
// grouped: [Bt*Hkv][P] the head's score bits grouped by first digit (ascending digit; order inside a
// group is unspecified).  Also records count[b][layer] = keep.
template <bool REG>
__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(const float* __restrict__ scores, int* __restrict__ idx, int* __restrict__ idx_out,
                   unsigned int* __restrict__ head_hist, unsigned int* __restrict__ head_offs,
                   uint32_t* __restrict__ grouped, int P, int keep, int* __restrict__ count, int Hkv, int L, int layer) {
  __shared__ unsigned int hist[kBins];
  __shared__ int sm_scan[33], sm_scan2[33];
  __shared__ int found[2];
  const int tid = threadIdx.x;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + (size_t)blockIdx.x * P;
  if (tid == 0 && blockIdx.x % Hkv == 0) count[(blockIdx.x / Hkv) * L + layer] = keep;

  const int chunk = (P + kSelThreads - 1) / kSelThreads;       // REG: chunk <= kRegChunk
  const int p0 = min(P, tid * chunk), p1 = min(P, p0 + chunk);
  const int n_mine = p1 - p0;
  uint32_t r[REG ? kRegChunk : 1];
  if (REG) {
#pragma unroll
    for (int e = 0; e < kRegChunk; ++e) r[e] = (e < n_mine) ? v[p0 + e] : 0u;
  }

  uint32_t prefix = 0, mask = 0;
  int need = keep, total = P;
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = digit_shift(pass);
    const uint32_t dm = digit_mask(pass);
    for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    if (REG) {
#pragma unroll
      for (int e = 0; e < kRegChunk; ++e)
        if (e < n_mine && (r[e] & mask) == prefix) atomicAdd(&hist[(r[e] >> shift) & dm], 1u);
    } else {
      for (int e = 0; e < n_mine; ++e) { const uint32_t u = v[p0 + e]; if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & dm], 1u); }
    }
    __syncthreads();
    if (pass == 0) {
      unsigned int* gh = head_hist + (size_t)blockIdx.x * kBins;
      for (int i = tid; i < kBins; i += kSelThreads) gh[i] = hist[i];
    }
    find_digit(hist, kBins, total, need, sm_scan, found, pass == 0 ? head_offs + (size_t)blockIdx.x * kBins : nullptr);
    const int d = found[0];
    const int cnt_d = (int)hist[d];
    if (pass == 0) {
      // group the head's scores by first digit: cursor[d] starts at the digit's offset
      const unsigned int* go = head_offs + (size_t)blockIdx.x * kBins;
      __syncthreads();
      for (int i = tid; i < kBins; i += kSelThreads) hist[i] = go[i];
      __syncthreads();
      uint32_t* dst = grouped + (size_t)blockIdx.x * P;
      if (REG) {
#pragma unroll
        for (int e = 0; e < kRegChunk; ++e)
          if (e < n_mine) dst[atomicAdd(&hist[r[e] >> 21], 1u)] = r[e];
      } else {
        for (int e = 0; e < n_mine; ++e) { const uint32_t u = v[p0 + e]; dst[atomicAdd(&hist[u >> 21], 1u)] = u; }
      }
    }
    total = cnt_d;
    need = found[1];
    prefix |= ((uint32_t)d) << shift;
    mask |= dm << shift;
    __syncthreads();
  }
  const uint32_t T = prefix;
  const int need_eq = need;                 // how many of the entries equal to T are kept (lowest positions)

  // Ordered compaction: each thread owns a contiguous run of positions.
  int gt = 0, eq = 0;
  if (REG) {
#pragma unroll
    for (int e = 0; e < kRegChunk; ++e) if (e < n_mine) { gt += (r[e] > T); eq += (r[e] == T); }
  } else {
    for (int e = 0; e < n_mine; ++e) { const uint32_t u = v[p0 + e]; gt += (u > T); eq += (u == T); }
  }
  int tot_gt, tot_eq;
  int g = block_excl_scan(gt, sm_scan, &tot_gt);
  int q = block_excl_scan(eq, sm_scan2, &tot_eq);
  int* my_idx = idx + (size_t)blockIdx.x * keep;
  int* my_out = idx_out ? idx_out + (size_t)blockIdx.x * keep : nullptr;
  if (REG) {
#pragma unroll
    for (int e = 0; e < kRegChunk; ++e) {
      if (e < n_mine) {
        const uint32_t u = r[e];
        const bool is_eq = (u == T);
        if (u > T || (is_eq && q < need_eq)) {
          const int out = g + min(q, need_eq);
          my_idx[out] = p0 + e;
          if (my_out) my_out[out] = p0 + e;
        }
        g += (u > T); q += is_eq;
      }
    }
  } else {
    for (int e = 0; e < n_mine; ++e) {
      const uint32_t u = v[p0 + e];
      const bool is_eq = (u == T);
      if (u > T || (is_eq && q < need_eq)) {
        const int out = g + min(q, need_eq);
        my_idx[out] = p0 + e;
        if (my_out) my_out[out] = p0 + e;
      }
      g += (u > T); q += is_eq;
    }
  }
}

// Rank of every held position among the held positions of its head, in (score descending, position
// ascending) order; equals its rank among all positions, because the held set is a top-n of that order.
// One CTA per (sample, head); dynamic shared memory = sort_n * 8 bytes, sort_n = power of two >= idx_stride.
__global__ void __launch_bounds__(kSelThreads)
rank_kernel(const float* __restrict__ scores, const int* __restrict__ idx, const int* __restrict__ held,
            int* __restrict__ rank_out, int P, int idx_stride, int sort_n, int Hkv, int L, int layer) {
  extern __shared__ __align__(16) unsigned long long skeys[];
  const int tid = threadIdx.x;
  const int n = held[(blockIdx.x / Hkv) * L + layer];
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + (size_t)blockIdx.x * P;
  const int* my_idx = idx + (size_t)blockIdx.x * idx_stride;
  for (int i = tid; i < sort_n; i += kSelThreads)
    skeys[i] = i < n ? (((unsigned long long)(~v[my_idx[i]]) << 32) | (unsigned int)i) : ~0ull;
  __syncthreads();
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
  for (int i = tid; i < n; i += kSelThreads)
    rank_out[(size_t)blockIdx.x * idx_stride + (int)(skeys[i] & 0xFFFFFFFFull)] = i;
}

}  // namespace dkv
