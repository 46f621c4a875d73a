// Update_Buffer_Length (Eq. 4-6) on the device: the K-th largest of all scores of the layers processed
// so far, the number of top-K hits per layer, then the integer budget arithmetic.
//
// Only per-layer counts leave the selection.  Every layer's scores were histogrammed by their first
// 11-bit digit when the layer was selected (select.cuh), so:
//   rb_locate   adds up the histograms of layers [0, l), finds the digit b* that holds the K-th
//               largest score, and counts each layer's scores above b* from its histogram;
//   rb_refine1  streams the history once, copies the scores whose first digit is b* (with their layer)
//               into a candidate list and histograms their next 11 bits;
//   rb_refine2  counts, per layer, the candidates above the second digit and histograms the last
//               10 bits of those that match it;
//   rb_budget   fixes the exact threshold T, gives the entries equal to T to the lowest layers first
//               (flat-index tie rule), and evaluates Eq. 5-6 in exact integers.
#pragma once
#include "common.cuh"
#include "select.cuh"

namespace dkv {

constexpr int kRbThreads = 256;

struct RbState {          // per sample
  int bstar;              // first digit of T
  int need1;              // entries still to take inside bucket b*
  int cand;               // entries in bucket b* over all layers and heads
  int pad;
};

// One CTA of 1024 threads per sample.
// layer_hist: [L][Bt][2048].  above: [Bt][L] scores above bucket b* per layer.
// hist1: [Bt][2048], above2: [Bt][L], hist2: [Bt][L][1024], cand_n: [Bt] are cleared here for the refine kernels.
__global__ void __launch_bounds__(1024)
rb_locate_kernel(const unsigned int* __restrict__ layer_hist, RbState* __restrict__ state,
                 unsigned int* __restrict__ above, unsigned int* __restrict__ hist1, unsigned int* __restrict__ above2,
                 unsigned int* __restrict__ hist2, unsigned int* __restrict__ cand_n, int Bt, int Hkv, int L, int l, int P,
                 long long k) {
  __shared__ unsigned int hist[kBins];
  __shared__ int sm_scan[33];
  __shared__ int found[2];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  {
    // two digits per thread, summed over the layers (consecutive threads read consecutive words)
    uint2 a = make_uint2(0, 0);
    for (int i = 0; i < l; ++i) {
      const uint2 x = reinterpret_cast<const uint2*>(layer_hist + ((size_t)i * Bt + b) * kBins)[tid];
      a.x += x.x; a.y += x.y;
    }
    hist[2 * tid] = a.x; hist[2 * tid + 1] = a.y;
    hist1[(size_t)b * kBins + 2 * tid] = 0; hist1[(size_t)b * kBins + 2 * tid + 1] = 0;
  }
  if (tid == 0) cand_n[b] = 0;
  for (int e = tid; e < L; e += 1024) above2[b * L + e] = 0;
  for (int e = tid; e < l * 1024; e += 1024) hist2[(size_t)b * L * 1024 + e] = 0;
  __syncthreads();
  const long long total = (long long)l * Hkv * P;
  find_digit(hist, kBins, (int)total, (int)k, sm_scan, found, nullptr);
  const int d = found[0];
  if (tid == 0) { RbState st; st.bstar = d; st.need1 = found[1]; st.cand = (int)hist[d]; st.pad = 0; state[b] = st; }
  // one warp per layer: the layer's scores in the digits above b*
  for (int i = warp; i < l; i += 32) {
    const unsigned int* lh = layer_hist + ((size_t)i * Bt + b) * kBins;
    unsigned int a = 0;
    for (int bin = d + 1 + lane; bin < kBins; bin += 32) a += lh[bin];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
    if (lane == 0) above[b * L + i] = a;
  }
}

// grid (slices, l, Bt): one pass over the scores of layers [0, l).  Scores whose first digit is b* go to the
// sample's candidate list (value, layer) and into the second-digit histogram.  The list has room for every
// score (cand[b] holds l*Hkv*P pairs at most); its order is arbitrary, only counts are taken from it.
// A block reads its slice once, in chunks of kRbChunk scores: matches are parked in shared memory, then the
// block reserves a range of the list with one atomic and copies them out.
constexpr int kRbChunk = 4096;
__global__ void __launch_bounds__(kRbThreads)
rb_refine1_kernel(const float* __restrict__ scores, const RbState* __restrict__ state, unsigned int* __restrict__ hist1,
                  uint2* __restrict__ cand, unsigned int* __restrict__ cand_n, int Bt, size_t per_layer /* Hkv*P */,
                  size_t cand_stride) {
  __shared__ unsigned int sh[kBins];
  __shared__ uint32_t parked[kRbChunk];
  __shared__ unsigned int s_cnt, s_base;
  const int b = blockIdx.z, i = blockIdx.y;
  const uint32_t d = (uint32_t)state[b].bstar;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + ((size_t)i * Bt + b) * per_layer;
  for (int j = threadIdx.x; j < kBins; j += kRbThreads) sh[j] = 0;
  const size_t per_block = (per_layer + gridDim.x - 1) / gridDim.x;
  const size_t e0 = (size_t)blockIdx.x * per_block, e1 = e0 + per_block < per_layer ? e0 + per_block : per_layer;
  uint2* list = cand + (size_t)b * cand_stride;
  for (size_t c0 = e0; c0 < e1; c0 += kRbChunk) {
    if (threadIdx.x == 0) s_cnt = 0;
    __syncthreads();
    const size_t c1 = c0 + kRbChunk < e1 ? c0 + kRbChunk : e1;
    uint32_t u[kRbChunk / kRbThreads];
#pragma unroll
    for (int j = 0; j < kRbChunk / kRbThreads; ++j) {          // all loads of the chunk in flight together
      const size_t e = c0 + threadIdx.x + (size_t)j * kRbThreads;
      u[j] = e < c1 ? v[e] : 0xFFFFFFFFu;                      // (a NaN pattern: its first digit 2047 never is b*)
    }
#pragma unroll
    for (int j = 0; j < kRbChunk / kRbThreads; ++j) {
      const size_t e = c0 + threadIdx.x + (size_t)j * kRbThreads;
      if (e < c1 && (u[j] >> 21) == d) {
        parked[atomicAdd(&s_cnt, 1u)] = u[j];
        atomicAdd(&sh[(u[j] >> 10) & 2047u], 1u);
      }
    }
    __syncthreads();
    const unsigned int n = s_cnt;
    if (n) {
      if (threadIdx.x == 0) s_base = atomicAdd(&cand_n[b], n);
      __syncthreads();
      for (unsigned int x = threadIdx.x; x < n; x += kRbThreads) list[s_base + x] = make_uint2(parked[x], (unsigned int)i);
    }
    __syncthreads();
  }
  for (int j = threadIdx.x; j < kBins; j += kRbThreads) { const unsigned int c = sh[j]; if (c) atomicAdd(&hist1[(size_t)b * kBins + j], c); }
}

// grid (slices, Bt) over the candidate list.  Every block re-derives the second digit s* from hist1; then per
// layer: candidates with a larger second digit (above2) and the last-10-bit histogram of those with second
// digit s* (hist2).
__global__ void __launch_bounds__(kRbThreads)
rb_refine2_kernel(const uint2* __restrict__ cand, const unsigned int* __restrict__ cand_n, const RbState* __restrict__ state,
                  const unsigned int* __restrict__ hist1, unsigned int* __restrict__ above2,
                  unsigned int* __restrict__ hist2, int L, size_t cand_stride) {
  __shared__ unsigned int sh[kBins];
  __shared__ int sm_scan[33];
  __shared__ int found[2];
  const int b = blockIdx.y;
  const RbState st = state[b];
  const unsigned int n = cand_n[b];
  if (blockIdx.x * kRbThreads >= n) return;
  for (int j = threadIdx.x; j < kBins; j += kRbThreads) sh[j] = hist1[(size_t)b * kBins + j];
  __syncthreads();
  find_digit(sh, kBins, st.cand, st.need1, sm_scan, found, nullptr);
  const uint32_t s2 = (uint32_t)found[0];
  const uint2* list = cand + (size_t)b * cand_stride;
  // the per-layer counters are few and hot: count in shared memory (sh is free again), one global add per layer
  __syncthreads();
  for (int j = threadIdx.x; j < L; j += kRbThreads) sh[j] = 0;
  __syncthreads();
  for (unsigned int e = blockIdx.x * kRbThreads + threadIdx.x; e < n; e += gridDim.x * kRbThreads) {
    const uint2 c = list[e];
    const uint32_t dd = (c.x >> 10) & 2047u;
    if (dd > s2) atomicAdd(&sh[c.y], 1u);
    else if (dd == s2) atomicAdd(&hist2[((size_t)b * L + c.y) * 1024 + (c.x & 1023u)], 1u);
  }
  __syncthreads();
  for (int j = threadIdx.x; j < L; j += kRbThreads) { const unsigned int v = sh[j]; if (v) atomicAdd(&above2[b * L + j], v); }
}

// One CTA of 1024 threads per sample: exact T, per-layer hits, Eq. 5-6.
// cnt_i = hits of layer i among the K largest (ties at T to the lowest layers first);
// Z_i = floor(Bl*cnt_i/max cnt); Z'_i = floor(Z_i*N*L/sum Z); count_i = min(count_i, Z'_i).
__global__ void __launch_bounds__(1024)
rb_budget_kernel(const RbState* __restrict__ state, const unsigned int* __restrict__ hist1,
                 const unsigned int* __restrict__ above, const unsigned int* __restrict__ above2,
                 const unsigned int* __restrict__ hist2, int* __restrict__ count, int* __restrict__ dbg_cnt,
                 int* __restrict__ dbg_z, int* __restrict__ dbg_zp, int* __restrict__ counts_out,
                 int Bt, int L, int l, int Bl, int N, int prorata, int minmax) {
  __shared__ unsigned int sh[kBins];
  __shared__ int sm_scan[33];
  __shared__ int found[2];
  __shared__ long long s_gt[128], s_eq[128];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const RbState st = state[b];
  for (int j = tid; j < kBins; j += 1024) sh[j] = hist1[(size_t)b * kBins + j];
  __syncthreads();
  find_digit(sh, kBins, st.cand, st.need1, sm_scan, found, nullptr);
  const int need2 = found[1];
  const int cand2 = (int)sh[found[0]];
  __syncthreads();
  // last digit: total histogram over layers
  for (int j = tid; j < kBins; j += 1024) {
    unsigned int s = 0;
    if (j < 1024) for (int i = 0; i < l; ++i) s += hist2[((size_t)b * L + i) * 1024 + j];
    sh[j] = s;
  }
  __syncthreads();
  find_digit(sh, kBins, cand2, need2, sm_scan, found, nullptr);
  const int t_low = found[0];
  long long ties = found[1];                  // entries equal to T that are taken, lowest layers first
  // per layer: entries above T and equal to T (one warp per layer)
  for (int i = warp; i < l; i += 32) {
    unsigned int g = 0;
    for (int j = t_low + 1 + lane; j < 1024; j += 32) g += hist2[((size_t)b * L + i) * 1024 + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) g += __shfl_xor_sync(0xFFFFFFFFu, g, o);
    if (lane == 0) {
      s_gt[i] = (long long)above[b * L + i] + above2[b * L + i] + g;
      s_eq[i] = hist2[((size_t)b * L + i) * 1024 + t_low];
    }
  }
  __syncthreads();
  // Eq. 5-6 with one thread per layer (warp 0; layers lane, lane + 32, ...): the ties go to the lowest layers
  // first, i.e. layer i takes min(eq_i, ties - sum of eq below i).
  if (warp == 0) {
    long long carry = 0, cmax = 0, cmin = 0x7FFFFFFFFFFFFFFFll;
    for (int i0 = 0; i0 < l; i0 += 32) {
      const int i = i0 + lane;
      const long long eq = i < l ? s_eq[i] : 0;
      long long incl = eq;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const long long y = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += y; }
      const long long before = carry + incl - eq;
      long long take = ties - before;
      take = take < 0 ? 0 : (take < eq ? take : eq);
      if (i < l) {
        s_gt[i] += take;                      // = cnt_i
        dbg_cnt[b * L + i] = (int)s_gt[i];
        cmax = s_gt[i] > cmax ? s_gt[i] : cmax;
        cmin = s_gt[i] < cmin ? s_gt[i] : cmin;
      }
      carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const long long y = __shfl_xor_sync(0xFFFFFFFFu, cmax, o); cmax = y > cmax ? y : cmax; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const long long y = __shfl_xor_sync(0xFFFFFFFFu, cmin, o); cmin = y < cmin ? y : cmin; }
    if (cmax <= 0) cmax = 1;
    long long sumz = 0;
    for (int i = lane; i < l; i += 32) {
      // Z_i: counts scaled by their maximum, or (variant) min-max scaled; all layers equal under min-max -> Bl each
      if (minmax) s_eq[i] = cmax == cmin ? (long long)Bl : ((long long)Bl * (s_gt[i] - cmin)) / (cmax - cmin);
      else s_eq[i] = ((long long)Bl * s_gt[i]) / cmax;
      dbg_z[b * L + i] = (int)s_eq[i];
      sumz += s_eq[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sumz += __shfl_xor_sync(0xFFFFFFFFu, sumz, o);
    if (sumz <= 0) sumz = 1;
    const long long B = (long long)N * (prorata ? l : L);      // Eq. 6's budget (variant: of the layers seen so far)
    for (int i = lane; i < l; i += 32) {
      const long long zp = (s_eq[i] * B) / sumz;              // Z'_i
      const int zpi = zp > 0x7FFFFFFF ? 0x7FFFFFFF : (int)zp;
      dbg_zp[b * L + i] = zpi;
      const int c = count[b * L + i];
      count[b * L + i] = c < zpi ? c : zpi;
    }
    for (int i = l + lane; i < L; i += 32) { dbg_cnt[b * L + i] = 0; dbg_z[b * L + i] = 0; dbg_zp[b * L + i] = 0; }
  }
  __syncthreads();
  if (counts_out) for (int i = tid; i < L; i += 1024) counts_out[b * L + i] = count[b * L + i];
}

}  // namespace dkv
