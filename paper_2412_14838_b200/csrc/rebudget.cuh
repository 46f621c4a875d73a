// Update_Buffer_Length (Eq. 4-6) on the device: a global top-K over the score history of the
// layers processed so far, counted per layer, then the integer budget arithmetic.
// Only per-layer counts leave the selection, so the K-th largest value T is found by a 3-pass
// radix select on the scores' bit patterns (non-negative floats order like unsigned ints), and
// the entries equal to T are handed out in flat-index order, i.e. to the lowest layers first.
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kRbBins = 2048;
constexpr int kRbThreads = 512;

struct RbState {          // per sample
  uint32_t prefix, mask;
  uint32_t remaining;     // how many of the entries matching `prefix` are still to be taken
  uint32_t pad;
};

__device__ __forceinline__ int rb_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ uint32_t rb_bins(int pass) { return pass == 2 ? 1024u : 2048u; }

// Start of an update: clear histograms and per-layer counters, state = (no prefix, k to take).
__global__ void rb_init_kernel(RbState* __restrict__ state, unsigned int* __restrict__ hist, unsigned int* __restrict__ cnt_gt,
                               unsigned int* __restrict__ cnt_eq, int Bt, int L, unsigned int k) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e < 3 * Bt * kRbBins) hist[e] = 0;
  if (e < Bt * L) { cnt_gt[e] = 0; cnt_eq[e] = 0; }
  if (e < Bt) { RbState st; st.prefix = 0; st.mask = 0; st.remaining = k; st.pad = 0; state[e] = st; }
}

// History layout: scores[layer][b][h][p].  grid (blocks per layer, l, Bt).
__global__ void __launch_bounds__(kRbThreads)
rb_hist_kernel(const float* __restrict__ scores, const RbState* __restrict__ state, unsigned int* __restrict__ hist,
               int pass, int Bt, size_t per_layer /* Hkv*P */) {
  __shared__ unsigned int sh[kRbBins];
  const int b = blockIdx.z, layer = blockIdx.y;
  for (int i = threadIdx.x; i < kRbBins; i += kRbThreads) sh[i] = 0;
  __syncthreads();
  const RbState st = state[b];
  const int shift = rb_shift(pass);
  const uint32_t bmask = rb_bins(pass) - 1u;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + ((size_t)layer * Bt + b) * per_layer;
  for (size_t i = (size_t)blockIdx.x * kRbThreads + threadIdx.x; i < per_layer; i += (size_t)gridDim.x * kRbThreads) {
    const uint32_t u = v[i];
    if ((u & st.mask) == st.prefix) atomicAdd(&sh[(u >> shift) & bmask], 1u);
  }
  __syncthreads();
  unsigned int* gh = hist + ((size_t)pass * Bt + b) * kRbBins;
  for (int i = threadIdx.x; i < kRbBins; i += kRbThreads) {
    const unsigned int c = sh[i];
    if (c) atomicAdd(&gh[i], c);
  }
}

// One block per sample: locate the bin holding the `remaining`-th largest entry and narrow the prefix.
__global__ void __launch_bounds__(1024)
rb_scan_kernel(RbState* __restrict__ state, const unsigned int* __restrict__ hist, int pass, int Bt) {
  __shared__ unsigned int cum[kRbBins];
  const int b = blockIdx.x;
  const unsigned int* gh = hist + ((size_t)pass * Bt + b) * kRbBins;
  for (int i = threadIdx.x; i < kRbBins; i += blockDim.x) cum[i] = gh[i];
  __syncthreads();
  if (threadIdx.x == 0) {
    RbState st = state[b];
    unsigned int above = 0;
    int bin = (int)rb_bins(pass) - 1;
    for (; bin > 0; --bin) {
      const unsigned int c = cum[bin];
      if (above + c >= st.remaining) break;
      above += c;
    }
    const int shift = rb_shift(pass);
    st.prefix |= ((uint32_t)bin) << shift;
    st.mask |= (rb_bins(pass) - 1u) << shift;
    st.remaining -= above;
    state[b] = st;
  }
}

// Per (layer, sample): entries above T and entries equal to T.  grid (blocks per layer, l, Bt).
__global__ void __launch_bounds__(kRbThreads)
rb_count_kernel(const float* __restrict__ scores, const RbState* __restrict__ state, unsigned int* __restrict__ cnt_gt,
                unsigned int* __restrict__ cnt_eq, int Bt, int L, size_t per_layer) {
  __shared__ unsigned int s_gt[kRbThreads / 32], s_eq[kRbThreads / 32];
  const int b = blockIdx.z, layer = blockIdx.y;
  const uint32_t T = state[b].prefix;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + ((size_t)layer * Bt + b) * per_layer;
  unsigned int gt = 0, eq = 0;
  for (size_t i = (size_t)blockIdx.x * kRbThreads + threadIdx.x; i < per_layer; i += (size_t)gridDim.x * kRbThreads) {
    const uint32_t u = v[i];
    gt += (u > T); eq += (u == T);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    gt += __shfl_xor_sync(0xFFFFFFFFu, gt, o);
    eq += __shfl_xor_sync(0xFFFFFFFFu, eq, o);
  }
  if ((threadIdx.x & 31) == 0) { s_gt[threadIdx.x >> 5] = gt; s_eq[threadIdx.x >> 5] = eq; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int g = 0, e = 0;
    for (int w = 0; w < kRbThreads / 32; ++w) { g += s_gt[w]; e += s_eq[w]; }
    if (g) atomicAdd(&cnt_gt[b * L + layer], g);
    if (e) atomicAdd(&cnt_eq[b * L + layer], e);
  }
}

// Eq. 5-6 in exact integers, one thread per sample (at most 128 layers).
// cnt_i = gt_i + share of the ties; Z_i = floor(Bl*cnt_i/max cnt); Z'_i = floor(Z_i*N*L/sum Z);
// count_i = min(count_i, Z'_i).
__global__ void rb_budget_kernel(const unsigned int* __restrict__ cnt_gt, const unsigned int* __restrict__ cnt_eq,
                                 int* __restrict__ count, int* __restrict__ dbg_cnt, int* __restrict__ dbg_z,
                                 int* __restrict__ dbg_zp, int* __restrict__ counts_out,
                                 int Bt, int L, int l, long long k, int Bl, int N) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= Bt) return;
  long long above = 0;
  for (int i = 0; i < l; ++i) above += cnt_gt[b * L + i];
  long long need = k - above;             // ties still to hand out, lowest layers first
  long long cmax = 0;
  for (int i = 0; i < l; ++i) {
    const long long e = cnt_eq[b * L + i];
    long long take = need < e ? need : e;
    if (take < 0) take = 0;
    need -= take;
    const long long c = (long long)cnt_gt[b * L + i] + take;
    dbg_cnt[b * L + i] = (int)c;
    cmax = c > cmax ? c : cmax;
  }
  if (cmax <= 0) cmax = 1;
  long long sumz = 0;
  for (int i = 0; i < l; ++i) {
    const long long z = ((long long)Bl * dbg_cnt[b * L + i]) / cmax;
    dbg_z[b * L + i] = (int)z;
    sumz += z;
  }
  if (sumz <= 0) sumz = 1;
  const long long B = (long long)N * L;
  for (int i = 0; i < l; ++i) {
    const long long zp = ((long long)dbg_z[b * L + i] * B) / sumz;
    const int zpi = zp > 0x7FFFFFFF ? 0x7FFFFFFF : (int)zp;
    dbg_zp[b * L + i] = zpi;
    const int c = count[b * L + i];
    count[b * L + i] = c < zpi ? c : zpi;
  }
  for (int i = l; i < L; ++i) { dbg_cnt[b * L + i] = 0; dbg_z[b * L + i] = 0; dbg_zp[b * L + i] = 0; }
  if (counts_out) for (int i = 0; i < L; ++i) counts_out[b * L + i] = count[b * L + i];
}

}  // namespace dkv
