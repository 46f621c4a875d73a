// Per-head top-B^l (Eq. 3; Algorithm 1's "topk(B^l)") under the total order
// (score descending, position ascending), plus what the later global top-K (Eq. 4) needs from
// this layer.  One CTA per (sample, KV head).
//
// Scores are non-negative floats, so their bit patterns order like unsigned integers.  The
// threshold T (bit pattern of the B^l-th largest score) is found by a 3-pass radix select,
// most significant digit first (11 + 11 + 10 bits), with a shared-memory histogram per pass.
// The kept positions are then compacted in position order and sorted by (score descending,
// position ascending): that is the order Algorithm 1's topk() returns and stores them in, and a
// later truncation to a smaller budget is a prefix of it.
// The first pass's histogram (top 11 bits: sign, exponent, 2 mantissa bits) is also kept per head
// in global memory with its prefix offsets, so that Update_Buffer_Length can locate the first digit
// of the global K-th value, and each layer's count of scores above it, from histograms alone.
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kSelThreads = 1024;
constexpr int kBins = 2048;               // 11-bit digits
constexpr int kRegChunk = 32;             // scores per thread held in registers

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

// Counter bump without a return value for digits that come in runs (pooled scores: neighbouring positions share
// their digit): a run of equal digits in adjacent lanes makes one atomicAdd of its length.  Equal digits that are
// not adjacent are added separately.  Must be called by all 32 lanes.
__device__ __forceinline__ void run_bump(unsigned int* counters, unsigned int digit, bool active) {
  const unsigned int lane = threadIdx.x & 31;
  const unsigned int key = active ? digit : 0xFFFFFFFFu;
  const unsigned int prev = __shfl_up_sync(0xFFFFFFFFu, key, 1);
  const bool head = lane == 0 || prev != key;
  const unsigned int heads = __ballot_sync(0xFFFFFFFFu, head);
  if (head && active) {
    const unsigned int later = heads & ~((2u << lane) - 1u);       // run heads after this lane (lane 31: none)
    const int next = later ? __ffs(later) - 1 : 32;
    atomicAdd(&counters[digit], (unsigned int)(next - (int)lane));
  }
}

// One compare-exchange step of a bitonic network on the 64 keys a warp holds in registers: lane j has
// a = key[base + j] and b = key[base + 32 + j].  `s` is the stride (32, 16, ..., 1), `size` the length of the
// bitonic sequences being merged; a block of `size` keys is sorted ascending if its first index has bit `size` clear.
__device__ __forceinline__ void bitonic_step64(unsigned long long& a, unsigned long long& b, int base, int lane, int s, int size) {
  if (s == 32) {
    const bool up = ((base + lane) & size) == 0;
    if ((a > b) == up) { const unsigned long long t = a; a = b; b = t; }
  } else {
    const unsigned long long pa = __shfl_xor_sync(0xFFFFFFFFu, a, s), pb = __shfl_xor_sync(0xFFFFFFFFu, b, s);
    const bool lower = (lane & s) == 0;                       // this lane holds the lower index of its pair
    const bool up_a = ((base + lane) & size) == 0, up_b = ((base + 32 + lane) & size) == 0;
    a = (lower == up_a) ? (a < pa ? a : pa) : (a > pa ? a : pa);
    b = (lower == up_b) ? (b < pb ? b : pb) : (b > pb ? b : pb);
  }
}

// Bitonic sort of keys[0 .. sort_n) ascending; sort_n a power of two >= 2.  Strides of 64 and more are
// done by the whole block in shared memory with a barrier per stage; the strides below that stay inside
// 64-key blocks, each owned by one warp, which holds its block in registers (two keys per lane) and
// exchanges by shuffles; the first six merge lengths (2 .. 64) run entirely in registers.  Arrays of
// fewer than 64 keys use shared memory throughout.  Ends with a block barrier.
__device__ __forceinline__ void bitonic_sort(unsigned long long* keys, int sort_n) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  if (sort_n < 64) {
    for (int size = 2; size <= sort_n; size <<= 1) {
      for (int s = size >> 1; s > 0; s >>= 1) {
        for (int t = threadIdx.x; t < (sort_n >> 1); t += blockDim.x) {
          const int lo = ((t & ~(s - 1)) << 1) | (t & (s - 1)), hi = lo + s;
          const bool up = ((lo & size) == 0);
          const unsigned long long a = keys[lo], b = keys[hi];
          if ((a > b) == up) { keys[lo] = b; keys[hi] = a; }
        }
        __syncthreads();
      }
    }
    return;
  }
  __syncthreads();
  for (int base = warp * 64; base < sort_n; base += nwarps * 64) {      // merge lengths 2 .. 64 in registers
    unsigned long long a = keys[base + lane], b = keys[base + 32 + lane];
    for (int size = 2; size <= 64; size <<= 1)
      for (int s = size >> 1; s > 0; s >>= 1) bitonic_step64(a, b, base, lane, s, size);
    keys[base + lane] = a; keys[base + 32 + lane] = b;
  }
  __syncthreads();
  for (int size = 128; size <= sort_n; size <<= 1) {
    for (int stride = size >> 1; stride >= 64; stride >>= 1) {
      for (int t = threadIdx.x; t < (sort_n >> 1); t += blockDim.x) {
        const int lo = ((t & ~(stride - 1)) << 1) | (t & (stride - 1));
        const int hi = lo + stride;
        const bool up = ((lo & size) == 0);
        const unsigned long long a = keys[lo], b = keys[hi];
        if ((a > b) == up) { keys[lo] = b; keys[hi] = a; }
      }
      __syncthreads();
    }
    for (int base = warp * 64; base < sort_n; base += nwarps * 64) {
      unsigned long long a = keys[base + lane], b = keys[base + 32 + lane];
#pragma unroll
      for (int s = 32; s > 0; s >>= 1) bitonic_step64(a, b, base, lane, s, size);
      keys[base + lane] = a; keys[base + 32 + lane] = b;
    }
    __syncthreads();
  }
}

// scores: [Bt*Hkv][P] of one layer.
// idx: [Bt*Hkv][keep] kept positions in buffer order = (score descending, position ascending).
// sorted_out (optional): the same positions ascending; rank_out (optional): rank of each of those.
// layer_hist: [Bt][2048] first-digit counts of the layer's scores, all heads of a sample added up (zeroed by
// the host before the launch); the rebudget works from these.
// Also records count[b][layer] = keep.
// Every warp owns a run of 32*chunk consecutive positions; lane j holds positions run + 32*e + j.
// Dynamic shared memory: 8*sort_n bytes, then 4*keep bytes.
template <bool REG>
__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(const float* __restrict__ scores, int* __restrict__ idx, int* __restrict__ sorted_out,
                   int* __restrict__ rank_out, unsigned int* __restrict__ layer_hist,
                   int P, int keep, int sort_n, int* __restrict__ count, int Hkv, int L, int layer) {
  extern __shared__ __align__(16) unsigned char dyn[];
  __shared__ unsigned int hist[kBins];
  __shared__ int sm_scan[33], sm_scan2[33];
  __shared__ int found[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores) + (size_t)blockIdx.x * P;
  if (tid == 0 && blockIdx.x % Hkv == 0) count[(blockIdx.x / Hkv) * L + layer] = keep;

  unsigned long long* keys = reinterpret_cast<unsigned long long*>(dyn);
  int* sel_pos = reinterpret_cast<int*>(dyn + (size_t)sort_n * 8);

  const int chunk = (P + kSelThreads - 1) / kSelThreads;       // REG: chunk <= kRegChunk
  const int run0 = warp * chunk * 32;
  const int n_e = REG ? kRegChunk : chunk;
  // which of this lane's slots hold a position: slots [0, n_ok)
  const int n_ok = min(chunk, max(0, (P - run0 - lane + 31) / 32));
  uint32_t r[REG ? kRegChunk : 1];
  if constexpr (REG) {
#pragma unroll
    for (int e = 0; e < kRegChunk; ++e) r[e] = e < n_ok ? v[run0 + e * 32 + lane] : 0u;
  }
#define DKV_SEL_FOR(e) _Pragma("unroll") for (int e = 0; e < n_e; ++e)
#define DKV_SEL_POS(e) (run0 + (e) * 32 + lane)
#define DKV_SEL_OK(e) ((e) < n_ok)
  auto val = [&](int e) -> uint32_t {
    if constexpr (REG) return r[e]; else return DKV_SEL_OK(e) ? v[DKV_SEL_POS(e)] : 0u;
  };

  // pass 0: first digit of every score; neighbours share digits after pooling, so lanes combine their bumps
  for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
  __syncthreads();
  DKV_SEL_FOR(e) run_bump(hist, val(e) >> 21, DKV_SEL_OK(e));
  __syncthreads();
  {
    unsigned int* gh = layer_hist + (size_t)(blockIdx.x / Hkv) * kBins;
    for (int i = tid; i < kBins; i += kSelThreads) { const unsigned int c = hist[i]; if (c) atomicAdd(&gh[i], c); }
  }
  find_digit(hist, kBins, P, keep, sm_scan, found, nullptr);
  uint32_t prefix = ((uint32_t)found[0]) << 21, mask = 2047u << 21;
  int need = found[1], total = (int)hist[found[0]];
  __syncthreads();
  // passes 1, 2: only the scores inside the first digit's bucket take part
  for (int pass = 1; pass < 3; ++pass) {
    const int shift = digit_shift(pass);
    const uint32_t dm = digit_mask(pass);
    for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    DKV_SEL_FOR(e) {
      const uint32_t u = val(e);
      if (DKV_SEL_OK(e) && (u & mask) == prefix) atomicAdd(&hist[(u >> shift) & dm], 1u);
    }
    __syncthreads();
    find_digit(hist, kBins, total, need, sm_scan, found, nullptr);
    const int d = found[0];
    total = (int)hist[d];
    need = found[1];
    prefix |= ((uint32_t)d) << shift;
    mask |= dm << shift;
    __syncthreads();
  }
  const uint32_t T = prefix;
  const int need_eq = need;                 // how many of the entries equal to T are kept (lowest positions)

  // Ordered compaction.  Position order inside a warp's run is (e, lane), so ballots give the order.
  int gt = 0, eq = 0;
  DKV_SEL_FOR(e) { const uint32_t u = val(e); if (DKV_SEL_OK(e)) { gt += (u > T); eq += (u == T); } }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { gt += __shfl_xor_sync(0xFFFFFFFFu, gt, o); eq += __shfl_xor_sync(0xFFFFFFFFu, eq, o); }
  int tot_gt, tot_eq;
  int g_run = block_excl_scan(lane == 0 ? gt : 0, sm_scan, &tot_gt);       // one value per warp, carried by lane 0
  int q_run = block_excl_scan(lane == 0 ? eq : 0, sm_scan2, &tot_eq);
  g_run = __shfl_sync(0xFFFFFFFFu, g_run, 0);
  q_run = __shfl_sync(0xFFFFFFFFu, q_run, 0);
  const unsigned int lt = (1u << lane) - 1u;
  int* my_sorted = sorted_out ? sorted_out + (size_t)blockIdx.x * keep : nullptr;
  DKV_SEL_FOR(e) {
    const uint32_t u = val(e);
    const bool ok = DKV_SEL_OK(e);
    const bool is_gt = ok && u > T, is_eq = ok && u == T;
    const unsigned int bg = __ballot_sync(0xFFFFFFFFu, is_gt), be = __ballot_sync(0xFFFFFFFFu, is_eq);
    if (bg | be) {                           // warp-uniform: most rows of 32 positions keep nothing
      const int g = g_run + __popc(bg & lt), q = q_run + __popc(be & lt);
      if (is_gt || (is_eq && q < need_eq)) {
        const int out = g + min(q, need_eq);
        const int p = DKV_SEL_POS(e);
        sel_pos[out] = p;
        if (my_sorted) my_sorted[out] = p;
        keys[out] = ((unsigned long long)(~u) << 32) | (unsigned int)out;
      }
      g_run += __popc(bg); q_run += __popc(be);
    }
  }
  for (int i = tid + keep; i < sort_n; i += kSelThreads) keys[i] = ~0ull;
  __syncthreads();
  bitonic_sort(keys, sort_n);
  int* my_idx = idx + (size_t)blockIdx.x * keep;
  for (int i = tid; i < keep; i += kSelThreads) {
    const int slot = (int)(keys[i] & 0xFFFFFFFFull);
    my_idx[i] = sel_pos[slot];
    if (rank_out) rank_out[(size_t)blockIdx.x * keep + slot] = i;
  }
#undef DKV_SEL_FOR
#undef DKV_SEL_POS
#undef DKV_SEL_OK
}

// Ascending list of the positions a head currently holds: sorted_out[b,h,0:held] (one CTA per head).
// Dynamic shared memory: ceil(P / 32) words (one bit per position).
__global__ void __launch_bounds__(kSelThreads)
kept_sorted_kernel(const int* __restrict__ idx, const int* __restrict__ held, int* __restrict__ sorted_out, int P,
                   int idx_stride, int Hkv, int L, int layer) {
  extern __shared__ unsigned int bits[];
  __shared__ int sm_scan[33];
  const int tid = threadIdx.x;
  const int n = held[(blockIdx.x / Hkv) * L + layer];
  const int words = (P + 31) / 32;
  for (int i = tid; i < words; i += kSelThreads) bits[i] = 0;
  __syncthreads();
  const int* my = idx + (size_t)blockIdx.x * idx_stride;
  for (int i = tid; i < n; i += kSelThreads) { const int p = my[i]; atomicOr(&bits[p >> 5], 1u << (p & 31)); }
  __syncthreads();
  const int per = (words + kSelThreads - 1) / kSelThreads;
  const int w0 = min(words, tid * per), w1 = min(words, w0 + per);
  int mine = 0;
  for (int w = w0; w < w1; ++w) mine += __popc(bits[w]);
  int tot;
  int out = block_excl_scan(mine, sm_scan, &tot);
  int* dst = sorted_out + (size_t)blockIdx.x * idx_stride;
  for (int w = w0; w < w1; ++w) {
    unsigned int m = bits[w];
    while (m) { const int b = __ffs(m) - 1; dst[out++] = w * 32 + b; m &= m - 1; }
  }
}

}  // namespace dkv
