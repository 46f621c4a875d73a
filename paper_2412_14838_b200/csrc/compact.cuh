// Algorithm 1's buffer build (gather kept rows + window rows) and its progressive truncation
// (keep the best count_i of the held rows, in position order, window last).
#pragma once
#include "common.cuh"
#include "select.cuh"

namespace dkv {

constexpr int kGatherRows = 4;      // rows per thread, all loads issued before the stores

// Gather: dst[b,h,i] = src[b,h, i < n ? idx[i] : P + (i - n)], i < n + ws.  16 bytes per thread per row.
// grid (row blocks, Bt*Hkv, 2 tensors).  n = kept positions per head (same for all heads); also records
// held[b][layer] = n.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src, uint4* __restrict__ kb,
                   uint4* __restrict__ vb, const int* __restrict__ idx, int n, int S, int P, int ws,
                   int row_stride /* rows per head in kb/vb */, int vec_per_row /* D*2/16 */,
                   int* __restrict__ held, int Hkv, int L, int layer) {
  const int bh = blockIdx.y;
  const uint4* src = (blockIdx.z == 0 ? k_src : v_src) + (size_t)bh * S * vec_per_row;
  uint4* dst = (blockIdx.z == 0 ? kb : vb) + (size_t)bh * row_stride * vec_per_row;
  if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.z == 0 && bh % Hkv == 0) held[(bh / Hkv) * L + layer] = n;
  const int rows_per_pass = 256 / vec_per_row;
  const int row0 = blockIdx.x * rows_per_pass * kGatherRows + threadIdx.x / vec_per_row;
  const int c = threadIdx.x % vec_per_row;
  uint4 val[kGatherRows];
#pragma unroll
  for (int j = 0; j < kGatherRows; ++j) {
    const int row = row0 + j * rows_per_pass;
    if (row < n + ws) {
      const int from = row < n ? idx[(size_t)bh * n + row] : P + (row - n);
      val[j] = src[(size_t)from * vec_per_row + c];
    }
  }
#pragma unroll
  for (int j = 0; j < kGatherRows; ++j) {
    const int row = row0 + j * rows_per_pass;
    if (row < n + ws) dst[(size_t)row * vec_per_row + c] = val[j];
  }
}

constexpr int kShrinkThreads = 256;
constexpr int kShrinkRows = 4;

// In-place shrink of one (layer, sample, head): grid (Bt*Hkv, layers); dynamic shared memory =
// max(2048, idx_stride) ints.  The best `want` of the `have` held positions under (score descending,
// position ascending) are found with the same 3-pass radix select as the per-head top-k, reading the
// held positions' scores from the history; because that order is total, this is the set Algorithm 1
// reaches by truncating its score-ordered buffer.  Kept rows only move towards the front
// (dst <= src, both increasing), so working through the destination rows in blocks, reading a whole
// block before writing it, never overwrites a row that is still to be read.
__global__ void __launch_bounds__(kShrinkThreads)
shrink_kernel(LayerPtrs ptrs, int layer0, const float* __restrict__ scores_all, int* __restrict__ idx_all,
              const int* __restrict__ count, const int* __restrict__ held, int Bt, int Hkv, int L, int P, int ws,
              int idx_stride /* Blc */, int row_stride, int vec_per_row, size_t layer_idx_stride /* Bt*Hkv*Blc */,
              size_t layer_score_stride /* Bt*Hkv*P */) {
  extern __shared__ unsigned int dyn[];      // histogram during the select, source map afterwards
  __shared__ int sm_scan[33], sm_scan2[33];
  __shared__ int found[2];
  const int layer = layer0 + blockIdx.y;
  const int bh = blockIdx.x, b = bh / Hkv;
  const int have = held[b * L + layer];
  const int want = min(count[b * L + layer], have);
  if (want == have) return;                                  // uniform across the block
  int* idx = idx_all + layer * layer_idx_stride + (size_t)bh * idx_stride;
  const uint32_t* v = reinterpret_cast<const uint32_t*>(scores_all) + layer * layer_score_stride + (size_t)bh * P;
  const int tid = threadIdx.x;
  const int chunk = (have + kShrinkThreads - 1) / kShrinkThreads;
  const int j0 = min(have, tid * chunk), j1 = min(have, j0 + chunk);
  int* src_map = reinterpret_cast<int*>(dyn);
  if (want > 0) {
    uint32_t prefix = 0, mask = 0;
    int need = want, total = have;
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = digit_shift(pass);
      const uint32_t dm = digit_mask(pass);
      for (int i = tid; i < kBins; i += kShrinkThreads) dyn[i] = 0;
      __syncthreads();
      for (int j = j0; j < j1; ++j) { const uint32_t u = v[idx[j]]; if ((u & mask) == prefix) atomicAdd(&dyn[(u >> shift) & dm], 1u); }
      __syncthreads();
      find_digit(dyn, kBins, total, need, sm_scan, found, nullptr);
      const int d = found[0];
      total = (int)dyn[d];
      need = found[1];
      prefix |= ((uint32_t)d) << shift;
      mask |= dm << shift;
      __syncthreads();
    }
    const uint32_t T = prefix;
    const int need_eq = need;
    int gt = 0, eq = 0;
    for (int j = j0; j < j1; ++j) { const uint32_t u = v[idx[j]]; gt += (u > T); eq += (u == T); }
    int tot_gt, tot_eq;
    int g = block_excl_scan(gt, sm_scan, &tot_gt);
    int q = block_excl_scan(eq, sm_scan2, &tot_eq);
    for (int j = j0; j < j1; ++j) {
      const uint32_t u = v[idx[j]];
      const bool is_eq = (u == T);
      if (u > T || (is_eq && q < need_eq)) src_map[g + min(q, need_eq)] = j;
      g += (u > T); q += is_eq;
    }
  }
  __syncthreads();
  // 1) kept positions
  for (int base = 0; base < want; base += kShrinkThreads) {
    const int d = base + tid;
    int vi = 0;
    if (d < want) vi = idx[src_map[d]];
    __syncthreads();
    if (d < want) idx[d] = vi;
    __syncthreads();
  }
  // 2) rows of K then V
  const int rows_per_pass = kShrinkThreads / vec_per_row;
  const int r_in = tid / vec_per_row, c = tid % vec_per_row;
  for (int t = 0; t < 2; ++t) {
    uint4* buf = reinterpret_cast<uint4*>(t == 0 ? ptrs.kb[layer] : ptrs.vb[layer]) + (size_t)bh * row_stride * vec_per_row;
    for (int base = 0; base < want + ws; base += rows_per_pass * kShrinkRows) {
      uint4 val[kShrinkRows];
#pragma unroll
      for (int j = 0; j < kShrinkRows; ++j) {
        const int d = base + j * rows_per_pass + r_in;
        if (d < want + ws) {
          const int from = d < want ? src_map[d] : have + (d - want);
          val[j] = buf[(size_t)from * vec_per_row + c];
        }
      }
      __syncthreads();
#pragma unroll
      for (int j = 0; j < kShrinkRows; ++j) {
        const int d = base + j * rows_per_pass + r_in;
        if (d < want + ws) buf[(size_t)d * vec_per_row + c] = val[j];
      }
      __syncthreads();
    }
  }
}

// After a shrink: the buffers of layers [layer0, layer0 + n) now hold min(held, count) rows.
__global__ void commit_held_kernel(int* __restrict__ held, const int* __restrict__ count, int Bt, int L, int layer0, int n) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= Bt * n) return;
  const int b = e / n, layer = layer0 + e % n;
  const int h = held[b * L + layer], c = count[b * L + layer];
  held[b * L + layer] = c < h ? c : h;
}

// len_out[b][h] = held[b][layer] + ws
__global__ void write_len_kernel(int* __restrict__ len_out, const int* __restrict__ held, int Bt, int Hkv, int L, int layer, int ws) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= Bt * Hkv) return;
  len_out[e] = held[(e / Hkv) * L + layer] + ws;
}

}  // namespace dkv
