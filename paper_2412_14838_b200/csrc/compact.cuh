// Algorithm 1's buffer build (gather kept rows + window rows) and its progressive truncation
// (keep the best count_i of the held rows, window last).  Rows are kept in the order Algorithm 1's
// topk() yields them: score descending, ties by position.
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kGatherRows = 4;      // rows per thread, all loads issued before the stores

// Gather: dst[b,h,i] = src[b,h, i < n ? idx[i] : P + (i - n)], i < n + ws.  16 bytes per thread per row.
// grid (row blocks, Bt*Hkv, 2 tensors).  n = kept positions per head (same for all heads), idx_stride = entries
// per head in idx; also records held[b][layer] = n.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src, uint4* __restrict__ kb,
                   uint4* __restrict__ vb, const int* __restrict__ idx, int n, int idx_stride, int S, int P, int ws,
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
      const int from = row < n ? idx[(size_t)bh * idx_stride + row] : P + (row - n);
      val[j] = __ldcs(&src[(size_t)from * vec_per_row + c]);      // read once: first in line for eviction from L2
    }
  }
#pragma unroll
  for (int j = 0; j < kGatherRows; ++j) {
    const int row = row0 + j * rows_per_pass;
    if (row < n + ws) __stcs(&dst[(size_t)row * vec_per_row + c], val[j]);
  }
}

constexpr int kShrinkThreads = 256;

// In-place truncation of one (layer, sample, head, tensor): grid (Bt*Hkv, layers, 2).
// The buffers are in Algorithm 1's own order (score descending), so cutting a layer from `have` to
// `want` kept rows keeps the first `want` rows where they are; only the ws window rows move, from
// [have, have+ws) to [want, want+ws).  The two ranges may overlap (dst < src): rows are moved in
// blocks, each block read completely before it is written.
__global__ void __launch_bounds__(kShrinkThreads)
shrink_kernel(LayerPtrs ptrs, int layer0, const int* __restrict__ count, const int* __restrict__ held, int Hkv, int L,
              int ws, int row_stride, int vec_per_row) {
  const int layer = layer0 + blockIdx.y;
  const int bh = blockIdx.x, b = bh / Hkv;
  const int have = held[b * L + layer];
  const int want = min(count[b * L + layer], have);
  if (want == have) return;                                  // uniform across the block
  uint4* buf = reinterpret_cast<uint4*>(blockIdx.z == 0 ? ptrs.kb[layer] : ptrs.vb[layer]) + (size_t)bh * row_stride * vec_per_row;
  const uint4* src = buf + (size_t)have * vec_per_row;
  uint4* dst = buf + (size_t)want * vec_per_row;
  const int n = ws * vec_per_row;
  for (int base = 0; base < n; base += kShrinkThreads) {
    const int e = base + threadIdx.x;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (e < n) val = src[e];
    __syncthreads();
    if (e < n) dst[e] = val;
    __syncthreads();
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
