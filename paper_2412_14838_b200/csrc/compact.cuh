// Algorithm 1's buffer build (gather kept rows + window rows) and its progressive truncation
// (keep the rows whose rank is below the layer's new count, in position order, window last).
#pragma once
#include "common.cuh"

namespace dkv {

// Gather: dst[b,h,i] = src[b,h, i < n ? idx[i] : P + (i - n)], i < n + ws.  16 bytes per thread.
// grid (row blocks, Bt*Hkv, 2 tensors).  n = kept positions held per head (same for all heads);
// also records held[b][layer] = n.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src, uint4* __restrict__ kb,
                   uint4* __restrict__ vb, const int* __restrict__ idx, int n, int S, int P, int ws,
                   int row_stride /* rows per head in kb/vb */, int vec_per_row /* D*2/16 */,
                   int* __restrict__ held, int Hkv, int L, int layer) {
  const uint4* src = blockIdx.z == 0 ? k_src : v_src;
  uint4* dst = blockIdx.z == 0 ? kb : vb;
  const int bh = blockIdx.y;
  if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.z == 0 && bh % Hkv == 0) held[(bh / Hkv) * L + layer] = n;
  const int rows_per_block = 256 / vec_per_row;
  const int row = blockIdx.x * rows_per_block + threadIdx.x / vec_per_row;
  const int c = threadIdx.x % vec_per_row;
  if (row >= n + ws) return;
  const int from = row < n ? idx[(size_t)bh * n + row] : P + (row - n);
  dst[((size_t)bh * row_stride + row) * vec_per_row + c] = src[((size_t)bh * S + from) * vec_per_row + c];
}

constexpr int kShrinkThreads = 1024;

// In-place shrink of one (layer, sample, head): grid (Bt*Hkv, layers), dynamic smem = idx_stride ints.
// Kept rows only move towards the front (dst <= src, both increasing), so working through the
// destination rows in blocks, reading a whole block before writing it, never overwrites a row
// that is still to be read.
__global__ void __launch_bounds__(kShrinkThreads)
shrink_kernel(LayerPtrs ptrs, int layer0, int* __restrict__ idx_all, int* __restrict__ rank_all,
              const int* __restrict__ count, const int* __restrict__ held, int Bt, int Hkv, int L, int ws,
              int idx_stride /* Blc */, int row_stride, int vec_per_row, size_t layer_idx_stride /* Bt*Hkv*Blc */) {
  extern __shared__ int src_map[];
  __shared__ int sm_a[33], sm_b[33];
  const int layer = layer0 + blockIdx.y;
  const int bh = blockIdx.x, b = bh / Hkv;
  const int have = held[b * L + layer];
  const int want = min(count[b * L + layer], have);
  if (want == have) return;                                  // uniform across the block
  int* idx = idx_all + layer * layer_idx_stride + (size_t)bh * idx_stride;
  int* rank = rank_all + layer * layer_idx_stride + (size_t)bh * idx_stride;
  const int tid = threadIdx.x;
  const int chunk = (have + kShrinkThreads - 1) / kShrinkThreads;
  const int j0 = min(have, tid * chunk), j1 = min(have, j0 + chunk);
  int mine = 0;
  for (int j = j0; j < j1; ++j) mine += (rank[j] < want);
  int before, total;
  {
    const int lane = tid & 31, warp = tid >> 5;
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
    if (lane == 31) sm_a[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      const int w = sm_a[lane];
      int s = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, s, o); if (lane >= o) s += t; }
      sm_b[lane] = s - w;
      if (lane == 31) sm_b[32] = s;
    }
    __syncthreads();
    before = sm_b[warp] + inc - mine;
    total = sm_b[32];                     // == want: ranks are a permutation of 0..have-1
  }
  {
    int o = before;
    for (int j = j0; j < j1; ++j) if (rank[j] < want) src_map[o++] = j;
  }
  __syncthreads();
  // 1) kept positions and ranks
  for (int base = 0; base < total; base += kShrinkThreads) {
    const int d = base + tid;
    int vi = 0, vr = 0;
    if (d < total) { const int sidx = src_map[d]; vi = idx[sidx]; vr = rank[sidx]; }
    __syncthreads();
    if (d < total) { idx[d] = vi; rank[d] = vr; }
    __syncthreads();
  }
  // 2) rows of K then V
  const int rows_per_iter = kShrinkThreads / vec_per_row;
  const int r_in = tid / vec_per_row, c = tid % vec_per_row;
  for (int t = 0; t < 2; ++t) {
    uint4* buf = reinterpret_cast<uint4*>(t == 0 ? ptrs.kb[layer] : ptrs.vb[layer]) + (size_t)bh * row_stride * vec_per_row;
    for (int base = 0; base < total + ws; base += rows_per_iter) {
      const int d = base + r_in;
      uint4 val = make_uint4(0, 0, 0, 0);
      const bool ok = d < total + ws;
      if (ok) {
        const int from = d < total ? src_map[d] : have + (d - total);
        val = buf[(size_t)from * vec_per_row + c];
      }
      __syncthreads();
      if (ok) buf[(size_t)d * vec_per_row + c] = val;
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
