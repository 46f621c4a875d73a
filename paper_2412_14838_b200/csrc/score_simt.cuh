// Window scoring (Eq. 1-2, Algorithm 1's scoring line) on plain CUDA cores: one thread per
// window-query row.  Two sweeps over the keys, because a token's score needs every row's softmax
// normaliser: sweep 1 gathers (max, sum) per row, sweep 2 emits sum_rows exp(logit - lse_row).
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kSimtTileKeys = 16;

// Partial softmax statistics of one row over one key range, in the base-2 domain:
// x = running max of t = logit * log2(e)/sqrt(D); y = sum of 2^(t - x).
template <int D>
__global__ void __launch_bounds__(256)
score_stats_simt(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k, float2* __restrict__ stats,
                 Shape s, int keys_per_split, int n_split, int m_stride) {
  __shared__ __align__(16) float ks[kSimtTileKeys][D];
  const int bh = blockIdx.y, b = bh / s.Hkv, h = bh % s.Hkv;
  const int rho = threadIdx.x;
  const bool active = rho < s.M;
  float qr[D];
  {
    const uint16_t* qp = q + ((size_t)(b * s.Hq + h * s.G) * s.ws + (active ? rho : 0)) * D;
#pragma unroll
    for (int d = 0; d < D; ++d) qr[d] = bf16_bits_to_float(qp[d]);
  }
  const int limit = s.P + (rho % s.ws);               // last key this row can see
  const float scale2 = kLog2e * rsqrtf((float)D);
  const int k0 = blockIdx.x * keys_per_split;
  const int k1 = min(s.S, k0 + keys_per_split);
  const uint16_t* kp = k + (size_t)bh * s.S * D;
  float mx = -INFINITY, l = 0.f;
  for (int tile = k0; tile < k1; tile += kSimtTileKeys) {
    __syncthreads();
    for (int e = threadIdx.x; e < kSimtTileKeys * D / 2; e += blockDim.x) {
      const int jj = e / (D / 2), d2 = e % (D / 2);
      const int j = tile + jj;
      uint32_t w = 0;
      if (j < k1) w = *reinterpret_cast<const uint32_t*>(kp + (size_t)j * D + 2 * d2);
      ks[jj][2 * d2] = __uint_as_float(w << 16);
      ks[jj][2 * d2 + 1] = __uint_as_float(w & 0xFFFF0000u);
    }
    __syncthreads();
    if (active) {
      for (int jj = 0; jj < kSimtTileKeys; ++jj) {
        const int j = tile + jj;
        if (j >= k1 || j > limit) break;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int d = 0; d < D; d += 4) {
          const float4 kv = *reinterpret_cast<const float4*>(&ks[jj][d]);
          a0 = fmaf(qr[d], kv.x, a0); a1 = fmaf(qr[d + 1], kv.y, a1);
          a2 = fmaf(qr[d + 2], kv.z, a2); a3 = fmaf(qr[d + 3], kv.w, a3);
        }
        const float t = ((a0 + a1) + (a2 + a3)) * scale2;
        if (t > mx) { l = l * fast_exp2(mx - t) + 1.f; mx = t; }
        else        { l += fast_exp2(t - mx); }
      }
    }
  }
  if (active) stats[((size_t)bh * n_split + blockIdx.x) * m_stride + rho] = make_float2(mx, l);
}

// Sweep 2: raw[j] = sum over rows of 2^(t_row,j - lse2_row) for prefix keys j < P.
template <int D>
__global__ void __launch_bounds__(256)
score_emit_simt(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k, const float2* __restrict__ stats,
                float* __restrict__ raw, Shape s, int keys_per_cta, int n_split, int m_stride) {
  __shared__ __align__(16) float ks[kSimtTileKeys][D];
  __shared__ float ps[kSimtTileKeys][257];
  const int bh = blockIdx.y, b = bh / s.Hkv, h = bh % s.Hkv;
  const int rho = threadIdx.x;
  const bool active = rho < s.M;
  float qr[D];
  {
    const uint16_t* qp = q + ((size_t)(b * s.Hq + h * s.G) * s.ws + (active ? rho : 0)) * D;
#pragma unroll
    for (int d = 0; d < D; ++d) qr[d] = bf16_bits_to_float(qp[d]);
  }
  float lse2 = INFINITY;
  if (active) {
    float mt = -INFINITY;
    for (int c = 0; c < n_split; ++c) mt = fmaxf(mt, stats[((size_t)bh * n_split + c) * m_stride + rho].x);
    float lt = 0.f;
    for (int c = 0; c < n_split; ++c) {
      const float2 st = stats[((size_t)bh * n_split + c) * m_stride + rho];
      lt += st.y * fast_exp2(st.x - mt);
    }
    lse2 = mt + log2f(lt);
  }
  const float scale2 = kLog2e * rsqrtf((float)D);
  const int k0 = blockIdx.x * keys_per_cta;
  const int k1 = min(s.P, k0 + keys_per_cta);
  const uint16_t* kp = k + (size_t)bh * s.S * D;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32, nwarps = blockDim.x / 32;
  for (int tile = k0; tile < k1; tile += kSimtTileKeys) {
    __syncthreads();
    for (int e = threadIdx.x; e < kSimtTileKeys * D / 2; e += blockDim.x) {
      const int jj = e / (D / 2), d2 = e % (D / 2);
      const int j = tile + jj;
      uint32_t w = 0;
      if (j < k1) w = *reinterpret_cast<const uint32_t*>(kp + (size_t)j * D + 2 * d2);
      ks[jj][2 * d2] = __uint_as_float(w << 16);
      ks[jj][2 * d2 + 1] = __uint_as_float(w & 0xFFFF0000u);
    }
    __syncthreads();
    for (int jj = 0; jj < kSimtTileKeys; ++jj) {
      float p = 0.f;
      if (active) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int d = 0; d < D; d += 4) {
          const float4 kv = *reinterpret_cast<const float4*>(&ks[jj][d]);
          a0 = fmaf(qr[d], kv.x, a0); a1 = fmaf(qr[d + 1], kv.y, a1);
          a2 = fmaf(qr[d + 2], kv.z, a2); a3 = fmaf(qr[d + 3], kv.w, a3);
        }
        p = fast_exp2(((a0 + a1) + (a2 + a3)) * scale2 - lse2);
      }
      ps[jj][rho] = p;
    }
    __syncthreads();
    for (int jj = warp; jj < kSimtTileKeys; jj += nwarps) {
      float acc = 0.f;
      for (int r = lane; r < (int)blockDim.x; r += 32) acc += ps[jj][r];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
      const int j = tile + jj;
      if (lane == 0 && j < k1) raw[(size_t)bh * s.P + j] = acc;
    }
  }
}

// Eq. 2's pooling: stride-1 max over an odd window, neighbours outside [0, P) ignored.
__global__ void maxpool_kernel(const float* __restrict__ raw, float* __restrict__ score,
                               float* __restrict__ copy_out, int P, int half, size_t total) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int j = (int)(e % P);
  const float* row = raw + (e - j);
  float v = row[j];
  for (int o = 1; o <= half; ++o) {
    if (j - o >= 0) v = fmaxf(v, row[j - o]);
    if (j + o < P) v = fmaxf(v, row[j + o]);
  }
  score[e] = v;
  if (copy_out) copy_out[e] = v;
}

}  // namespace dkv
