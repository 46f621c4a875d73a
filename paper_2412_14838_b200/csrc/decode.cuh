// Decoding over the compressed cache (Section 4.3: the decoding phase is the model's own attention, Eq. 1,
// run over what the prefill phase kept).  After Algorithm 1 every layer holds, per head, count_i kept rows
// followed by the ws window rows in a fixed-stride buffer, and count_i differs from layer to layer: the
// lengths are read from the device-side counts, nothing comes back to the host.
//
// One launch covers a range of layers.  Work item = (layer, sample, KV head), split along the rows into
// `splits` thread blocks (the buffers of one layer are only a few MB, so one block per head would leave the
// GPU idle).  A block streams its rows of K and V once: every warp takes rows w, w+8, ..., each lane holding
// D/32 of a row's elements, scores them against the G*nq queries of the head group (in chunks of four, dot
// products completed by warp shuffles), and keeps a running (max, sum, weighted value sum) per query.  Partial
// results go to a scratch array; the block that finishes last for a head (a counter per head) merges the
// partials in split order, so the result does not depend on the order in which blocks finish.
// HBM-bound: the bytes that must move are the valid K and V rows, once.
#pragma once
#include "common.cuh"

namespace dkv {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecQT = 4;          // queries scored together
constexpr int kDecRows = 4;        // rows a warp has in flight

constexpr int kDecMaxSplits = 64; // thread blocks that may share a head
constexpr int kDecMaxLayers = 64;  // layers per launch (the pointers travel as a kernel argument)

struct DecodePtrs {                // per-layer device pointers, indexed by layer - layer0
  const void* q[kDecMaxLayers];
  const void* kb[kDecMaxLayers];
  const void* vb[kDecMaxLayers];
  float* out[kDecMaxLayers];
};

template <int DPL> struct RowFrag;
template <> struct RowFrag<4> {    // D = 128: four bf16 per lane
  uint2 raw;
  __device__ __forceinline__ void load(const uint16_t* row, int lane) { raw = *reinterpret_cast<const uint2*>(row + lane * 4); }
  __device__ __forceinline__ void to_float(float* f) const {
    f[0] = __uint_as_float(raw.x << 16); f[1] = __uint_as_float(raw.x & 0xFFFF0000u);
    f[2] = __uint_as_float(raw.y << 16); f[3] = __uint_as_float(raw.y & 0xFFFF0000u);
  }
};
template <> struct RowFrag<2> {    // D = 64: two bf16 per lane
  uint32_t raw;
  __device__ __forceinline__ void load(const uint16_t* row, int lane) { raw = *reinterpret_cast<const uint32_t*>(row + lane * 2); }
  __device__ __forceinline__ void to_float(float* f) const {
    f[0] = __uint_as_float(raw << 16); f[1] = __uint_as_float(raw & 0xFFFF0000u);
  }
};

// q_dec [Bt, Hq, nq, D] bf16; kb, vb [Bt, Hkv, row_stride, D] bf16; out [Bt, Hq, nq, D] fp32.
// held [Bt][L]: kept rows of every layer; valid rows = held + ws.
// scratch: [layers][Bt*Hkv][splits][GQ][D + 2] floats (value sums, then max and sum); tickets: [layers][Bt*Hkv],
// zero before the first launch and left at zero by every launch.
// grid (splits, Bt*Hkv, layers).
template <int D>
__global__ void __launch_bounds__(kDecThreads)
decode_attend_kernel(DecodePtrs ptrs, int layer0, const int* __restrict__ held, int Hkv, int G, int nq, int L, int ws,
                     int row_stride, float scale2, float* __restrict__ scratch, unsigned int* __restrict__ tickets) {
  constexpr int DPL = D / 32;
  __shared__ float q_s[kDecQT][D];
  __shared__ float part_s[kDecWarps][kDecQT][D + 2];
  __shared__ int last_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int splits = gridDim.x, split = blockIdx.x, bh = blockIdx.y, lz = blockIdx.z, layer = layer0 + lz;
  const int b = bh / Hkv, h = bh % Hkv, BH = gridDim.y, GQ = G * nq;
  const int len = held[b * L + layer] + ws;
  const int rps = (len + splits - 1) / splits;
  const int r0 = split * rps, r1 = min(len, r0 + rps);
  const uint16_t* kbase = reinterpret_cast<const uint16_t*>(ptrs.kb[lz]) + (size_t)bh * row_stride * D;
  const uint16_t* vbase = reinterpret_cast<const uint16_t*>(ptrs.vb[lz]) + (size_t)bh * row_stride * D;
  const uint16_t* qbase = reinterpret_cast<const uint16_t*>(ptrs.q[lz]) + (size_t)(b * Hkv + h) * GQ * D;   // head group h: GQ rows
  float* my_scratch = scratch + ((size_t)(lz * BH + bh) * splits + split) * GQ * (D + 2);

  for (int c0 = 0; c0 < GQ; c0 += kDecQT) {
    __syncthreads();
    for (int e = tid; e < kDecQT * D; e += kDecThreads) {
      const int qi = e / D, d = e % D;
      q_s[qi][d] = c0 + qi < GQ ? bf16_bits_to_float(qbase[(size_t)(c0 + qi) * D + d]) : 0.f;
    }
    __syncthreads();
    float qr[kDecQT][DPL];
#pragma unroll
    for (int qi = 0; qi < kDecQT; ++qi)
#pragma unroll
      for (int d = 0; d < DPL; ++d) qr[qi][d] = q_s[qi][lane * DPL + d] * scale2;
    float m[kDecQT], l[kDecQT], acc[kDecQT][DPL];
#pragma unroll
    for (int qi = 0; qi < kDecQT; ++qi) {
      m[qi] = -INFINITY; l[qi] = 0.f;
#pragma unroll
      for (int d = 0; d < DPL; ++d) acc[qi][d] = 0.f;
    }
    // the rows of the next round are requested before the current round is worked on
    RowFrag<DPL> kn[kDecRows], vn[kDecRows];
#pragma unroll
    for (int j = 0; j < kDecRows; ++j) {
      const int row = r0 + warp + j * kDecWarps;
      if (row < r1) { kn[j].load(kbase + (size_t)row * D, lane); vn[j].load(vbase + (size_t)row * D, lane); }
    }
    for (int r = r0 + warp; r < r1; r += kDecWarps * kDecRows) {
      RowFrag<DPL> kf[kDecRows], vf[kDecRows];
#pragma unroll
      for (int j = 0; j < kDecRows; ++j) { kf[j] = kn[j]; vf[j] = vn[j]; }
#pragma unroll
      for (int j = 0; j < kDecRows; ++j) {
        const int row = r + kDecWarps * kDecRows + j * kDecWarps;
        if (row < r1) { kn[j].load(kbase + (size_t)row * D, lane); vn[j].load(vbase + (size_t)row * D, lane); }
      }
      float s[kDecRows][kDecQT];
#pragma unroll
      for (int j = 0; j < kDecRows; ++j) {
        float kk[DPL];
        kf[j].to_float(kk);
#pragma unroll
        for (int qi = 0; qi < kDecQT; ++qi) {
          float a = 0.f;
#pragma unroll
          for (int d = 0; d < DPL; ++d) a = fmaf(qr[qi][d], kk[d], a);
          s[j][qi] = a;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int j = 0; j < kDecRows; ++j)
#pragma unroll
          for (int qi = 0; qi < kDecQT; ++qi) s[j][qi] += __shfl_xor_sync(0xFFFFFFFFu, s[j][qi], o);
#pragma unroll
      for (int qi = 0; qi < kDecQT; ++qi) {
        float mn = m[qi];
#pragma unroll
        for (int j = 0; j < kDecRows; ++j) if (r + j * kDecWarps < r1) mn = fmaxf(mn, s[j][qi]);
        const float corr = fast_exp2(m[qi] - mn);              // 0 on the first rows (m = -inf)
        m[qi] = mn;
        l[qi] *= corr;
#pragma unroll
        for (int d = 0; d < DPL; ++d) acc[qi][d] *= corr;
#pragma unroll
        for (int j = 0; j < kDecRows; ++j) {
          if (r + j * kDecWarps < r1) {
            const float p = fast_exp2(s[j][qi] - mn);
            float vv[DPL];
            vf[j].to_float(vv);
            l[qi] += p;
#pragma unroll
            for (int d = 0; d < DPL; ++d) acc[qi][d] = fmaf(p, vv[d], acc[qi][d]);
          }
        }
      }
    }
    // the block's partial result: the eight warps merged in warp order
#pragma unroll
    for (int qi = 0; qi < kDecQT; ++qi) {
#pragma unroll
      for (int d = 0; d < DPL; ++d) part_s[warp][qi][lane * DPL + d] = acc[qi][d];
      if (lane == 0) { part_s[warp][qi][D] = m[qi]; part_s[warp][qi][D + 1] = l[qi]; }
    }
    __syncthreads();
    for (int e = tid; e < kDecQT * (D + 2); e += kDecThreads) {
      const int qi = e / (D + 2), d = e % (D + 2);
      if (c0 + qi >= GQ) continue;
      float mm = -INFINITY;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) mm = fmaxf(mm, part_s[w][qi][D]);
      float v = 0.f;
      if (d == D) v = mm;
      else if (mm > -INFINITY) {
        const int src = d < D ? d : D + 1;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) v += part_s[w][qi][src] * fast_exp2(part_s[w][qi][D] - mm);
      }
      my_scratch[(size_t)(c0 + qi) * (D + 2) + d] = v;
    }
  }
  // the block that arrives last for this head merges the splits (in split order)
  __threadfence();
  __syncthreads();
  if (tid == 0) last_s = atomicAdd(&tickets[lz * BH + bh], 1u) == (unsigned int)(splits - 1);
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  const float* head_scratch = scratch + (size_t)(lz * BH + bh) * splits * GQ * (D + 2);
  float* out = ptrs.out[lz] + (size_t)(b * Hkv + h) * GQ * D;
  float* wgt_s = &part_s[0][0][0];                      // [splits][kDecQT] weights, then [kDecQT] denominators
  for (int c0 = 0; c0 < GQ; c0 += kDecQT) {
    __syncthreads();
    // weight of every split for the chunk's queries: 2^(max of the split - overall max)
    if (tid < kDecQT * 32) {
      const int qi = tid >> 5, gq = c0 + qi;
      float mm = -INFINITY;
      if (gq < GQ) for (int sp = lane; sp < splits; sp += 32) mm = fmaxf(mm, head_scratch[((size_t)sp * GQ + gq) * (D + 2) + D]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xFFFFFFFFu, mm, o));
      float den = 0.f;
      if (gq < GQ) for (int sp = lane; sp < splits; sp += 32) {
        const float* pr = head_scratch + ((size_t)sp * GQ + gq) * (D + 2);
        const float wgt = fast_exp2(pr[D] - mm);
        wgt_s[sp * kDecQT + qi] = wgt;
        den = fmaf(pr[D + 1], wgt, den);
      }
      // the denominators are added in a fixed order: lane partial sums, then a butterfly
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xFFFFFFFFu, den, o);
      if (lane == 0) wgt_s[kDecMaxSplits * kDecQT + qi] = den;
    }
    __syncthreads();
    for (int e = tid; e < kDecQT * D; e += kDecThreads) {
      const int qi = e / D, d = e % D, gq = c0 + qi;
      if (gq >= GQ) continue;
      float num = 0.f;
#pragma unroll 8
      for (int sp = 0; sp < splits; ++sp) num = fmaf(head_scratch[((size_t)sp * GQ + gq) * (D + 2) + d], wgt_s[sp * kDecQT + qi], num);
      out[(size_t)gq * D + d] = num / wgt_s[kDecMaxSplits * kDecQT + qi];
    }
  }
  if (tid == 0) tickets[lz * BH + bh] = 0;
}

// ------------------------------------------------------------------------------------------------------
// Fixed-pattern budgets (the methods the paper compares with, Section 5.1 "Baselines", as policies only).

// count[b][i] = min(count[b][i], schedule_i); schedule: policy 0 = N in every layer, policy 1 = the pyramid
// N + floor(N (L-1-2i) / (2 (L-1))) (floor towards minus infinity; N when L = 1).
__global__ void policy_counts_kernel(int* __restrict__ count, int* __restrict__ counts_out, int Bt, int L, int N, int policy) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= Bt * L) return;
  const int i = e % L;
  long long want = N;
  if (policy == 1 && L > 1) {
    const long long num = (long long)N * (L - 1 - 2 * i), den = 2ll * (L - 1);
    want = N + (num >= 0 ? num / den : -((-num + den - 1) / den));
  }
  const int c = count[e];
  const int v = want < c ? (int)want : c;
  count[e] = v;
  if (counts_out) counts_out[e] = v;
}

// Kept positions without scores: the first n_sink and the last n_recent prefix positions of every head,
// ascending (sinks plus a window of the most recent tokens).  idx [Bt*Hkv][idx_stride]; count[b][layer] = n.
__global__ void positions_kernel(int* __restrict__ idx, int* __restrict__ count, int P, int idx_stride, int n_sink,
                                 int first_recent, int n, int Hkv, int L, int layer) {
  const int bh = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e == 0 && bh % Hkv == 0) count[(bh / Hkv) * L + layer] = n;
  if (e >= n) return;
  idx[(size_t)bh * idx_stride + e] = e < n_sink ? e : first_recent + (e - n_sink);
}

}  // namespace dkv
