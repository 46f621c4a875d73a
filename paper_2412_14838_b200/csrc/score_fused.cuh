// Window scoring (Eq. 1-2) with the keys read ONCE: both sweeps of score_tc.cuh run on key tiles that
// stay in shared memory in between.
//
// A layer is worked through in rounds of whole heads.  In a round every active CTA owns one pair of
// adjacent 128-key tiles of one head (so a head of up to 2 x #CTAs tiles fits one round).  The CTA loads
// its pair by TMA, runs sweep 1 on it (per-row softmax statistics, published to global memory), and keeps
// the tiles.  When all pairs of the head have published, the last CTA to arrive merges them into the
// head's log-sum-exp per window row and raises the head's flag; every CTA of the head then runs sweep 2
// (per-key sums) on the tiles it still holds, trades the three raw scores on each side of its range with
// its neighbours through global memory, max-pools and writes the scores.  Rounds are software-pipelined
// by one: sweep 1 of round r is issued before sweep 2 of round r-1, which hides the wait for the flag.
//
// Waiting on other CTAs needs all CTAs of the grid resident at once: the grid is never larger than the
// number of SMs and every wait is bounded, so a violated assumption ends in an error status, not a hang.
// Counters and flags are never cleared: each launch brings a fresh `epoch` and compares against it.
//
// Applies when the window rows fit one MMA block (ws*G <= 128) and a head has at most 2 x grid tiles;
// other shapes use the two-sweep kernel.
#pragma once
#include "score_tc.cuh"

namespace dkv {
namespace tc {

struct FusedParams {
  int S, P, ws, M, D, heads, half, tph, nq16;
  int pp;                  // tile pairs per head, ceil(tph / 2)
  int hpr;                 // heads per round, floor(grid / pp) >= 1
  int n_rounds;            // ceil(heads / hpr)
  float scale2;
  uint32_t idesc_stats, idesc_emit;
  unsigned int epoch;      // launch number on these flag arrays, >= 1
  float2* part;            // [heads][pp][128] sweep-1 statistics of every pair
  float* lse;              // [heads][128] merged log2-sum-exp per window row
  unsigned int* done;      // [heads] pairs that have published (accumulates over launches)
  unsigned int* ready;     // [heads] epoch of the last launch whose lse is complete
  unsigned int* halo_flag; // [heads][pp] epoch of the last launch whose edge scores are written
  float* halo_val;         // [heads][pp][2 * kHaloMax] first and last raw scores of the pair's range
  float* scores;           // [heads][P]
  float* copy_out;
  int* status;
};

constexpr int kHaloMax = 128;   // pooling half-width supported (pool_kernel <= 255)
constexpr int kFusedSmemBytes = 1024 + kQRegion + kKRegion + kMiscBytes + kRawBytes + 256;

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned int* p, unsigned int v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait for *p >= want (monotone counters).
__device__ __forceinline__ void flag_wait(const unsigned int* p, unsigned int want, volatile int* abort_flag, int* status,
                                          int code) {
  if (*abort_flag) return;
  const long long t0 = clock64();
  while ((int)(ld_acquire(p) - want) < 0) {
    if (*abort_flag) return;
    if (clock64() - t0 > kWaitCycles) { *abort_flag = 1; atomicCAS(status, 0, code); return; }
  }
}

struct RoundWork { bool active; int head, pair, tile0, ntiles; };

__device__ __forceinline__ RoundWork round_work(const FusedParams& p, int r, int cta) {
  RoundWork w;
  const int h0 = r * p.hpr;
  const int nh = min(p.hpr, p.heads - h0);
  w.active = r < p.n_rounds && cta < nh * p.pp;
  w.head = h0 + cta / p.pp;
  w.pair = cta % p.pp;
  w.tile0 = 2 * w.pair;
  w.ntiles = min(2, p.tph - w.tile0);
  return w;
}

__global__ void __launch_bounds__(kThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                   const __grid_constant__ FusedParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_smem = smem;                              // [2 buffers][half][128 rows][128 B]
  uint8_t* k_smem = smem + kQRegion;                   // [4 slots][half][128 rows][128 B]
  float* lse_s = reinterpret_cast<float*>(k_smem + kKRegion);          // [128]
  float2* merge_s = reinterpret_cast<float2*>(lse_s + 256);            // [3][256]
  float* raw_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(lse_s) + kMiscBytes);   // [part][stride]
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(raw_s) + kRawBytes);
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  __shared__ int last_s;
  const uint32_t bar0 = smem_u32(bars);
  auto FULL = [&](int s) { return bar0 + 8u * s; };               // K slot filled
  auto EMPTY = [&](int s) { return bar0 + 8u * (4 + s); };        // K slot (and the round's Q buffer) read for the last time
  auto TFULL = [&](int t) { return bar0 + 8u * (8 + t); };
  auto TEMPTY = [&](int t) { return bar0 + 8u * (10 + t); };
  auto QFULL = [&](int b) { return bar0 + 8u * (12 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_s;
  const int halves = p.D / 64;
  const int R = p.n_rounds;

  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < 4; ++s) { mbar_init(FULL(s), 1); mbar_init(EMPTY(s), 1); }
    for (int t = 0; t < 2; ++t) { mbar_init(TFULL(t), 1); mbar_init(TEMPTY(t), 16); mbar_init(QFULL(t), 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int uses[4] = {0, 0, 0, 0};
      for (int r = 0; r < R; ++r) {
        const RoundWork w = round_work(p, r, blockIdx.x);
        if (!w.active) continue;
        const int qb = r & 1;
        // the two slots and the query buffer of this parity were last read by sweep 2 of round r-2
        for (int i = 0; i < 2; ++i) {
          const int s = qb * 2 + i;
          mbar_wait(EMPTY(s), (uses[s] & 1) ^ 1, abort_flag, p.status, 201);
        }
        if (*abort_flag) break;
        mbar_expect_tx(QFULL(qb), (uint32_t)halves * kHalfBytes);
        for (int h = 0; h < halves; ++h)
          tma_load_3d(smem_u32(q_smem + qb * (2 * kHalfBytes) + h * kHalfBytes), &q_map, QFULL(qb), 64 * h, 0, w.head);
        for (int i = 0; i < 2; ++i) {
          const int s = qb * 2 + i;
          if (i < w.ntiles) {
            mbar_expect_tx(FULL(s), (uint32_t)halves * kHalfBytes);
            for (int h = 0; h < halves; ++h)
              tma_load_3d(smem_u32(k_smem + (s * 2 + h) * kHalfBytes), &k_map, FULL(s), 64 * h, (w.tile0 + i) * kTileKeys, w.head);
            ++uses[s];
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int uses[4] = {0, 0, 0, 0}, quses[2] = {0, 0};
      int tile = 0;
      const int ksteps = p.D / 16;
      for (int r = 0; r <= R; ++r) {
        const RoundWork w = round_work(p, r, blockIdx.x);
        if (w.active) {                                            // sweep 1 of round r
          const int qb = r & 1;
          mbar_wait(QFULL(qb), quses[qb] & 1, abort_flag, p.status, 203);
          ++quses[qb];
          for (int i = 0; i < w.ntiles; ++i, ++tile) {
            const int s = qb * 2 + i, t = tile & 1, nt = tile >> 1;
            mbar_wait(FULL(s), uses[s] & 1, abort_flag, p.status, 204);
            ++uses[s];
            mbar_wait(TEMPTY(t), (nt & 1) ^ 1, abort_flag, p.status, 205);
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(t * kStageCols);
            for (int ks = 0; ks < ksteps; ++ks) {
              const uint64_t a = smem_desc(smem_u32(q_smem + qb * (2 * kHalfBytes) + (ks >> 2) * kHalfBytes) + (ks & 3) * 32);
              const uint64_t b = smem_desc(smem_u32(k_smem + (s * 2 + (ks >> 2)) * kHalfBytes) + (ks & 3) * 32);
              tc_mma(d_tmem, a, b, p.idesc_stats, ks > 0);
            }
            tc_commit(TFULL(t));
          }
        }
        const RoundWork v = round_work(p, r - 1, blockIdx.x);
        if (r >= 1 && v.active) {                                  // sweep 2 of round r-1, on the tiles still held
          const int qb = (r - 1) & 1;
          for (int i = 0; i < v.ntiles; ++i, ++tile) {
            const int s = qb * 2 + i, t = tile & 1, nt = tile >> 1;
            mbar_wait(TEMPTY(t), (nt & 1) ^ 1, abort_flag, p.status, 206);
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(t * kStageCols);
            for (int ks = 0; ks < ksteps; ++ks) {
              const uint64_t a = smem_desc(smem_u32(k_smem + (s * 2 + (ks >> 2)) * kHalfBytes) + (ks & 3) * 32);
              const uint64_t b = smem_desc(smem_u32(q_smem + qb * (2 * kHalfBytes) + (ks >> 2) * kHalfBytes) + (ks & 3) * 32);
              tc_mma(d_tmem, a, b, p.idesc_emit, ks > 0);
            }
            tc_commit(EMPTY(s));
            tc_commit(TFULL(t));
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const int part = (warp - 2) >> 2;          // which quarter of the accumulator columns
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    const int row = quad * 32 + lane;          // TMEM lane = window row (sweep 1) or key within the tile (sweep 2)
    const int sid = threadIdx.x - 64;          // 0..511 among the softmax threads
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const int raw_stride = kMaxSegTiles * kTileKeys;
    int tile = 0;
    for (int r = 0; r <= R; ++r) {
      const RoundWork w = round_work(p, r, blockIdx.x);
      if (w.active) {
        // ---------------------------------------------------------------- sweep 1: (max, sum) per window row
        float mx = -INFINITY, sum = 0.f;
        const int limit = p.P + (row % p.ws);
        for (int i = 0; i < w.ntiles; ++i, ++tile) {
          const int t = tile & 1, nt = tile >> 1;
          mbar_wait(TFULL(t), nt & 1, abort_flag, p.status, 207);
          tc_fence_after();
          float xv[32];
          tc_ld32(lane_addr + (uint32_t)(t * kStageCols + part * 32), xv);
          tc_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(TEMPTY(t));
          const int kb = (w.tile0 + i) * kTileKeys + part * 32;
          if (kb + 31 > p.P) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (kb + e > limit) xv[e] = -INFINITY;
          }
          float cm = fmax3(xv[0], xv[1], xv[2]);
#pragma unroll
          for (int e = 3; e < 31; e += 2) cm = fmax3(cm, xv[e], xv[e + 1]);
          cm = fmaxf(cm, xv[31]);
          if (cm == -INFINITY) continue;
          const float mnew = fmaxf(mx, cm * p.scale2);
          if (mnew > mx) { sum *= fast_exp2(mx - mnew); mx = mnew; }
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
          const float neg = -mx;
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            s0 += fast_exp2(fmaf(xv[e], p.scale2, neg));
            s1 += fast_exp2(fmaf(xv[e + 1], p.scale2, neg));
            s2 += fast_exp2(fmaf(xv[e + 2], p.scale2, neg));
            s3 += fast_exp2(fmaf(xv[e + 3], p.scale2, neg));
          }
          sum += (s0 + s1) + (s2 + s3);
        }
        if (part > 0) merge_s[(part - 1) * 256 + row] = make_float2(mx, sum);
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (part == 0) {
          float m = mx;
#pragma unroll
          for (int q = 0; q < 3; ++q) m = fmaxf(m, merge_s[q * 256 + row].x);
          float l = 0.f;
          if (m > -INFINITY) {
            l = sum * fast_exp2(mx - m);
#pragma unroll
            for (int q = 0; q < 3; ++q) { const float2 o = merge_s[q * 256 + row]; l += o.y * fast_exp2(o.x - m); }
          }
          p.part[((size_t)w.head * p.pp + w.pair) * 128 + row] = make_float2(m, l);
          __threadfence();
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (sid == 0) last_s = (atomicAdd(&p.done[w.head], 1u) + 1u == p.epoch * (unsigned int)p.pp);
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (last_s) {
          // last pair of the head to arrive: merge all pairs' statistics, four threads per window row
          __threadfence();
          const int rr = sid >> 2, qq = sid & 3;
          float m = -INFINITY, l = 0.f;
          const float2* src = p.part + (size_t)w.head * p.pp * 128 + rr;
          for (int c = qq; c < p.pp; c += 4) {
            const float2 st = __ldcg(src + (size_t)c * 128);
            const float mn = fmaxf(m, st.x);
            if (mn > -INFINITY) { l = l * fast_exp2(m - mn) + st.y * fast_exp2(st.x - mn); m = mn; }
          }
#pragma unroll
          for (int o = 1; o < 4; o <<= 1) {
            const float om = __shfl_xor_sync(0xFFFFFFFFu, m, o), ol = __shfl_xor_sync(0xFFFFFFFFu, l, o);
            const float mn = fmaxf(m, om);
            // the same expression on both sides of the exchange, so all four lanes end with the same bits
            const float a = (m >= om) ? l : ol, am = (m >= om) ? m : om, b = (m >= om) ? ol : l, bm = (m >= om) ? om : m;
            l = (mn > -INFINITY) ? a * fast_exp2(am - mn) + b * fast_exp2(bm - mn) : 0.f;
            m = mn;
          }
          if (qq == 0) p.lse[(size_t)w.head * 128 + rr] = (rr < p.M) ? m + log2f(l) : INFINITY;
          __threadfence();
          asm volatile("bar.sync 1, 512;" ::: "memory");
          if (sid == 0) st_release(&p.ready[w.head], p.epoch);
        }
      }
      const RoundWork v = round_work(p, r - 1, blockIdx.x);
      if (r >= 1 && v.active) {
        // ---------------------------------------------------------------- sweep 2: one thread per key
        if (sid == 0) flag_wait(&p.ready[v.head], p.epoch, abort_flag, p.status, 208);
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (sid < 128) lse_s[sid] = __ldcg(&p.lse[(size_t)v.head * 128 + sid]);
        asm volatile("bar.sync 1, 512;" ::: "memory");
        const int nchunk = p.nq16 >> 4;
        float* my_raw = raw_s + part * raw_stride;
        for (int i = 0; i < v.ntiles; ++i, ++tile) {
          const int t = tile & 1, nt = tile >> 1;
          mbar_wait(TFULL(t), nt & 1, abort_flag, p.status, 209);
          tc_fence_after();
          const uint32_t taddr = lane_addr + (uint32_t)(t * kStageCols);
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
          const int c0 = part, c1 = part + 4;              // nq16 <= 128: at most eight 16-column chunks
          float x0[16], x1[16];
          if (c0 < nchunk) tc_ld16(taddr + c0 * 16, x0);
          if (c1 < nchunk) tc_ld16(taddr + c1 * 16, x1);
          tc_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(TEMPTY(t));
          if (c0 < nchunk) {
#pragma unroll
            for (int e = 0; e < 16; e += 4) {
              const float4 ls = *reinterpret_cast<const float4*>(&lse_s[c0 * 16 + e]);
              a0 += fast_exp2(fmaf(x0[e], p.scale2, -ls.x));
              a1 += fast_exp2(fmaf(x0[e + 1], p.scale2, -ls.y));
              a2 += fast_exp2(fmaf(x0[e + 2], p.scale2, -ls.z));
              a3 += fast_exp2(fmaf(x0[e + 3], p.scale2, -ls.w));
            }
          }
          if (c1 < nchunk) {
#pragma unroll
            for (int e = 0; e < 16; e += 4) {
              const float4 ls = *reinterpret_cast<const float4*>(&lse_s[c1 * 16 + e]);
              a0 += fast_exp2(fmaf(x1[e], p.scale2, -ls.x));
              a1 += fast_exp2(fmaf(x1[e + 1], p.scale2, -ls.y));
              a2 += fast_exp2(fmaf(x1[e + 2], p.scale2, -ls.z));
              a3 += fast_exp2(fmaf(x1[e + 3], p.scale2, -ls.w));
            }
          }
          my_raw[kHaloMax + i * kTileKeys + row] = (a0 + a1) + (a2 + a3);
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        // raw score of key k0 + x sits at raw_s[kHaloMax + x]; add up the four column parts in a fixed order
        const int k0 = v.tile0 * kTileKeys, nk = v.ntiles * kTileKeys;
        for (int x = sid; x < nk; x += kSoftmaxThreads) {
          float s = raw_s[kHaloMax + x];
#pragma unroll
          for (int q = 1; q < kParts; ++q) s += raw_s[q * raw_stride + kHaloMax + x];
          raw_s[kHaloMax + x] = s;
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        // publish the edge scores, then fetch the neighbours' (they publish before they wait, so this ends)
        const int H = p.half;
        float* hv = p.halo_val + ((size_t)v.head * p.pp + v.pair) * (2 * kHaloMax);
        if (sid < H) { hv[sid] = raw_s[kHaloMax + sid]; hv[kHaloMax + sid] = raw_s[kHaloMax + nk - H + sid]; }
        __threadfence();
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (sid == 0) st_release(&p.halo_flag[(size_t)v.head * p.pp + v.pair], p.epoch);
        const bool has_left = v.pair > 0, has_right = v.pair + 1 < p.pp;
        if (sid == 0 && has_left) flag_wait(&p.halo_flag[(size_t)v.head * p.pp + v.pair - 1], p.epoch, abort_flag, p.status, 210);
        if (sid == 32 && has_right) flag_wait(&p.halo_flag[(size_t)v.head * p.pp + v.pair + 1], p.epoch, abort_flag, p.status, 211);
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (sid < H) {
          if (has_left) raw_s[kHaloMax - H + sid] = __ldcg(hv - 2 * kHaloMax + kHaloMax + sid);    // left pair's last H
          if (has_right) raw_s[kHaloMax + nk + sid] = __ldcg(hv + 2 * kHaloMax + sid);               // right pair's first H
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        // Eq. 2's pooling; neighbours outside [0, P) are ignored
        for (int x = sid; x < nk; x += kSoftmaxThreads) {
          const int o = k0 + x;
          if (o >= p.P) continue;
          float s = raw_s[kHaloMax + x];
          for (int d = 1; d <= H; ++d) {
            if (o - d >= 0) s = fmaxf(s, raw_s[kHaloMax + x - d]);
            if (o + d < p.P) s = fmaxf(s, raw_s[kHaloMax + x + d]);
          }
          const size_t at = (size_t)v.head * p.P + o;
          p.scores[at] = s;
          if (p.copy_out) p.copy_out[at] = s;
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

}  // namespace tc
}  // namespace dkv
