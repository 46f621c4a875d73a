// Window scoring (Eq. 1-2, Algorithm 1's scoring line) on the sm_100a tensor cores.
//
// A token's score needs the softmax normaliser of every window row, which is only known after
// all keys have been seen, so the keys are swept twice:
//   sweep 1 (kStats)  logits = Q_win . K^T, one TMEM lane per window row; every thread keeps the
//                     running (max, sum) of its own row over the CTA's key range;
//   sweep 2 (kEmit)   logits^T = K . Q_win^T, one TMEM lane per KEY; every thread adds up
//                     2^(logit - lse_row) over the rows of its own key, which is the token's score
//                     with no cross-thread reduction; the CTA then max-pools its key range.
// Both sweeps share one pipeline: a TMA producer warp streams 128-key tiles of K (bf16, 128-byte
// swizzle) through a shared-memory ring; two threads in different warps issue tcgen05.mma (tile i goes to
// issuer i mod 2) into TMEM accumulator stages; sixteen warps read the accumulators back with tcgen05.ld
// in two groups that alternate tiles, each warp one TMEM lane quadrant x half the columns.
// Work is split evenly: the flattened (head, key tile) space for sweep 1 and the flattened
// (head, prefix position) space for sweep 2 are cut into one contiguous slice per CTA.
// One launch runs up to two jobs back to back through the same pipeline (sweep 2 of one layer, then
// sweep 1 of the next), so the fixed cost of a launch is paid once per layer.
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace dkv {
namespace tc {

constexpr int kTileKeys = 128;
constexpr int kMmaWarp2 = 18;
constexpr int kStages = 4;                 // K tiles in flight
constexpr int kThreads = 608;              // warp 0: TMA, warps 1 and 18: MMA (even / odd tiles), warps 2..17: softmax
constexpr int kSoftmaxThreads = 512;
constexpr int kParts = 4;                  // softmax warps per TMEM lane quadrant: 2 tile groups x 2 column halves
constexpr int kMaxSegTiles = 16;           // sweep 2: tiles per pooled segment
// TMEM accumulator stages: four of 128 columns when the window rows fit one 128-row block (ws*G <= 128),
// else two of 256.  A softmax group then always has a second accumulator being filled while it reads one.
constexpr int kHalfBytes = 128 * 128;      // one 128-row x 64-column bf16 box
constexpr int kQRegion = 2 * 2 * kHalfBytes;          // up to 256 rows x 128 columns
constexpr int kKRegion = kStages * 2 * kHalfBytes;    // ring of 128 x 128 tiles
constexpr int kMiscBytes = 1024 /*lse*/ + 3 * 256 * 8 /*merge*/;
constexpr int kRawBytes = 2 * kMaxSegTiles * kTileKeys * 4;   // sweep 2: one partial-sum array per column half
constexpr int kSmemBytes = 1024 /*align*/ + kQRegion + kKRegion + kMiscBytes + kRawBytes + 256 /*barriers*/;
constexpr long long kDefaultWaitCycles = 4000000000ll;  // ~2 s: a wait that long is reported, not spun on
constexpr uint32_t kSuspendNs = 4000;                   // a waiting thread sleeps in the barrier unit, not in a polling loop
constexpr long long kDrainCycles = 2000000ll;           // ~1 ms: wait for own copies / MMAs in flight after an abort

enum Mode { kNone = 0, kStats = 1, kEmit = 2 };

struct Params {
  int S, P, ws, M, D, heads, half;
  int tph;                 // key tiles per head, ceil(S / 128)
  int nq16;                // window rows rounded up to 16 (MMA N of sweep 2)
  int nmblk;               // 128-row blocks of window rows (MMA M blocks of sweep 1)
  int slots;               // partial-statistics slots per head
  int m_stride;            // floats2 per slot
  float scale2;            // log2(e) / sqrt(D)
  uint32_t idesc;          // tcgen05 instruction descriptor of this sweep
  float2* stats;
  float* scores;           // [heads][P] pooled scores (sweep 2)
  float* copy_out;         // optional second copy
  int* status;             // device status words; [0] = first error
  int stats_grid;          // CTAs of the launch that ran sweep 1 for this layer
  int mode;                // kNone: nothing to do
  float out_scale;         // sweep 2: factor on the raw scores before pooling (1, or 1/(ws*G) for the window mean)
  int pool_avg;            // sweep 2: 0 = max-pool, 1 = average over the neighbours that exist
  int nl;                  // layers this job covers (1..kMaxGroup); `heads` counts the heads of all of them
  int hpl;                 // heads per layer
  int back;                // sweep 2: 1 = every CTA walks its slice from the end to the start, so that it begins
                           // with the keys sweep 1 streamed last (those still in L2)
  long long wait_cycles;   // limit of every mbarrier wait, in clock64 ticks
  int retain_tiles;        // sweep 1: the last `retain_tiles` key tiles of a CTA's slice are kept in L2 for sweep 2, which starts
                           // with them; every other key tile of either sweep is marked to be evicted first (0: no marking)
  int withhold_tile;       // test hook: CTA 0 never loads its key tile number `withhold_tile` of this job (-1: off),
                           // so that the wait for it runs out and the timeout path can be exercised
};

constexpr int kMaxGroup = 8;               // layers one job may cover
struct Maps {                              // tensor maps of a job's layers, in storage order
  CUtensorMap q[kMaxGroup], k[kMaxGroup];
  const float* lse[kMaxGroup];             // sweep 2: the caller's natural-log normalisers [heads per layer][M] of each
                                           // layer (then sweep 1 never ran for the job), or null
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"     // may suspend the thread for up to the hint (ns)
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
  return ok != 0;
}
// Bounded wait: true once the barrier's phase is complete; gives up after `limit` clock ticks (false), records the failure (status[0] = the first wait site that
// gave up, status[2] = its CTA) and lets the kernel run to its end: once the CTA's abort flag is up no wait
// blocks, no further copy or MMA is issued, and the CTA drains what it has in flight before it frees its
// tensor memory.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int code,
                                          long long limit) {
  if (mbar_try(bar, parity)) return true;      // the usual case costs one instruction: the control threads share
  if (*abort_flag) return false;               // their schedulers with the softmax warps and every instruction waits its turn
  const long long t0 = clock64();
  while (!mbar_try(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      if (atomicCAS(status, 0, code) == 0) status[2] = (int)blockIdx.x;
      return false;
    }
  }
  return true;
}
// After an abort: wait a short while for something of this CTA's own that is still in flight.  Never records.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try(bar, parity)) if (clock64() - t0 > kDrainCycles) return;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// The same copy with an L2 eviction policy for the lines it brings in.
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The eight k-steps of a 128-dim tile issued as one block: the descriptors of the steps differ in their low words
// only (32 bytes = 2 units per step inside a 64-column half, A_HALF / B_HALF units to the second half), so the
// issuing thread spends two additions per MMA instead of rebuilding two 64-bit descriptors.
template <int A_HALF, int B_HALF>
__device__ __forceinline__ void tc_mma_x8(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
#define DKV_MMA_STEP(OFF, P)                                                                             \
      "add.u32 la, %1, " OFF ";\n\tadd.u32 lb, %2, " OFF ";\n\tmov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\t" \
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, " P ";\n\t"
#define DKV_MMA_STEP2(OFF, P)                                                                            \
      "add.u32 la, %1, %5;\n\tadd.u32 la, la, " OFF ";\n\tadd.u32 lb, %2, %6;\n\tadd.u32 lb, lb, " OFF ";\n\t"    \
      "mov.b64 da, {la, %3};\n\tmov.b64 db, {lb, %3};\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, " P ";\n\t"
  asm volatile(
      "{\n\t.reg .pred pf, pt;\n\t.reg .b64 da, db;\n\t.reg .b32 la, lb;\n\t"
      "setp.ne.b32 pf, 0, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
      DKV_MMA_STEP("0", "pf") DKV_MMA_STEP("2", "pt") DKV_MMA_STEP("4", "pt") DKV_MMA_STEP("6", "pt")
      DKV_MMA_STEP2("0", "pt") DKV_MMA_STEP2("2", "pt") DKV_MMA_STEP2("4", "pt") DKV_MMA_STEP2("6", "pt")
      "}"
      ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "n"(A_HALF), "n"(B_HALF) : "memory");
#undef DKV_MMA_STEP
#undef DKV_MMA_STEP2
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Packed fp32 pairs (one instruction for two lanes of arithmetic): the softmax warps' instruction count is what
// the single-thread producer and issuers compete with for issue slots.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// 2^t for two arguments at once on the FMA and integer pipes instead of the special-function unit: the integer
// part is split off by adding 1.5 * 2^23 (it lands in the low mantissa bits), a quartic takes 2^f on [-0.5, 0.5]
// (largest relative error 2.7e-6, mean 4e-8), and the integer part is added to the result's exponent field.  Arguments
// below -126 count as -126 (2^-126: nothing next to any sum this kernel forms).
__device__ __forceinline__ uint64_t poly_exp2_pair(uint64_t t) {
  float t0, t1;
  unpack2(t, t0, t1);
  const uint64_t tc = pack2(fmaxf(t0, -126.f), fmaxf(t1, -126.f));
  const uint64_t y = add2(tc, pack2(12582912.f, 12582912.f));
  const uint64_t n = add2(y, pack2(-12582912.f, -12582912.f));
  const uint64_t f = fma2(n, pack2(-1.f, -1.f), tc);
  uint64_t p = fma2(f, pack2(0.00957010f, 0.00957010f), pack2(0.05591786f, 0.05591786f));
  p = fma2(p, f, pack2(0.24024744f, 0.24024744f));
  p = fma2(p, f, pack2(0.69312179f, 0.69312179f));
  p = fma2(p, f, pack2(0.99999928f, 0.99999928f));
  float p0, p1, y0, y1;
  unpack2(p, p0, p1); unpack2(y, y0, y1);
  return pack2(__uint_as_float(__float_as_uint(p0) + (__float_as_uint(y0) << 23)),
               __uint_as_float(__float_as_uint(p1) + (__float_as_uint(y1) << 23)));
}
constexpr int kPolyEvery = 4;    // one pair of exponentials in kPolyEvery goes to poly_exp2_pair (0: none)
__device__ __forceinline__ constexpr bool poly_pair(int pair) { return kPolyEvery > 0 && pair % kPolyEvery == 0; }
// (s.x, s.y) += (2^(x0 * scale + c0), 2^(x1 * scale + c1)); poly (known once the caller's loop is unrolled) picks the unit that takes the exponentials
__device__ __forceinline__ uint64_t exp2_acc2(bool poly, uint64_t sum, float x0, float x1, uint64_t scale,
                                              uint64_t c) {
  const uint64_t t = fma2(pack2(x0, x1), scale, c);
  if (poly) return add2(sum, poly_exp2_pair(t));
  float t0, t1;
  unpack2(t, t0, t1);
  return add2(sum, pack2(fast_exp2(t0), fast_exp2(t1)));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major, 128-byte swizzle, rows 128 B apart, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
  d |= (uint64_t)1 << 46;                            // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                            // 128-byte swizzle
  return d;
}

// ------------------------------------------------------------------------------------------ work split
struct Seg {
  int bh;        // head (sample * Hkv + kv head)
  int key0;      // first key of the first tile (may be negative in sweep 2: the pooling halo)
  int ntiles;
  int out0, out1;  // sweep 2: prefix positions this segment writes
  bool new_head;
};

struct SegIter {
  long long u, u_end;
  int uph, half, cur_bh, mode, back;
  __device__ SegIter(const Params& p, int cta, int grid) {
    mode = p.mode;
    back = p.mode == kEmit && p.back;
    uph = mode == kStats ? p.tph : p.P;
    const long long total = (long long)p.heads * uph;
    u = total * cta / grid;
    u_end = total * (cta + 1) / grid;
    half = p.half;
    cur_bh = -1;
  }
  __device__ bool next(Seg& s) {
    if (u >= u_end) return false;
    if (back) {
      // the last segment of what is left: it ends at u_end and starts at the head's first position, the
      // slice's start or one segment's length before its end, whichever comes last
      const int bh = (int)((u_end - 1) / uph);
      long long b = (long long)bh * uph;
      if (b < u) b = u;
      if (b < u_end - (kMaxSegTiles * kTileKeys - 2 * half)) b = u_end - (kMaxSegTiles * kTileKeys - 2 * half);
      const int off = (int)(b - (long long)bh * uph), len = (int)(u_end - b);
      s.bh = bh;
      s.out0 = off; s.out1 = off + len; s.key0 = off - half;
      s.ntiles = (len + 2 * half + kTileKeys - 1) / kTileKeys;
      s.new_head = bh != cur_bh;
      cur_bh = bh;
      u_end = b;
      return true;
    }
    const int bh = (int)(u / uph), off = (int)(u % uph);
    long long e = (long long)(bh + 1) * uph;
    if (e > u_end) e = u_end;
    if (mode == kEmit && e > u + (kMaxSegTiles * kTileKeys - 2 * half)) e = u + (kMaxSegTiles * kTileKeys - 2 * half);
    const int len = (int)(e - u);
    s.bh = bh;
    if (mode == kStats) {
      s.key0 = off * kTileKeys; s.ntiles = len; s.out0 = s.out1 = 0;
    } else {
      s.out0 = off; s.out1 = off + len; s.key0 = off - half;
      s.ntiles = (len + 2 * half + kTileKeys - 1) / kTileKeys;
    }
    s.new_head = bh != cur_bh;
    cur_bh = bh;
    u = e;
    return true;
  }
};

// CTA that owns key tile x of the flattened (head, tile) space, when `total` tiles are cut into `grid` slices.
__host__ __device__ __forceinline__ int tile_owner(long long x, long long total, int grid) {
  return (int)(((x + 1) * grid + total - 1) / total) - 1;
}

// ------------------------------------------------------------------------------------------ kernel
// job0 uses maps0, job1 uses maps1; a job with mode kNone is skipped.
// kFast: both jobs have exactly 128 window rows of 128 dims (ws*G = 128, D = 128, the shape of the 32/8-head models):
// the row-block count, the chunk count and the k-step count are then compile-time constants.
template <bool kFast>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ Maps maps0, const __grid_constant__ Maps maps1,
                const __grid_constant__ Params job0, const __grid_constant__ Params job1) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_smem = smem;                              // [half][256 rows][128 B]
  uint8_t* k_smem = smem + kQRegion;                   // [stage][half][128 rows][128 B]
  float* nlse_s = reinterpret_cast<float*>(k_smem + kKRegion);         // [256] minus lse2 per window row (sweep 2)
  float2* merge_s = reinterpret_cast<float2*>(nlse_s + 256);            // [3][256] partials of column parts 1..3 (sweep 1)
  float* raw_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(nlse_s) + kMiscBytes);   // [half][kMaxSegTiles * 128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(raw_s) + kRawBytes);
  // barriers: full[kStages], empty[kStages], tmem_full[4], tmem_empty[4], q_full, drain[2]
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  const uint32_t bar0 = smem_u32(bars);
  auto FULL = [&](int s) { return bar0 + 8u * s; };
  auto EMPTY = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto TFULL = [&](int t) { return bar0 + 8u * (2 * kStages + t); };
  auto TEMPTY = [&](int t) { return bar0 + 8u * (2 * kStages + 4 + t); };
  const uint32_t QFULL = bar0 + 8u * (2 * kStages + 8);
  auto DRAIN = [&](int i) { return bar0 + 8u * (2 * kStages + 9 + i); };   // one per MMA issuer, used after an abort only

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_s;
  auto NMBLK = [](const Params& p) { return kFast ? 1 : p.nmblk; };
  auto DIMS = [](const Params& p) { return kFast ? 128 : p.D; };

  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(FULL(s), 1); mbar_init(EMPTY(s), 1); }
    for (int t = 0; t < 4; ++t) { mbar_init(TFULL(t), 1); mbar_init(TEMPTY(t), 8); }
    mbar_init(QFULL, 1);
    mbar_init(DRAIN(0), 1); mbar_init(DRAIN(1), 1);
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
      int tile = 0, nq = 0;
      int withheld = -1;                       // the tile (counted over the launch) whose copy the test hook skipped
      bool ok = true;                          // false once a wait has run out, here or in another thread
      for (int jb = 0; jb < 2 && ok; ++jb) {
        const Params& p = jb ? job1 : job0;
        if (p.mode == kNone) continue;
        const Maps& maps = jb ? maps1 : maps0;
        const int halves = DIMS(p) / 64;
        const uint32_t tile_bytes = (uint32_t)halves * kHalfBytes;
        const int withhold = blockIdx.x == 0 ? p.withhold_tile : -1;
        SegIter it(p, blockIdx.x, gridDim.x);
        Seg sg;
        int job_tile = 0;
        const int keep_from = p.mode == kStats ? (int)(it.u_end - it.u) - p.retain_tiles : 0x7fffffff;
        const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
        while (ok && it.next(sg)) {
          const int hh = sg.bh % p.hpl;
          const CUtensorMap* q_map = &maps.q[sg.bh / p.hpl];
          const CUtensorMap* k_map = &maps.k[sg.bh / p.hpl];
          if (sg.new_head) {
            // every MMA that read the previous queries must have finished: the last tile of either issuer
            for (int last = tile - 1; last >= 0 && last >= tile - 2; --last)
              ok = ok && mbar_wait(EMPTY(last % kStages), (last / kStages) & 1, abort_flag, p.status, 101, p.wait_cycles);
            if (ok) {
              mbar_expect_tx(QFULL, (uint32_t)(NMBLK(p) * halves) * kHalfBytes);
              for (int h = 0; h < halves; ++h)
                for (int mb = 0; mb < NMBLK(p); ++mb)
                  tma_load_3d(smem_u32(q_smem + h * (2 * kHalfBytes) + mb * kHalfBytes), q_map, QFULL, 64 * h, 128 * mb, hh);
              ++nq;
            }
          }
          for (int i = 0; i < sg.ntiles; ++i, ++tile, ++job_tile) {
            const int s = tile % kStages, n = tile / kStages;
            if (!mbar_wait(EMPTY(s), (n & 1) ^ 1, abort_flag, p.status, 102, p.wait_cycles)) { ok = false; break; }
            if (job_tile == withhold) { withheld = tile; continue; }   // test hook: this tile never arrives
            mbar_expect_tx(FULL(s), tile_bytes);
            if (p.retain_tiles > 0) {
              const uint64_t pol = job_tile >= keep_from ? pol_last : pol_first;
              for (int h = 0; h < halves; ++h)
                tma_load_3d_hint(smem_u32(k_smem + (s * 2 + h) * kHalfBytes), k_map, FULL(s), 64 * h, sg.key0 + i * kTileKeys, hh, pol);
            } else {
              for (int h = 0; h < halves; ++h)
                tma_load_3d(smem_u32(k_smem + (s * 2 + h) * kHalfBytes), k_map, FULL(s), 64 * h, sg.key0 + i * kTileKeys, hh);
            }
          }
        }
      }
      if (!ok || *abort_flag) {
        // copies of this CTA that may still be on their way must land before its shared memory is given up:
        // for every ring stage, the last tile (below `tile`) whose copy went there
        for (int s = 0; s < kStages; ++s) {
          int last = tile - 1 - ((tile - 1 - s) % kStages + kStages) % kStages;
          if (last == withheld) last -= kStages;
          if (last >= 0) mbar_drain(FULL(s), (last / kStages) & 1);
        }
        if (nq > 0) mbar_drain(QFULL, (nq - 1) & 1);
      }
    }
  } else if (warp == 1 || warp == kMmaWarp2) {
    // ------------------------------------------------------------------ MMA issuers
    // Two threads on different schedulers share the work: tile i belongs to issuer i & 1, which is also its
    // accumulator stage.  One thread alone needs about as long to issue a tile's instructions as the
    // tensor core needs to run them.
    if (lane == 0) {
      const int which = warp == 1 ? 0 : 1;
      const uint64_t kdesc0 = smem_desc(smem_u32(k_smem)), qdesc0 = smem_desc(smem_u32(q_smem));
      const uint32_t kq_lo[2] = {(uint32_t)kdesc0, (uint32_t)qdesc0}, desc_hi = (uint32_t)(kdesc0 >> 32);
      int tile = 0, nq = 0;
      bool q_wait = false;
      for (int jb = 0; jb < 2; ++jb) {
        const Params& p = jb ? job1 : job0;
        if (p.mode == kNone) continue;
        const int ksteps = DIMS(p) / 16;
        const int tmask = NMBLK(p) == 1 ? 3 : 1, tshift = NMBLK(p) == 1 ? 2 : 1, scols = NMBLK(p) == 1 ? 128 : 256;
        SegIter it(p, blockIdx.x, gridDim.x);
        Seg sg;
        while (it.next(sg)) {
          // the wait for a head's queries is taken at this issuer's first tile of the head (it may have none)
          if (sg.new_head) { q_wait = true; ++nq; }
          // this thread's tiles only: every other one, by the parity of the tile's number over the launch
          const int tile0 = tile;
          tile += sg.ntiles;
          for (int i = (which ^ tile0) & 1, tile_ = tile0 + i; i < sg.ntiles; i += 2, tile_ += 2) {
            const int tile = tile_;
            bool ok = true;
            if (q_wait) {
              q_wait = false;
              ok = mbar_wait(QFULL, (nq - 1) & 1, abort_flag, p.status, 103, p.wait_cycles);
            }
            const int s = tile % kStages, n = tile / kStages, t = tile & tmask, nt = tile >> tshift;
            ok = ok && mbar_wait(FULL(s), n & 1, abort_flag, p.status, 104, p.wait_cycles);
            ok = ok && mbar_wait(TEMPTY(t), (nt & 1) ^ 1, abort_flag, p.status, 105, p.wait_cycles);
            if (!ok) continue;                           // nothing more is issued once a wait has run out
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(t * scols);
            if (ksteps == 8) {
              // low descriptor words: the tile's ring stage, the queries' row block; 16-byte units
              const uint32_t k_lo = kq_lo[0] + ((uint32_t)(s * 2 * kHalfBytes) >> 4);
              if (p.mode == kStats) {
                for (int mb = 0; mb < NMBLK(p); ++mb)
                  tc_mma_x8<((2 * kHalfBytes) >> 4), (kHalfBytes >> 4)>(d_tmem + mb * 128, kq_lo[1] + ((uint32_t)(mb * kHalfBytes) >> 4),
                                                                     k_lo, desc_hi, p.idesc);
              } else {
                tc_mma_x8<(kHalfBytes >> 4), ((2 * kHalfBytes) >> 4)>(d_tmem, k_lo, kq_lo[1], desc_hi, p.idesc);
              }
            } else if (p.mode == kStats) {
              for (int mb = 0; mb < NMBLK(p); ++mb)
                for (int ks = 0; ks < ksteps; ++ks) {
                  const uint64_t a = smem_desc(smem_u32(q_smem + (ks >> 2) * (2 * kHalfBytes) + mb * kHalfBytes) + (ks & 3) * 32);
                  const uint64_t b = smem_desc(smem_u32(k_smem + (s * 2 + (ks >> 2)) * kHalfBytes) + (ks & 3) * 32);
                  tc_mma(d_tmem + mb * 128, a, b, p.idesc, ks > 0);
                }
            } else {
              for (int ks = 0; ks < ksteps; ++ks) {
                const uint64_t a = smem_desc(smem_u32(k_smem + (s * 2 + (ks >> 2)) * kHalfBytes) + (ks & 3) * 32);
                const uint64_t b = smem_desc(smem_u32(q_smem + (ks >> 2) * (2 * kHalfBytes)) + (ks & 3) * 32);
                tc_mma(d_tmem, a, b, p.idesc, ks > 0);
              }
            }
            tc_commit(EMPTY(s));      // the K slot may be refilled once these MMAs have read it
            tc_commit(TFULL(t));      // the accumulator is complete
          }
        }
      }
      if (*abort_flag) {
        // the MMAs this thread has issued must have finished before the tensor memory is freed
        tc_commit(DRAIN(which));
        mbar_drain(DRAIN(which), 0);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const int part = (warp - 2) >> 2;          // 0..3: group (tile parity) and half of the accumulator columns
    const int grp = part >> 1, half = part & 1;
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    const int row = quad * 32 + lane;          // TMEM lane = window row (sweep 1) or key within the tile (sweep 2)
    const int sid = threadIdx.x - 64;          // 0..511 among the softmax threads
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    int tile = 0;
    for (int jb = 0; jb < 2; ++jb) {
      const Params& p = jb ? job1 : job0;
      if (p.mode == kNone) continue;
      SegIter it(p, blockIdx.x, gridDim.x);
      Seg sg;
      const int tmask = NMBLK(p) == 1 ? 3 : 1, tshift = NMBLK(p) == 1 ? 2 : 1, scols = NMBLK(p) == 1 ? 128 : 256;
      const uint64_t scale22 = pack2(p.scale2, p.scale2);
      while (it.next(sg)) {
        if (p.mode == kStats) {
          // ------------------------------------------------------------ sweep 1: (max, sum) per window row
          float mx[2] = {-INFINITY, -INFINITY}, sum[2] = {0.f, 0.f};
          const int limit0 = p.P + (row % p.ws), limit1 = p.P + ((row + 128) % p.ws);
          // this thread's tiles only: every other one, by the parity of the tile's number over the launch
          const int tile0 = tile;
          tile += sg.ntiles;
          for (int i = (grp ^ tile0) & 1, tile_ = tile0 + i; i < sg.ntiles; i += 2, tile_ += 2) {
            const int tile = tile_;
            const int t = tile & tmask, nt = tile >> tshift;
            mbar_wait(TFULL(t), nt & 1, abort_flag, p.status, 106, p.wait_cycles);
            tc_fence_after();
            const uint32_t taddr = lane_addr + (uint32_t)(t * scols + half * 64);
            const int kb0 = sg.key0 + i * kTileKeys + half * 64;
            const bool need_mask = kb0 + 63 > p.P;
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
              if (mb >= NMBLK(p)) break;
#pragma unroll
              for (int hh = 0; hh < 2; ++hh) {
                float xv[32];
                tc_ld32(taddr + mb * 128 + hh * 32, xv);
                tc_wait_ld();
                if (mb + 1 == NMBLK(p) && hh == 1) {              // last read of this stage: release it
                  tc_fence_before();
                  __syncwarp();
                  if (lane == 0) mbar_arrive(TEMPTY(t));
                }
                if (need_mask) {
                  const int limit = mb ? limit1 : limit0;
                  const int kb = kb0 + hh * 32;
#pragma unroll
                  for (int e = 0; e < 32; ++e) if (kb + e > limit) xv[e] = -INFINITY;
                }
                float cm = fmax3(xv[0], xv[1], xv[2]);
#pragma unroll
                for (int e = 3; e < 31; e += 2) cm = fmax3(cm, xv[e], xv[e + 1]);
                cm = fmaxf(cm, xv[31]);
                if (cm == -INFINITY) continue;
                const float mnew = fmaxf(mx[mb], cm * p.scale2);
                if (mnew > mx[mb]) { sum[mb] *= fast_exp2(mx[mb] - mnew); mx[mb] = mnew; }
                uint64_t s01 = 0ull, s23 = 0ull;            // four partial sums, as two packed pairs
                const uint64_t neg2 = pack2(-mx[mb], -mx[mb]);
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                  s01 = exp2_acc2(poly_pair(e / 2), s01, xv[e], xv[e + 1], scale22, neg2);
                  s23 = exp2_acc2(poly_pair(e / 2 + 1), s23, xv[e + 2], xv[e + 3], scale22, neg2);
                }
                float s0, s1, s2, s3;
                unpack2(s01, s0, s1); unpack2(s23, s2, s3);
                sum[mb] += (s0 + s1) + (s2 + s3);
              }
            }
          }
          // merge the four column parts and publish this CTA's statistics for the head
          if (part > 0) {
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) merge_s[(part - 1) * 256 + row + 128 * mb] = make_float2(mx[mb], sum[mb]);
          }
          asm volatile("bar.sync 1, 512;" ::: "memory");
          if (part == 0) {
            const long long total = (long long)p.heads * p.tph;
            const int slot = blockIdx.x - tile_owner((long long)sg.bh * p.tph, total, gridDim.x);
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
              const int r = row + 128 * mb;
              if (mb < NMBLK(p) && r < p.M) {
                float m = mx[mb];
#pragma unroll
                for (int q = 0; q < 3; ++q) m = fmaxf(m, merge_s[q * 256 + r].x);
                float l = 0.f;
                if (m > -INFINITY) {
                  l = sum[mb] * fast_exp2(mx[mb] - m);
#pragma unroll
                  for (int q = 0; q < 3; ++q) { const float2 o = merge_s[q * 256 + r]; l += o.y * fast_exp2(o.x - m); }
                }
                p.stats[((size_t)sg.bh * p.slots + slot) * p.m_stride + r] = make_float2(m, l);
              }
            }
          }
          asm volatile("bar.sync 1, 512;" ::: "memory");
        } else {
          // ------------------------------------------------------------ sweep 2: one thread per key
          const int nb = sg.bh;
          if (sg.new_head && sid < 256) {
            // lse2 of every window row from the partial statistics of sweep 1
            const long long total = (long long)p.heads * p.tph;
            const int c_lo = tile_owner((long long)nb * p.tph, total, p.stats_grid);
            const int c_hi = tile_owner((long long)(nb + 1) * p.tph - 1, total, p.stats_grid);
            float lse = INFINITY;
            const float* lse_in = (jb ? maps1 : maps0).lse[nb / p.hpl];
            if (lse_in) {
              if (sid < p.M) lse = lse_in[(size_t)(nb % p.hpl) * p.M + sid] * kLog2e;
            } else if (sid < p.M) {
              float m = -INFINITY;
              for (int c = 0; c <= c_hi - c_lo; ++c) m = fmaxf(m, p.stats[((size_t)nb * p.slots + c) * p.m_stride + sid].x);
              float l = 0.f;
              for (int c = 0; c <= c_hi - c_lo; ++c) {
                const float2 st = p.stats[((size_t)nb * p.slots + c) * p.m_stride + sid];
                l += st.y * fast_exp2(st.x - m);
              }
              lse = m + log2f(l);
            }
            nlse_s[sid] = -lse;
          }
          asm volatile("bar.sync 1, 512;" ::: "memory");
          const int nchunk = kFast ? 8 : p.nq16 >> 4;               // 16-column chunks; this warp takes half, half+2, ...
          float* my_raw = raw_s + half * (kMaxSegTiles * kTileKeys);
          // this thread's tiles only: every other one, by the parity of the tile's number over the launch
          const int tile0 = tile;
          tile += sg.ntiles;
          for (int i = (grp ^ tile0) & 1, tile_ = tile0 + i; i < sg.ntiles; i += 2, tile_ += 2) {
            const int tile = tile_;
            const int t = tile & tmask, nt = tile >> tshift;
            mbar_wait(TFULL(t), nt & 1, abort_flag, p.status, 107, p.wait_cycles);
            tc_fence_after();
            const uint32_t taddr = lane_addr + (uint32_t)(t * scols);
            uint64_t a01 = 0ull, a23 = 0ull;               // four partial sums, as two packed pairs
            if (half >= nchunk) {                              // a single chunk (ws*G <= 16): nothing for this warp to read
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(TEMPTY(t));
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {                  // two 16-column chunks per round
              const int c0 = half + 4 * jj, c1 = c0 + 2;
              if (c0 >= nchunk) break;
              float x0[16], x1[16];
              tc_ld16(taddr + c0 * 16, x0);
              if (c1 < nchunk) tc_ld16(taddr + c1 * 16, x1);
              tc_wait_ld();
              if (c0 + 4 >= nchunk) {                          // this warp's last read of the stage: release it
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(TEMPTY(t));
              }
#pragma unroll
              for (int e = 0; e < 16; e += 4) {
                const ulonglong2 ls = *reinterpret_cast<const ulonglong2*>(&nlse_s[c0 * 16 + e]);   // minus lse, four rows
                a01 = exp2_acc2(poly_pair(e / 2), a01, x0[e], x0[e + 1], scale22, ls.x);
                a23 = exp2_acc2(poly_pair(e / 2 + 1), a23, x0[e + 2], x0[e + 3], scale22, ls.y);
              }
              if (c1 < nchunk) {
#pragma unroll
                for (int e = 0; e < 16; e += 4) {
                  const ulonglong2 ls = *reinterpret_cast<const ulonglong2*>(&nlse_s[c1 * 16 + e]);
                  a01 = exp2_acc2(poly_pair(e / 2), a01, x1[e], x1[e + 1], scale22, ls.x);
                  a23 = exp2_acc2(poly_pair(e / 2 + 1), a23, x1[e + 2], x1[e + 3], scale22, ls.y);
                }
              }
            }
            float a0, a1, a2, a3;
            unpack2(a01, a0, a1); unpack2(a23, a2, a3);
            my_raw[i * kTileKeys + row] = (a0 + a1) + (a2 + a3);
          }
          asm volatile("bar.sync 1, 512;" ::: "memory");
          // add up the two column halves in a fixed order; raw_s[x] then belongs to key key0 + x
          for (int x = sid; x < sg.ntiles * kTileKeys; x += kSoftmaxThreads)
            raw_s[x] = (raw_s[x] + raw_s[kMaxSegTiles * kTileKeys + x]) * p.out_scale;
          asm volatile("bar.sync 1, 512;" ::: "memory");
          // Eq. 2's pooling over this segment
          for (int o = sg.out0 + sid; o < sg.out1; o += kSoftmaxThreads) {
            const int x = o - sg.key0;
            float v = raw_s[x];
            if (p.pool_avg) {
              int cnt = 1;
              for (int d = 1; d <= p.half; ++d) {
                if (o - d >= 0) { v += raw_s[x - d]; ++cnt; }
                if (o + d < p.P) { v += raw_s[x + d]; ++cnt; }
              }
              v = v / (float)cnt;
            } else {
              for (int d = 1; d <= p.half; ++d) {
                if (o - d >= 0) v = fmaxf(v, raw_s[x - d]);
                if (o + d < p.P) v = fmaxf(v, raw_s[x + d]);
              }
            }
            const size_t at = (size_t)nb * p.P + o;
            p.scores[at] = v;
            if (p.copy_out) p.copy_out[at] = v;
          }
          asm volatile("bar.sync 1, 512;" ::: "memory");
        }
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
