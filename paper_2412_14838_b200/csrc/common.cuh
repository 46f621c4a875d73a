// Shared definitions of the libdkv kernels: problem shape, small device helpers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dkv {

// Derived problem shape (names follow the paper: L layers, Hkv = H heads scored, G query heads per
// KV head, ws window, P = S - ws prefix tokens, N = wt - ws, Bl = B^l, m update interval).
struct Shape {
  int L, Hq, Hkv, D, Bt, S, ws, pool, N, Bl, m;
  int G;      // Hq / Hkv
  int P;      // S - ws
  int M;      // ws * G window-query rows per KV head
  int Blc;    // min(Bl, P)
  int rows;   // Blc + ws : row stride of the budget buffers
};

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Per-layer device pointers passed by value to kernels that work on several layers at once.
struct LayerPtrs {
  void* kb[128];
  void* vb[128];
};

}  // namespace dkv
