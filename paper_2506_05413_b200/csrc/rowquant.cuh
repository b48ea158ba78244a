// Device helpers shared by the row transform kernels of libsmoothrot: the packed fp32 pair
// arithmetic of sm_100, the warp maximum and the step size of the symmetric 4-bit quantizer.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace smoothrot {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Step size of Eq. 1's symmetric form with a clip ratio: clip * max / 7.
__device__ __forceinline__ float step_from_absmax(float amax, float clip) {
  return amax == 0.0f ? 1.0f : __fdiv_rn(__fmul_rn(clip, amax), 7.0f);
}

// Two fp32 values in one 64-bit register, for the packed add/sub/mul/fma of sm_100.
typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// Two fp16 values (one 32-bit word) to fp32 with the mixed-precision fma of sm_100
// (x * 1 + 0, exact): it issues on the FMA pipe, where cvt.f32.f16 would queue on the
// quarter-rate conversion unit.
__device__ __forceinline__ f32x2 half2_to_f32x2(uint32_t raw) {
  float lo, hi;
  asm("{\n\t.reg .b16 l, h, one;\n\t"
      "mov.b32 {l, h}, %2;\n\t"
      "mov.b16 one, 0x3C00;\n\t"
      "fma.rn.f32.f16 %0, l, one, %3;\n\t"
      "fma.rn.f32.f16 %1, h, one, %3;\n\t}"
      : "=f"(lo), "=f"(hi)
      : "r"(raw), "f"(0.0f));
  return pack2(lo, hi);
}

}  // namespace smoothrot
