// KV-cache quantizer of libsmoothrot: Eq. 1's asymmetric form on groups of 128 consecutive
// values (Experimental settings, "Quantization": KV caches use asymmetric quantization with a
// group size of 128 and a clip ratio of 0.95), and its dequantizer  Q(x) = (x_int - z) * step.
//
// Pure streaming work: 2 bytes in, 0.5 + 8/128 bytes out per value.  Half a warp owns one group at
// a time: a lane holds 8 consecutive values (one 16-byte load), min and max travel through
// shuffles, every decision (step, zero point, codes) is taken in fp32 with operations in a
// fixed order, so the result does not depend on the launch shape.
#include "common.cuh"

namespace smoothrot {

constexpr int kKvGroup = 128;
constexpr int kKvThreads = 256;

// Half a warp owns a group: a lane holds 8 consecutive values (one 16-byte load) and writes one
// 32-bit word of codes.  The step and the zero point come from true fp32 divisions (once per
// group); the per-value division x / step is a multiplication by the correctly rounded
// reciprocal, which can move a code by one only where x / step lies within an ulp of a rounding
// boundary.
__global__ void __launch_bounds__(kKvThreads)
kv_quant_kernel(const __half* __restrict__ X, int64_t rows, int64_t groups_per_row, int64_t ldx, float clip,
                uint8_t* __restrict__ q_out, float* __restrict__ step_out, float* __restrict__ zero_out) {
  const int sub = threadIdx.x & 15;
  const int64_t half_warp = (int64_t(blockIdx.x) * kKvThreads + threadIdx.x) >> 4;
  const int64_t half_warps = (int64_t(gridDim.x) * kKvThreads) >> 4;
  const int64_t total = rows * groups_per_row;
  // whole warps stay together (shuffles): the loop bound is rounded up to a pair of groups
  for (int64_t g = half_warp; g < ((total + 1) & ~int64_t(1)); g += half_warps) {
    const bool live = g < total;
    const int64_t gg = live ? g : total - 1;
    const int64_t r = gg / groups_per_row;
    const int64_t c = gg - r * groups_per_row;
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(X + r * ldx + c * kKvGroup) + sub);
    float v[8];
    {
      const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        v[2 * i] = f.x;
        v[2 * i + 1] = f.y;
      }
    }
    float hi = v[0], lo = v[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) {
      hi = fmaxf(hi, v[i]);
      lo = fminf(lo, v[i]);
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    }
    hi = __fmul_rn(clip, hi);
    lo = __fmul_rn(clip, lo);
    const float step = hi == lo ? 1.0f : __fdiv_rn(__fsub_rn(hi, lo), 15.0f);
    const float zero = -rintf(__fdiv_rn(lo, step));
    const float inv = __frcp_rn(step);
    uint32_t packed = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float q = fminf(fmaxf(__fadd_rn(rintf(__fmul_rn(v[i], inv)), zero), 0.0f), 15.0f);
      packed |= uint32_t(q) << (4 * i);
    }
    if (live) {
      reinterpret_cast<uint32_t*>(q_out + r * (groups_per_row * (kKvGroup / 2)) + c * (kKvGroup / 2))[sub] = packed;
      if (sub == 0) {
        step_out[g] = step;
        zero_out[g] = zero;
      }
    }
  }
}

__global__ void __launch_bounds__(kKvThreads)
kv_dequant_kernel(const uint8_t* __restrict__ q, const float* __restrict__ step, const float* __restrict__ zero,
                  int64_t rows, int64_t groups_per_row, __half* __restrict__ Y, int64_t ldy) {
  const int sub = threadIdx.x & 15;
  const int64_t half_warp = (int64_t(blockIdx.x) * kKvThreads + threadIdx.x) >> 4;
  const int64_t half_warps = (int64_t(gridDim.x) * kKvThreads) >> 4;
  const int64_t total = rows * groups_per_row;
  for (int64_t g = half_warp; g < total; g += half_warps) {
    const int64_t r = g / groups_per_row;
    const int64_t c = g - r * groups_per_row;
    const uint32_t packed =
        __ldg(reinterpret_cast<const uint32_t*>(q + r * (groups_per_row * (kKvGroup / 2)) + c * (kKvGroup / 2)) + sub);
    const float s = __ldg(step + g), z = __ldg(zero + g);
    uint4 out;
    __half2* h = reinterpret_cast<__half2*>(&out);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = __fmul_rn(__fsub_rn(float((packed >> (8 * i)) & 0xFu), z), s);
      const float b = __fmul_rn(__fsub_rn(float((packed >> (8 * i + 4)) & 0xFu), z), s);
      h[i] = __floats2half2_rn(a, b);
    }
    reinterpret_cast<uint4*>(Y + r * ldy + c * kKvGroup)[sub] = out;
  }
}

static unsigned kv_grid(int64_t groups) {
  const int64_t want = (groups * 16 + kKvThreads - 1) / kKvThreads;     // half a warp per group ...
  const int64_t cap = int64_t(device_sm_count()) * 8 * 4;               // ... up to a few waves, then grid-stride
  return unsigned(want < cap ? (want < 1 ? 1 : want) : cap);
}

}  // namespace smoothrot

extern "C" {

int smoothrot_kv_quant(const void* X_f16, int64_t rows, int64_t C, int64_t ldx, float clip, uint8_t* q_out,
                       float* step_out, float* zero_out, void* stream) {
  using namespace smoothrot;
  if (rows < 0 || C <= 0 || C % kKvGroup != 0) return SMOOTHROT_INVALID_ARG;
  if (!(clip > 0.0f) || clip > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (rows == 0) return SMOOTHROT_OK;
  if (X_f16 == nullptr || q_out == nullptr || step_out == nullptr || zero_out == nullptr || ldx < C)
    return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X_f16) || ldx % 8 != 0 || !aligned16(q_out)) return SMOOTHROT_BAD_ALIGNMENT;
  const int64_t gpr = C / kKvGroup;
  kv_quant_kernel<<<kv_grid(rows * gpr), kKvThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __half*>(X_f16), rows, gpr, ldx, clip, q_out, step_out, zero_out);
  count_launch();
  return launch_status();
}

int smoothrot_kv_dequant(const uint8_t* q, const float* step, const float* zero, int64_t rows, int64_t C,
                         void* Y_f16, int64_t ldy, void* stream) {
  using namespace smoothrot;
  if (rows < 0 || C <= 0 || C % kKvGroup != 0) return SMOOTHROT_INVALID_ARG;
  if (rows == 0) return SMOOTHROT_OK;
  if (q == nullptr || step == nullptr || zero == nullptr || Y_f16 == nullptr || ldy < C) return SMOOTHROT_INVALID_ARG;
  if (!aligned16(q) || !aligned16(Y_f16) || ldy % 8 != 0) return SMOOTHROT_BAD_ALIGNMENT;
  const int64_t gpr = C / kKvGroup;
  kv_dequant_kernel<<<kv_grid(rows * gpr), kKvThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      q, step, zero, rows, gpr, static_cast<__half*>(Y_f16), ldy);
  count_launch();
  return launch_status();
}

}  // extern "C"
