// Online activation quantizer without a rotation:  v = x * pre,  per-token symmetric INT4, packed.
//
// Methodology section, last paragraph: every quantized layer quantizes its activations online, in
// the forward pass, while only two layers also rotate them there (the down-projection and the
// attention output projection).  The other layers see activations that
// are already in the rotated basis and only quantize them; this is that kernel.
//
// Pure streaming work, 2 bytes in and half a byte out per value: T threads share a row, a thread
// holds up to 4 (long rows: 8) chunks of 8 consecutive values (16-byte loads, chunk c of thread t is chunk t + c T
// of the row), so that the 8 codes of a chunk are exactly one aligned 32-bit word of the output and
// no transposition is needed.  The next row's loads are in flight during the arithmetic; the threads
// of a row meet once, for the row maximum.
#include "common.cuh"
#include "rowquant.cuh"

namespace smoothrot {
namespace {

constexpr int kPlainThreads = 256;
constexpr int kPlainMaxChunks = 8;          // chunks per thread: a row has at most 8 * 8 * 256 values

__device__ __forceinline__ void plain_group_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// T: threads per row (64, 128 or 256); CH: chunks per thread (4 keeps the registers low enough for
// four CTAs per SM, 8 is for the longest rows)
template <int T, int CH>
__global__ void __launch_bounds__(kPlainThreads, CH <= 4 ? 4 : 2)
plain_quant_kernel(const __half* __restrict__ x, int64_t ld, int rows, int K, const float* __restrict__ pre,
                   bool low_clamp, float clip, uint8_t* __restrict__ q_out, float* __restrict__ step_out) {
  __shared__ float red[kPlainThreads / 32];
  constexpr int groups = kPlainThreads / T;
  constexpr int warps = T / 32;
  const int group = threadIdx.x / T;
  const int t = threadIdx.x - group * T;
  const int chunks = K >> 3;
  const int row_stride = gridDim.x * groups;

  uint4 raw[CH];
  int m = blockIdx.x * groups + group;
  if (m < rows) {
    const uint4* src = reinterpret_cast<const uint4*>(x + int64_t(m) * ld);
#pragma unroll
    for (int c = 0; c < CH; ++c)
      raw[c] = t + c * T < chunks ? __ldcs(src + t + c * T) : make_uint4(0u, 0u, 0u, 0u);
  }
  for (; m < rows; m += row_stride) {
    f32x2 v[CH][4];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      v[c][0] = half2_to_f32x2(raw[c].x);
      v[c][1] = half2_to_f32x2(raw[c].y);
      v[c][2] = half2_to_f32x2(raw[c].z);
      v[c][3] = half2_to_f32x2(raw[c].w);
    }
    const int next = m + row_stride;
    if (next < rows) {                       // the next row of this group is on its way during the arithmetic
      const uint4* src = reinterpret_cast<const uint4*>(x + int64_t(next) * ld);
#pragma unroll
      for (int c = 0; c < CH; ++c)
        raw[c] = t + c * T < chunks ? __ldcs(src + t + c * T) : make_uint4(0u, 0u, 0u, 0u);
    }
    if (pre != nullptr) {
      const float4* p = reinterpret_cast<const float4*>(pre);
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        if (t + c * T < chunks) {
          const float4 a = __ldg(p + 2 * (t + c * T)), b = __ldg(p + 2 * (t + c * T) + 1);
          v[c][0] = mul2(v[c][0], pack2(a.x, a.y));
          v[c][1] = mul2(v[c][1], pack2(a.z, a.w));
          v[c][2] = mul2(v[c][2], pack2(b.x, b.y));
          v[c][3] = mul2(v[c][3], pack2(b.z, b.w));
        }
      }
    }
    float amax = 0.0f;
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float a, b;
        unpack2(v[c][k], a, b);
        amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
      }
    amax = warp_max(amax);
    if (warps > 1) {
      const int w0 = group * warps;
      if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
      plain_group_sync(1 + group, T);
      amax = red[w0];
#pragma unroll
      for (int w = 1; w < warps; ++w) amax = fmaxf(amax, red[w0 + w]);
      plain_group_sync(1 + group, T);      // red is written again by the next row
    }
    const float step = step_from_absmax(amax, clip);
    if (t == 0) step_out[m] = step;
    // x / step as the correctly rounded fp32 quotient, without a division per value: multiply by
    // the rounded reciprocal, then one residual correction (r = x - q step exactly in an fma, q + r / step
    // rounded once).  Unlike the rotated paths, whose values are sums with dense mantissas, fp16 inputs
    // divided by a step that itself comes from an fp16 maximum land on rounding ties all the time
    // (2.50000005 rounds to 2.5 in fp32 and then to the even code 2), so the quotient has to be the
    // same fp32 number the definition rounds.
    const float inv = __frcp_rn(step);
    const f32x2 inv2 = pack2(inv, inv), neg_step2 = pack2(-step, -step);
    // Round to nearest even and bias by 8: the low byte of the float's bit pattern is code + 8.
    const float kMagic = 12582912.0f + 8.0f;             // 1.5 * 2^23 + 8
    const f32x2 magic2 = pack2(kMagic, kMagic);
    uint32_t* q_row = reinterpret_cast<uint32_t*>(q_out + int64_t(m) * (K >> 1));
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      uint32_t lo[4], hi[4];                 // even / odd positions of the chunk
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float q0, q1;
        f32x2 q = mul2(v[c][k], inv2);
        q = fma2(fma2(q, neg_step2, v[c][k]), inv2, q);
        unpack2(add2(q, magic2), q0, q1);
        if (low_clamp) {
          q0 = fmaxf(fminf(q0, 12582912.0f + 15.0f), 12582912.0f);
          q1 = fmaxf(fminf(q1, 12582912.0f + 15.0f), 12582912.0f);
        }
        lo[k] = __float_as_uint(q0);
        hi[k] = __float_as_uint(q1);
      }
      uint32_t even = __byte_perm(__byte_perm(lo[0], lo[1], 0x0040), __byte_perm(lo[2], lo[3], 0x0040), 0x5410);
      uint32_t odd = __byte_perm(__byte_perm(hi[0], hi[1], 0x0040), __byte_perm(hi[2], hi[3], 0x0040), 0x5410);
      if (!low_clamp) {
        // the row maximum sits below 8.5 steps: a byte is code + 8 in [0, 16], and 16 comes down to 15
        even -= (even >> 4) & 0x01010101u;
        odd -= (odd >> 4) & 0x01010101u;
      }
      // byte k: code 2k in bits 0-3, code 2k + 1 in bits 4-7; offset binary -> two's complement
      if (t + c * T < chunks) q_row[t + c * T] = (even | (odd << 4)) ^ 0x88888888u;
    }
  }
}

}  // namespace
}  // namespace smoothrot

extern "C" {

int smoothrot_quant_act_plain(const void* X_f16, int64_t M, int64_t K, int64_t ldx, const float* pre, float clip_a,
                              uint8_t* Xq_out, float* dx_out, void* stream) {
  using namespace smoothrot;
  if (M < 0 || K <= 0) return SMOOTHROT_INVALID_ARG;
  if (!(clip_a > 0.0f) || clip_a > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (K % 8 != 0 || K > 8 * kPlainMaxChunks * 256) return SMOOTHROT_UNSUPPORTED_K;
  if (M == 0) return SMOOTHROT_OK;
  if (X_f16 == nullptr || Xq_out == nullptr || dx_out == nullptr || ldx < K || M > 0x7fffffffLL)
    return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X_f16) || ldx % 8 != 0 || !aligned16(Xq_out) || (pre != nullptr && !aligned16(pre)))
    return SMOOTHROT_BAD_ALIGNMENT;
  const bool low = 7.0f / clip_a >= 8.49f;               // codes below -8 can only come up then
  // the fewest values per thread that still cover the row with at most 256 threads
  const int64_t chunks = K / 8;
  const int CH = chunks <= 4 * 256 ? 4 : 8;
  const int T = chunks <= CH * 64 ? 64 : (chunks <= CH * 128 ? 128 : 256);
  const int groups = kPlainThreads / T;
  int64_t grid = (M + groups - 1) / groups;
  const int64_t cap = int64_t(device_sm_count()) * (CH <= 4 ? 4 : 2);
  if (grid > cap) grid = cap;
  auto launch = [&](auto kern) {
    kern<<<unsigned(grid), kPlainThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(X_f16), ldx, int(M), int(K), pre, low, clip_a, Xq_out, dx_out);
    count_launch();
    return launch_status();
  };
  if (CH == 4) {
    if (T == 64) return launch(plain_quant_kernel<64, 4>);
    if (T == 128) return launch(plain_quant_kernel<128, 4>);
    return launch(plain_quant_kernel<256, 4>);
  }
  return launch(plain_quant_kernel<256, 8>);
}

}  // extern "C"
