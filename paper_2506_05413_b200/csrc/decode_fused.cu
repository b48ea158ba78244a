// Fused decode layer of libsmoothrot: for a handful of tokens, the online activation path
// (x * pre) H / sqrt(K) -> per-token INT4 (Fig. 2, "hadamard" then "quantize") and the quantized
// product with the packed weights (Eq. 2 on Eq. 1's integer codes) in ONE kernel.
//
// With one to four tokens the two calls of the layer cost about the same fixed time each (a kernel
// that loads, computes and stores needs 4 to 5 microseconds from launch to last store whatever it
// touches), and the rotation of a token is tiny: 4096 x 12 additions.  So every CTA of the decode
// kernel redoes it for itself, in shared memory, while its share of the weights is already on its way
// from HBM: the loads of the weight rows are issued first, the rotation and quantization of the
// tokens run in their shadow, and the products follow as in w4a4_decode_kernel, row group after
// row group with the next group's weights in flight.  The tokens' codes never leave the SM (CTA 0
// can export them for inspection).
//
// K = 4096: 256 threads hold 16 values each; three rounds of four butterfly stages in registers with
// two exchanges through shared memory (indices 16t+i, then (t&15)+16i+256(t>>4), then t+256i; one
// float of padding per 16 keeps all three patterns free of bank conflicts).
#include "common.cuh"
#include "decode.cuh"
#include "rowquant.cuh"

namespace smoothrot {
namespace gemm {
namespace {

constexpr int kFusedK = 4096;
constexpr int kFusedThreads = 256;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kFusedMaxTokens = 4;
constexpr int kFusedChunksPerWarp = kFusedK / 128 / kFusedWarps;   // 64-byte chunks of a packed row per warp: 4

__device__ __forceinline__ int padded(int j) { return j + (j >> 4); }

// Four butterfly stages between 16 values held by one thread.
__device__ __forceinline__ void butterflies16(float (&v)[16]) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if ((k & h) == 0) {
        const float a = v[k], b = v[k + h];
        v[k] = a + b;
        v[k + h] = a - b;
      }
    }
  }
}

__global__ void __launch_bounds__(kFusedThreads)
fused_decode_kernel(const __half* __restrict__ X, int M, int64_t ldx, const float* __restrict__ pre, float clip,
                    bool low_clamp, const uint8_t* __restrict__ Wq, int N, const float* __restrict__ dw,
                    __half* __restrict__ Y, int64_t ldy, uint8_t* __restrict__ xq_out, float* __restrict__ dx_out) {
  constexpr int K = kFusedK;
  __shared__ float buf[K + K / 16];                              // the row during the rotation
  __shared__ __align__(16) uint32_t xs[kFusedMaxTokens][2][K / 8];   // codes as int8 lanes (16 * code): even / odd positions
  __shared__ float sred[kFusedWarps];
  __shared__ float sdx[kFusedMaxTokens];
  __shared__ int red[kFusedWarps][128];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int64_t row_bytes = K / 2;
  const int groups = (N + 15) >> 4;                       // row groups of 16 output channels
  // this warp's weights for one row group: 4 chunks of 64 bytes of rows g and g + 8
  // (a row past the end repeats the last one)
  auto load_weights = [&](uint4 (&w)[kFusedChunksPerWarp][2], int group) {
    const uint8_t* r0 = Wq + int64_t(min(group * 16 + g, N - 1)) * row_bytes + t * 16;
    const uint8_t* r1 = Wq + int64_t(min(group * 16 + 8 + g, N - 1)) * row_bytes + t * 16;
#pragma unroll
    for (int u = 0; u < kFusedChunksPerWarp; ++u) {
      const int cc = warp + u * kFusedWarps;
      w[u][0] = load_stream_16(r0 + cc * 64);
      w[u][1] = load_stream_16(r1 + cc * 64);
    }
  };

  // 1. the weights of the first row group are on their way before anything else
  uint4 w[kFusedChunksPerWarp][2], w_next[kFusedChunksPerWarp][2];
  int group = blockIdx.x;
  if (group < groups) load_weights(w, group);
  const int out_m = tid >> 4;                             // the token of the output this thread finishes (tid < 128)

  // 2. the tokens: rotate, quantize, leave the codes in shared memory
  for (int m = 0; m < M; ++m) {
    float v[16];
    {
      const uint4* src = reinterpret_cast<const uint4*>(X + int64_t(m) * ldx + tid * 16);
      const uint4 a = __ldg(src), b = __ldg(src + 1);
      const uint32_t raw[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int k = 0; k < 8; ++k) unpack2(half2_to_f32x2(raw[k]), v[2 * k], v[2 * k + 1]);
      if (pre != nullptr) {
        const float4* ps = reinterpret_cast<const float4*>(pre + tid * 16);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float4 s = __ldg(ps + k);
          v[4 * k] *= s.x;
          v[4 * k + 1] *= s.y;
          v[4 * k + 2] *= s.z;
          v[4 * k + 3] *= s.w;
        }
      }
    }
    butterflies16(v);                                   // index bits 0-3
#pragma unroll
    for (int i = 0; i < 16; ++i) buf[padded(tid * 16 + i)] = v[i];
    __syncthreads();
    const int jb = (tid & 15) + 256 * (tid >> 4);
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = buf[padded(jb + 16 * i)];
    butterflies16(v);                                   // bits 4-7
#pragma unroll
    for (int i = 0; i < 16; ++i) buf[padded(jb + 16 * i)] = v[i];
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = buf[padded(tid + 256 * i)];
    butterflies16(v);                                   // bits 8-11: v[i] is the unnormalised value at tid + 256 i

    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
    amax = warp_max(amax);
    if (lane == 0) sred[warp] = amax;
    __syncthreads();                                    // also: every read of buf is done
    amax = sred[0];
#pragma unroll
    for (int k = 1; k < kFusedWarps; ++k) amax = fmaxf(amax, sred[k]);
    amax *= 0.015625f;                                  // 1 / sqrt(4096): the maximum of the normalised row
    const float step = step_from_absmax(amax, clip);
    const float inv = __frcp_rn(step) * 0.015625f;      // 1 / step for the unnormalised values (exact scaling)
    if (tid == 0) {
      sdx[m] = step;
      if (blockIdx.x == 0 && dx_out != nullptr) dx_out[m] = step;
    }
    // round half to even by the 1.5 * 2^23 constant; clamp to [-8, 7]; int8 lane = 16 * code
    uint8_t* lanes = reinterpret_cast<uint8_t*>(&xs[m][tid & 1][0]);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      float q = __fmaf_rn(v[i], inv, 12582912.0f);
      q = low_clamp ? fmaxf(fminf(q, 12582912.0f + 7.0f), 12582912.0f - 8.0f) : fminf(q, 12582912.0f + 7.0f);
      const int j = tid + 256 * i;
      lanes[(j >> 3) * 4 + ((j >> 1) & 3)] = uint8_t(__float_as_uint(q) << 4);
    }
    // the next token's first write to sred comes after two more barriers; buf is free since the barrier above
  }
  __syncthreads();
  if (blockIdx.x == 0 && xq_out != nullptr) {
    // export of the packed codes: byte i of a row = code 2i (bits 0-3) | code 2i+1 (bits 4-7)
    for (int idx = tid; idx < M * (K / 2); idx += kFusedThreads) {
      const int m = idx / (K / 2), i = idx - m * (K / 2);
      const uint8_t* even = reinterpret_cast<const uint8_t*>(&xs[m][0][0]);
      const uint8_t* odd = reinterpret_cast<const uint8_t*>(&xs[m][1][0]);
      // codes 2i and 2i + 1 sit in lane i of their planes (word i >> 2, slot i & 3)
      xq_out[int64_t(m) * (K / 2) + i] = uint8_t((even[i] >> 4) | (odd[i] & 0xF0u));
    }
  }

  // 3. row groups blockIdx.x, blockIdx.x + gridDim.x, ...: rows g, g + 8 of the group against token g
  //    (tokens past M contribute zeros); the next group's weights are in flight during the products
  const bool live = g < M;
  const uint32_t* xe = &xs[live ? g : 0][0][0];
  const uint32_t* xo = &xs[live ? g : 0][1][0];
  for (; group < groups; group += gridDim.x) {
    const int next = group + gridDim.x;
    if (next < groups) load_weights(w_next, next);
    const int out_n = group * 16 + (tid & 15);
    const float out_dw = (tid < 128 && out_n < N) ? __ldg(dw + out_n) : 0.0f;
    int c[4] = {0, 0, 0, 0};
#pragma unroll
    for (int u = 0; u < kFusedChunksPerWarp; ++u) {
      const int word = ((warp + u * kFusedWarps) * 4 + t) * 4;   // first packed word of this lane's 16 bytes
      uint4 b0 = make_uint4(0u, 0u, 0u, 0u), b1 = b0;
      if (live) {
        b0 = *reinterpret_cast<const uint4*>(xe + word);
        b1 = *reinterpret_cast<const uint4*>(xo + word);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t wa = word_of(w[u][0], i), wb = word_of(w[u][1], i);
        mma_s8_16x8x32(c, even_codes_x16(wa), even_codes_x16(wb), odd_codes_x16(wa), odd_codes_x16(wb),
                       word_of(b0, i), word_of(b1, i));
      }
    }
    // add the warps' sums (int32, fixed order), dequantize, store
    red[warp][(2 * t) * 16 + g] = c[0];
    red[warp][(2 * t + 1) * 16 + g] = c[1];
    red[warp][(2 * t) * 16 + g + 8] = c[2];
    red[warp][(2 * t + 1) * 16 + g + 8] = c[3];
    __syncthreads();
    if (tid < 128 && out_m < M && out_n < N) {
      int sum = 0;
#pragma unroll
      for (int k = 0; k < kFusedWarps; ++k) sum += red[k][tid];
      sum >>= 8;                                         // the sums are 256 * acc, exactly
      Y[int64_t(out_m) * ldy + out_n] = __float2half_rn(float(sum) * (sdx[out_m] * out_dw));
    }
    __syncthreads();                                     // red is written again by the next group
#pragma unroll
    for (int u = 0; u < kFusedChunksPerWarp; ++u) {
      w[u][0] = w_next[u][0];
      w[u][1] = w_next[u][1];
    }
  }
}

}  // namespace
}  // namespace gemm
}  // namespace smoothrot

extern "C" {

int smoothrot_linear_decode(const void* X_f16, int64_t M, int64_t K, int64_t ldx, const float* pre, float clip_a,
                            const uint8_t* Wq, const float* dw, int64_t N, void* Y_f16, int64_t ldy,
                            uint8_t* Xq_out, float* dx_out, void* stream) {
  using namespace smoothrot;
  using namespace smoothrot::gemm;
  if (M < 0 || N < 0 || K <= 0) return SMOOTHROT_INVALID_ARG;
  if (!(clip_a > 0.0f) || clip_a > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (K != kFusedK) return SMOOTHROT_UNSUPPORTED_K;
  if (M > kFusedMaxTokens || N % 8 != 0 || N > 0x3fffffffLL) return SMOOTHROT_INVALID_ARG;
  if (M == 0 || N == 0) return SMOOTHROT_OK;
  if (X_f16 == nullptr || Wq == nullptr || dw == nullptr || Y_f16 == nullptr || ldx < K || ldy < N)
    return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X_f16) || ldx % 8 != 0 || !aligned16(Wq) || (pre != nullptr && !aligned16(pre)))
    return SMOOTHROT_BAD_ALIGNMENT;
  const bool low = 7.0f / clip_a >= 8.49f;               // codes below -8 can only come up then
  // every CTA rotates the tokens once, so there are no more CTAs than fit the machine at a time
  // (2 per SM at this register count), each taking the same number of row groups
  const int64_t groups = (N + 15) / 16;
  const int64_t slots = int64_t(device_sm_count()) * 2;
  const int64_t per_cta = (groups + slots - 1) / slots;
  const unsigned grid = unsigned((groups + per_cta - 1) / per_cta);
  fused_decode_kernel<<<grid, kFusedThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __half*>(X_f16), int(M), ldx, pre, clip_a, low, Wq, int(N), dw, static_cast<__half*>(Y_f16), ldy,
      Xq_out, dx_out);
  count_launch();
  return launch_status();
}

}  // extern "C"
