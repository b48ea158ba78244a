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

// Thread-block cluster helpers: rank and size of the cluster, the address of one of this CTA's
// shared-memory locations in another CTA of the cluster, the two halves of the cluster barrier.
__device__ __forceinline__ uint32_t fused_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t fused_cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t fused_peer_address(const void* own, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
               : "=r"(r) : "r"(uint32_t(__cvta_generic_to_shared(own))), "r"(rank));
  return r;
}
__device__ __forceinline__ void fused_cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void fused_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

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

// This warp's weights for one row group of 16 output channels: CW chunks of 64 bytes of rows g and
// g + 8 (a row past the end repeats the last one).  K = 1024 * CW.
template <int CW>
__device__ __forceinline__ void fused_load_weights(uint4 (&w)[CW][2], const uint8_t* __restrict__ Wq, int N, int group,
                                                   int warp, int g, int t) {
  constexpr int64_t row_bytes = 1024 * CW / 2;
  const uint8_t* r0 = Wq + int64_t(min(group * 16 + g, N - 1)) * row_bytes + t * 16;
  const uint8_t* r1 = Wq + int64_t(min(group * 16 + 8 + g, N - 1)) * row_bytes + t * 16;
#pragma unroll
  for (int u = 0; u < CW; ++u) {
    const int cc = warp + u * kFusedWarps;
    w[u][0] = load_stream_16(r0 + cc * 64);
    w[u][1] = load_stream_16(r1 + cc * 64);
  }
}

// The product phase shared by the fused kernels: row groups `group`, group + gridDim.x, ... against the
// tokens' codes in shared memory (xs: per token the even-position and the odd-position plane of int8
// lanes, K / 8 words each; tokens past M contribute zeros); rows g, g + 8 of a group against token g;
// the next group's weights are in flight during the products.  `w` holds the first group's weights.
template <int CW>
__device__ __forceinline__ void fused_products(const uint32_t* xs, const float* sdx, int (*red)[128], uint4 (&w)[CW][2],
                                               int group, int groups, const uint8_t* __restrict__ Wq, int M, int N,
                                               const float* __restrict__ dw, __half* __restrict__ Y, int64_t ldy) {
  constexpr int kPlane = 1024 * CW / 8;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int out_m = tid >> 4;                             // the token of the output this thread finishes (tid < 128)
  const bool live = g < M;
  const uint32_t* xe = xs + (live ? g : 0) * 2 * kPlane;
  const uint32_t* xo = xe + kPlane;
  uint4 w_next[CW][2];
  for (; group < groups; group += gridDim.x) {
    const int next = group + gridDim.x;
    if (next < groups) fused_load_weights<CW>(w_next, Wq, N, next, warp, g, t);
    const int out_n = group * 16 + (tid & 15);
    const float out_dw = (tid < 128 && out_n < N) ? __ldg(dw + out_n) : 0.0f;
    int c[4] = {0, 0, 0, 0};
#pragma unroll
    for (int u = 0; u < CW; ++u) {
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
    for (int u = 0; u < CW; ++u) {
      w[u][0] = w_next[u][0];
      w[u][1] = w_next[u][1];
    }
  }
}

// Export of the packed codes (CTA 0 only): byte i of a row = code 2i (bits 0-3) | code 2i + 1 (bits 4-7);
// codes 2i and 2i + 1 sit in lane i of the two planes.
__device__ __forceinline__ void fused_export_codes(const uint32_t* xs, int M, int K, uint8_t* __restrict__ xq_out) {
  const uint8_t* lanes = reinterpret_cast<const uint8_t*>(xs);
  for (int idx = threadIdx.x; idx < M * (K / 2); idx += kFusedThreads) {
    const int m = idx / (K / 2), i = idx - m * (K / 2);
    const uint8_t even = lanes[(m * 2) * (K / 2) + i], odd = lanes[(m * 2 + 1) * (K / 2) + i];
    xq_out[int64_t(m) * (K / 2) + i] = uint8_t((even >> 4) | (odd & 0xF0u));
  }
}

__global__ void __launch_bounds__(kFusedThreads, 2)
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
  const int groups = (N + 15) >> 4;                       // row groups of 16 output channels

  // 1. the weights of the first row group are on their way before anything else
  uint4 w[kFusedChunksPerWarp][2];
  const int group = blockIdx.x;
  if (group < groups) fused_load_weights<kFusedChunksPerWarp>(w, Wq, N, group, warp, g, t);

  // 2. the tokens: rotate, quantize, leave the codes in shared memory
  // all tokens' values are requested at once: one trip to L2 instead of one per token
  uint4 raw_all[kFusedMaxTokens][2];
#pragma unroll
  for (int m = 0; m < kFusedMaxTokens; ++m) {
    const uint4* src = reinterpret_cast<const uint4*>(X + int64_t(m < M ? m : 0) * ldx + tid * 16);
    raw_all[m][0] = __ldg(src);
    raw_all[m][1] = __ldg(src + 1);
  }
  float4 scale[4];                                     // the diagonal of this thread's 16 values, once for all tokens
#pragma unroll
  for (int k = 0; k < 4; ++k)
    scale[k] = pre != nullptr ? __ldg(reinterpret_cast<const float4*>(pre + tid * 16) + k) : make_float4(1.f, 1.f, 1.f, 1.f);
  // With several tokens the CTAs of a cluster divide them (token m is rotated by the CTA of rank
  // m mod size) and fetch each other's codes through the cluster's shared-memory window afterwards.
  const uint32_t crank = fused_cluster_rank(), csize = fused_cluster_size();
#pragma unroll
  for (int m = 0; m < kFusedMaxTokens; ++m) {
    if (m >= M) break;
    if (uint32_t(m) % csize != crank) continue;
    float v[16];
    {
      const uint4 a = raw_all[m][0], b = raw_all[m][1];
      const uint32_t raw[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int k = 0; k < 8; ++k) unpack2(half2_to_f32x2(raw[k]), v[2 * k], v[2 * k + 1]);
      if (pre != nullptr) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float4 s = scale[k];
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
  if (csize > 1) {
    fused_cluster_arrive();               // this CTA's tokens are in its shared memory ...
    fused_cluster_wait();                 // ... and so are everybody else's
    for (int m = 0; m < M; ++m) {
      const uint32_t owner = uint32_t(m) % csize;
      if (owner == crank) continue;
      const uint32_t src = fused_peer_address(&xs[m][0][0], owner);
      uint4* dst = reinterpret_cast<uint4*>(&xs[m][0][0]);
      for (int i = tid; i < 2 * (K / 8) / 4; i += kFusedThreads) {
        uint4 val;
        asm volatile("ld.shared::cluster.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(src + uint32_t(i) * 16u) : "memory");
        dst[i] = val;
      }
      if (tid == 0) {
        float st;
        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(st) : "r"(fused_peer_address(&sdx[m], owner)) : "memory");
        sdx[m] = st;
        if (blockIdx.x == 0 && dx_out != nullptr) dx_out[m] = st;
      }
    }
    __syncthreads();
    fused_cluster_arrive();               // done reading the others' shared memory (waited for before leaving)
  }
  if (blockIdx.x == 0 && xq_out != nullptr) fused_export_codes(&xs[0][0][0], M, K, xq_out);

  // 3. the products, row group after row group
  fused_products<kFusedChunksPerWarp>(&xs[0][0][0], sdx, red, w, group, groups, Wq, M, N, dw, Y, ldy);
  if (csize > 1) fused_cluster_wait();    // nobody leaves while its shared memory may still be read
}

// The same layer for inputs that need no online rotation (every quantized layer quantizes its input
// online, only two rotate it first): x * pre, per-token INT4 with the correctly rounded quotient of
// smoothrot_quant_act_plain, then the products.  Quantizing a token is a few dozen instructions per
// thread, so up to 8 tokens (one token tile of the MMA) are taken.  K = 1024 * CW.
template <int CW>
__global__ void __launch_bounds__(kFusedThreads, 2)
fused_plain_decode_kernel(const __half* __restrict__ X, int M, int64_t ldx, const float* __restrict__ pre, float clip,
                          const uint8_t* __restrict__ Wq, int N, const float* __restrict__ dw,
                          __half* __restrict__ Y, int64_t ldy, uint8_t* __restrict__ xq_out,
                          float* __restrict__ dx_out) {
  constexpr int K = 1024 * CW;
  constexpr int kTokens = 8;
  constexpr int kChunks = K / 8;                                   // chunks of 8 values = packed words of a row
  constexpr int kPerThread = (kChunks + kFusedThreads - 1) / kFusedThreads;
  __shared__ __align__(16) uint32_t xs[kTokens][2][kChunks];      // int8 lanes (16 * code): even / odd positions
  __shared__ float sred[kFusedWarps];
  __shared__ float sdx[kTokens];
  __shared__ int red[kFusedWarps][128];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int groups = (N + 15) >> 4;
  uint4 w[CW][2];
  const int group = blockIdx.x;
  if (group < groups) fused_load_weights<CW>(w, Wq, N, group, warp, g, t);

  // a token's values are requested while the token before it is quantized (the loop over the tokens
  // is kept rolled: unrolled, every token runs its own copy of the code and waits for it to be fetched)
  auto fetch = [&](uint4 (&raw)[kPerThread], int m) {
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int c = tid + i * kFusedThreads;
      raw[i] = c < kChunks ? __ldg(reinterpret_cast<const uint4*>(X + int64_t(m) * ldx) + c) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  uint4 raw_next[kPerThread];
  fetch(raw_next, 0);
  // the diagonal of this thread's chunks, once for all tokens
  f32x2 scale[kPerThread][4];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int c = tid + i * kFusedThreads;
    float4 a = make_float4(1.f, 1.f, 1.f, 1.f), b = a;
    if (pre != nullptr && c < kChunks) {
      a = __ldg(reinterpret_cast<const float4*>(pre) + 2 * c);
      b = __ldg(reinterpret_cast<const float4*>(pre) + 2 * c + 1);
    }
    scale[i][0] = pack2(a.x, a.y);
    scale[i][1] = pack2(a.z, a.w);
    scale[i][2] = pack2(b.x, b.y);
    scale[i][3] = pack2(b.z, b.w);
  }
#pragma unroll 1
  for (int m = 0; m < M; ++m) {
    uint4 raw_cur[kPerThread];
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) raw_cur[i] = raw_next[i];
    if (m + 1 < M) fetch(raw_next, m + 1);
    f32x2 v[kPerThread][4];
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const uint4 raw = raw_cur[i];
      v[i][0] = half2_to_f32x2(raw.x);
      v[i][1] = half2_to_f32x2(raw.y);
      v[i][2] = half2_to_f32x2(raw.z);
      v[i][3] = half2_to_f32x2(raw.w);
      if (pre != nullptr) {
#pragma unroll
        for (int k = 0; k < 4; ++k) v[i][k] = mul2(v[i][k], scale[i][k]);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float a, b;
        unpack2(v[i][k], a, b);
        amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
      }
    }
    amax = warp_max(amax);
    __syncthreads();                                    // sred of the previous token has been read
    if (lane == 0) sred[warp] = amax;
    __syncthreads();
    amax = sred[0];
#pragma unroll
    for (int k = 1; k < kFusedWarps; ++k) amax = fmaxf(amax, sred[k]);
    const float step = step_from_absmax(amax, clip);
    if (tid == 0) {
      sdx[m] = step;
      if (blockIdx.x == 0 && dx_out != nullptr) dx_out[m] = step;
    }
    // the correctly rounded fp32 quotient x / step (reciprocal, one residual correction), rounded half
    // to even by the 1.5 * 2^23 constant, clamped to [-8, 7]; an int8 lane is 16 * code
    const float inv = __frcp_rn(step);
    const f32x2 inv2 = pack2(inv, inv), neg_step2 = pack2(-step, -step), magic2 = pack2(12582912.0f, 12582912.0f);
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int c = tid + i * kFusedThreads;
      uint32_t even[4], odd[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        f32x2 q = mul2(v[i][k], inv2);
        q = fma2(fma2(q, neg_step2, v[i][k]), inv2, q);
        float q0, q1;
        unpack2(add2(q, magic2), q0, q1);
        q0 = fmaxf(fminf(q0, 12582912.0f + 7.0f), 12582912.0f - 8.0f);
        q1 = fmaxf(fminf(q1, 12582912.0f + 7.0f), 12582912.0f - 8.0f);
        even[k] = __float_as_uint(q0) << 4;
        odd[k] = __float_as_uint(q1) << 4;
      }
      if (c < kChunks) {
        xs[m][0][c] = __byte_perm(__byte_perm(even[0], even[1], 0x0040), __byte_perm(even[2], even[3], 0x0040), 0x5410);
        xs[m][1][c] = __byte_perm(__byte_perm(odd[0], odd[1], 0x0040), __byte_perm(odd[2], odd[3], 0x0040), 0x5410);
      }
    }
  }
  __syncthreads();
  if (blockIdx.x == 0 && xq_out != nullptr) fused_export_codes(&xs[0][0][0], M, K, xq_out);
  fused_products<CW>(&xs[0][0][0], sdx, red, w, group, groups, Wq, M, N, dw, Y, ldy);
}

// The same layer for the attention output projection: the tokens go through the head-mixing
// transform of smoothrot_quant_act_heads, (x * pre)(H_32 (x) I_128) / sqrt(32), 5 butterfly stages.
// 64 threads rotate one token (a thread owns two neighbouring positions of every head, as in
// heads_quant.cu), so the four groups of the CTA take up to four tokens side by side.
__global__ void __launch_bounds__(kFusedThreads, 2)
fused_heads_decode_kernel(const __half* __restrict__ X, int M, int64_t ldx, const float* __restrict__ pre, float clip,
                          bool low_clamp, const uint8_t* __restrict__ Wq, int N, const float* __restrict__ dw,
                          __half* __restrict__ Y, int64_t ldy, uint8_t* __restrict__ xq_out,
                          float* __restrict__ dx_out) {
  constexpr int K = kFusedK, NH = 32, HD = 128, CW = kFusedChunksPerWarp;
  __shared__ __align__(16) uint32_t xs[kFusedMaxTokens][2][K / 8];
  __shared__ float sred[kFusedWarps];
  __shared__ float sdx[kFusedMaxTokens];
  __shared__ int red[kFusedWarps][128];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int groups = (N + 15) >> 4;
  uint4 w[CW][2];
  const int group = blockIdx.x;
  if (group < groups) fused_load_weights<CW>(w, Wq, N, group, warp, g, t);

  const int m = tid >> 6;                 // the token this thread works on
  const int p = tid & 63;                 // it owns positions 2p, 2p + 1 of every head
  const bool have = m < M;
  f32x2 v[NH];
  {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(X + int64_t(have ? m : 0) * ldx) + p;
#pragma unroll
    for (int h = 0; h < NH; ++h) v[h] = half2_to_f32x2(__ldg(src + h * (HD / 2)));
    if (pre != nullptr) {
      const float2* ps = reinterpret_cast<const float2*>(pre) + p;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const float2 sc = __ldg(ps + h * (HD / 2));
        v[h] = mul2(v[h], pack2(sc.x, sc.y));
      }
    }
  }
#pragma unroll
  for (int hb = 1; hb < NH; hb <<= 1) {
#pragma unroll
    for (int k = 0; k < NH; ++k) {
      if ((k & hb) == 0) {
        const f32x2 a = v[k], b = v[k + hb];
        v[k] = add2(a, b);
        v[k + hb] = sub2(a, b);
      }
    }
  }
  float amax = 0.0f;
#pragma unroll
  for (int h = 0; h < NH; ++h) {
    float a, b;
    unpack2(v[h], a, b);
    amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
  }
  amax = warp_max(amax);
  if (lane == 0) sred[warp] = amax;
  __syncthreads();
  amax = fmaxf(sred[2 * m], sred[2 * m + 1]) * 0.17677669529663687f;    // 1 / sqrt(32): the normalised maximum
  const float step = step_from_absmax(amax, clip);
  if (p == 0 && have) {
    sdx[m] = step;
    if (blockIdx.x == 0 && dx_out != nullptr) dx_out[m] = step;
  }
  if (have) {
    const float inv = __frcp_rn(step) * 0.17677669529663687f;           // 1 / step for the unnormalised values
    uint8_t* even = reinterpret_cast<uint8_t*>(&xs[m][0][0]);
    uint8_t* odd = reinterpret_cast<uint8_t*>(&xs[m][1][0]);
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      float a, b;
      unpack2(v[h], a, b);
      float q0 = __fmaf_rn(a, inv, 12582912.0f), q1 = __fmaf_rn(b, inv, 12582912.0f);
      q0 = low_clamp ? fmaxf(fminf(q0, 12582912.0f + 7.0f), 12582912.0f - 8.0f) : fminf(q0, 12582912.0f + 7.0f);
      q1 = low_clamp ? fmaxf(fminf(q1, 12582912.0f + 7.0f), 12582912.0f - 8.0f) : fminf(q1, 12582912.0f + 7.0f);
      // position j = h * 128 + 2p (even) and j + 1: lane h * 64 + p of the even / odd plane
      even[h * (HD / 2) + p] = uint8_t(__float_as_uint(q0) << 4);
      odd[h * (HD / 2) + p] = uint8_t(__float_as_uint(q1) << 4);
    }
  }
  __syncthreads();
  if (blockIdx.x == 0 && xq_out != nullptr) fused_export_codes(&xs[0][0][0], M, K, xq_out);
  fused_products<CW>(&xs[0][0][0], sdx, red, w, group, groups, Wq, M, N, dw, Y, ldy);
}

}  // namespace
}  // namespace gemm
}  // namespace smoothrot

extern "C" {

int smoothrot_linear_decode(const void* X_f16, int64_t M, int64_t K, int64_t ldx, int rotation, const float* pre,
                            float clip_a, const uint8_t* Wq, const float* dw, int64_t N, void* Y_f16, int64_t ldy,
                            uint8_t* Xq_out, float* dx_out, void* stream) {
  using namespace smoothrot;
  using namespace smoothrot::gemm;
  if (M < 0 || N < 0 || K <= 0 || (rotation != 0 && rotation != 1)) return SMOOTHROT_INVALID_ARG;
  if (!(clip_a > 0.0f) || clip_a > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (rotation ? K != kFusedK : (K != 1024 && K != 2048 && K != 4096)) return SMOOTHROT_UNSUPPORTED_K;
  if (M > (rotation ? kFusedMaxTokens : 8) || N % 8 != 0 || N > 0x3fffffffLL) return SMOOTHROT_INVALID_ARG;
  if (M == 0 || N == 0) return SMOOTHROT_OK;
  if (X_f16 == nullptr || Wq == nullptr || dw == nullptr || Y_f16 == nullptr || ldx < K || ldy < N)
    return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X_f16) || ldx % 8 != 0 || !aligned16(Wq) || (pre != nullptr && !aligned16(pre)))
    return SMOOTHROT_BAD_ALIGNMENT;
  // every CTA prepares the tokens once, so there are no more CTAs than fit the machine at a time
  // (2 per SM), each taking the same number of row groups
  const int64_t groups = (N + 15) / 16;
  const int64_t slots = int64_t(device_sm_count()) * 2;
  const int64_t per_cta = (groups + slots - 1) / slots;
  const unsigned grid = unsigned((groups + per_cta - 1) / per_cta);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __half* x = static_cast<const __half*>(X_f16);
  __half* y = static_cast<__half*>(Y_f16);
  if (rotation) {
    const bool low = 7.0f / clip_a >= 8.49f;             // codes below -8 can only come up then
    // several tokens: clusters of 2 or 4 CTAs share the rotations (the grid is rounded up to whole
    // clusters; a CTA without row groups still rotates its tokens for the others)
    const unsigned cs = M >= 3 ? 4u : (M == 2 ? 2u : 1u);
    if (cs > 1) {
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3((grid + cs - 1) / cs * cs, 1, 1);
      cfg.blockDim = dim3(kFusedThreads, 1, 1);
      cfg.dynamicSmemBytes = 0;
      cfg.stream = st;
      cudaLaunchAttribute attr{};
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = cs;
      attr.val.clusterDim.y = 1;
      attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      const int m_int = int(M), n_int = int(N);
      if (cudaLaunchKernelEx(&cfg, fused_decode_kernel, x, m_int, ldx, pre, clip_a, low, Wq, n_int, dw, y, ldy, Xq_out,
                             dx_out) != cudaSuccess) {
        (void)cudaGetLastError();
        return SMOOTHROT_CUDA_ERROR;
      }
    } else {
      fused_decode_kernel<<<grid, kFusedThreads, 0, st>>>(x, int(M), ldx, pre, clip_a, low, Wq, int(N), dw, y, ldy,
                                                          Xq_out, dx_out);
    }
  } else if (K == 4096) {
    fused_plain_decode_kernel<4><<<grid, kFusedThreads, 0, st>>>(x, int(M), ldx, pre, clip_a, Wq, int(N), dw, y, ldy,
                                                                 Xq_out, dx_out);
  } else if (K == 2048) {
    fused_plain_decode_kernel<2><<<grid, kFusedThreads, 0, st>>>(x, int(M), ldx, pre, clip_a, Wq, int(N), dw, y, ldy,
                                                                 Xq_out, dx_out);
  } else {
    fused_plain_decode_kernel<1><<<grid, kFusedThreads, 0, st>>>(x, int(M), ldx, pre, clip_a, Wq, int(N), dw, y, ldy,
                                                                 Xq_out, dx_out);
  }
  count_launch();
  return launch_status();
}

int smoothrot_linear_decode_heads(const void* X_f16, int64_t M, int64_t n_heads, int64_t head_dim, int64_t ldx,
                                  const float* pre, float clip_a, const uint8_t* Wq, const float* dw, int64_t N,
                                  void* Y_f16, int64_t ldy, uint8_t* Xq_out, float* dx_out, void* stream) {
  using namespace smoothrot;
  using namespace smoothrot::gemm;
  if (M < 0 || N < 0 || n_heads <= 0 || head_dim <= 0) return SMOOTHROT_INVALID_ARG;
  if (!(clip_a > 0.0f) || clip_a > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (n_heads != 32 || head_dim != 128) return SMOOTHROT_UNSUPPORTED_K;
  if (M > kFusedMaxTokens || N % 8 != 0 || N > 0x3fffffffLL) return SMOOTHROT_INVALID_ARG;
  if (M == 0 || N == 0) return SMOOTHROT_OK;
  const int64_t K = n_heads * head_dim;
  if (X_f16 == nullptr || Wq == nullptr || dw == nullptr || Y_f16 == nullptr || ldx < K || ldy < N)
    return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X_f16) || ldx % 8 != 0 || !aligned16(Wq) || (pre != nullptr && !aligned16(pre)))
    return SMOOTHROT_BAD_ALIGNMENT;
  const bool low = 7.0f / clip_a >= 8.49f;
  const int64_t groups = (N + 15) / 16;
  const int64_t slots = int64_t(device_sm_count()) * 2;
  const int64_t per_cta = (groups + slots - 1) / slots;
  const unsigned grid = unsigned((groups + per_cta - 1) / per_cta);
  fused_heads_decode_kernel<<<grid, kFusedThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __half*>(X_f16), int(M), ldx, pre, clip_a, low, Wq, int(N), dw, static_cast<__half*>(Y_f16), ldy,
      Xq_out, dx_out);
  count_launch();
  return launch_status();
}

}  // extern "C"
