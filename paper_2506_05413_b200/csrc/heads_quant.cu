// Head-mixing online transform of libsmoothrot:  v = (x * pre) (H_heads (x) I_head_dim) / sqrt(heads),
// followed by the per-token symmetric 4-bit quantizer of the activation path.
//
// Methodology section: the forward pass contains two online Hadamard transforms, for which the paper
// defers to QuaRot.  The one in front of the down-projection is the full rotation of
// rotate_quant.cu; this is the other one, in front of the attention output projection, where the
// per-head factor of the rotation is folded into the value projection offline and only the mixing of
// the heads is left for the forward pass.
//
// The transform touches log2(heads) butterfly stages only (5 for 32 heads, against 12 for a full
// 4096-point rotation), and every butterfly joins values that sit head_dim apart.  So a thread owns two
// neighbouring positions of *every* head: it loads heads x 4 bytes with a stride of one head (a warp
// reads 128 contiguous bytes per head), holds the heads x 2 values as packed fp32 pairs, and runs all
// stages in registers with packed add/sub; there is no shared-memory transpose and no staging buffer.
// head_dim / 2 threads cover a row; they meet once, for the row maximum.  The next row's loads are in
// flight while the current row is transformed.  Codes leave as 32-bit words after a 4 x 4 byte transpose
// among neighbouring lanes (a lane's four heads against four lanes' positions).
#include <math.h>

#include <type_traits>

#include "common.cuh"
#include "rowquant.cuh"

namespace smoothrot {
namespace {

constexpr int kHeadsThreads = 256;

// Walsh butterflies over the index of the pairs (natural order): log2(NP) stages of packed add/sub.
template <int NP>
__device__ __forceinline__ void butterflies_over_heads(f32x2* v) {
#pragma unroll
  for (int h = 1; h < NP; h <<= 1) {
#pragma unroll
    for (int k = 0; k < NP; ++k) {
      if ((k & h) == 0) {
        const f32x2 a = v[k], b = v[k + h];
        v[k] = add2(a, b);
        v[k + h] = sub2(a, b);
      }
    }
  }
}

__device__ __forceinline__ void group_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// kQuant: codes + step sizes; otherwise the rotated row as fp32 (test export).
// kLowClamp: the general two-sided clamp, needed when the row maximum can reach 8.5 steps or more.
// HD (head_dim) is a template parameter so that the strides between heads are immediates; the
// diagonal and the clamp are uniform run-time branches.
template <int NH, int HD, bool kQuant>
__global__ void __launch_bounds__(kHeadsThreads, NH <= 32 ? 2 : 1)
heads_kernel(const __half* __restrict__ x, int64_t ld, int rows, const float* __restrict__ pre, bool low_clamp,
             float inv_sqrt_heads, float clip, uint8_t* __restrict__ q_out, float* __restrict__ step_out,
             float* __restrict__ y_out) {
  __shared__ float red[kHeadsThreads / 32];
  constexpr int head_dim = HD;
  constexpr int group_threads = head_dim >> 1;             // threads per row: 32, 64 or 128
  constexpr int groups = kHeadsThreads / group_threads;
  const bool kHasPre = pre != nullptr;
  const bool kLowClamp = low_clamp;
  const int group = threadIdx.x / group_threads;
  const int t = threadIdx.x - group * group_threads;       // this thread owns positions 2t, 2t + 1 of every head
  constexpr int warps = group_threads >> 5;
  const int row_stride = gridDim.x * groups;
  constexpr int K = NH * head_dim;

  uint32_t raw[NH];
  int m = blockIdx.x * groups + group;
  if (m < rows) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(x + int64_t(m) * ld) + t;
#pragma unroll
    for (int h = 0; h < NH; ++h) raw[h] = __ldcs(src + h * group_threads);
  }
  for (; m < rows; m += row_stride) {
    f32x2 v[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) v[h] = half2_to_f32x2(raw[h]);
    // the next row of this group is on its way during the arithmetic
    const int next = m + row_stride;
    if (next < rows) {
      const uint32_t* src = reinterpret_cast<const uint32_t*>(x + int64_t(next) * ld) + t;
#pragma unroll
      for (int h = 0; h < NH; ++h) raw[h] = __ldcs(src + h * group_threads);
    }
    if (kHasPre) {
      const float2* p = reinterpret_cast<const float2*>(pre) + t;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const float2 s = __ldg(p + h * group_threads);
        v[h] = mul2(v[h], pack2(s.x, s.y));
      }
    }
    butterflies_over_heads<NH>(v);

    if (!kQuant) {
      float2* y = reinterpret_cast<float2*>(y_out + int64_t(m) * K) + t;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        float a, b;
        unpack2(v[h], a, b);
        y[h * group_threads] = make_float2(a * inv_sqrt_heads, b * inv_sqrt_heads);
      }
      continue;
    }

    float amax = 0.0f;
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      float a, b;
      unpack2(v[h], a, b);
      amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
    }
    amax = warp_max(amax);
    if (warps > 1) {
      const int w0 = group * warps;
      if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
      group_sync(1 + group, group_threads);
      amax = red[w0];
      for (int w = 1; w < warps; ++w) amax = fmaxf(amax, red[w0 + w]);
      group_sync(1 + group, group_threads);             // red is written again by the next row
    }
    amax *= inv_sqrt_heads;                              // the maximum of the normalised row
    const float step = step_from_absmax(amax, clip);
    if (t == 0) step_out[m] = step;
    const float inv = __frcp_rn(step) * inv_sqrt_heads;  // 1 / step for the unnormalised values
    const f32x2 inv2 = pack2(inv, inv);

    // Round to nearest even and bias by 8: the low byte of the float's bit pattern is code + 8.
    const float kMagic = 12582912.0f + 8.0f;             // 1.5 * 2^23 + 8
    const f32x2 magic2 = pack2(kMagic, kMagic);
    const int r = t & 3;
    const uint32_t sel1 = (r & 1) ? 0x3715u : 0x6240u;   // 4 x 4 byte transpose, step 1 (own = a, partner = b)
    const uint32_t sel2 = (r & 2) ? 0x3276u : 0x5410u;   // step 2
    uint8_t* q_row = q_out + int64_t(m) * (K >> 1) + (t & ~3);
#pragma unroll
    for (int j = 0; j < NH / 4; ++j) {
      uint32_t lo[4], hi[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float q0, q1;
        unpack2(fma2(v[4 * j + k], inv2, magic2), q0, q1);
        if (kLowClamp) {
          q0 = fmaxf(fminf(q0, 12582912.0f + 15.0f), 12582912.0f);
          q1 = fmaxf(fminf(q1, 12582912.0f + 15.0f), 12582912.0f);
        }
        lo[k] = __float_as_uint(q0);
        hi[k] = __float_as_uint(q1);
      }
      // byte k of each word: head 4j + k; `even` holds position 2t, `odd` position 2t + 1
      uint32_t even = __byte_perm(__byte_perm(lo[0], lo[1], 0x0040), __byte_perm(lo[2], lo[3], 0x0040), 0x5410);
      uint32_t odd = __byte_perm(__byte_perm(hi[0], hi[1], 0x0040), __byte_perm(hi[2], hi[3], 0x0040), 0x5410);
      if (!kLowClamp) {
        // the row maximum sits below 8.5 steps: a byte is code + 8 in [0, 16], and 16 comes down to 15
        even -= (even >> 4) & 0x01010101u;
        odd -= (odd >> 4) & 0x01010101u;
      }
      uint32_t w = (even | (odd << 4)) ^ 0x88888888u;    // offset binary -> two's complement nibbles
      // lanes t = 4q .. 4q + 3 hold output bytes 4q .. 4q + 3 of heads 4j .. 4j + 3: transpose so that
      // lane r gets the aligned word of head 4j + r
      uint32_t p = __shfl_xor_sync(0xffffffffu, w, 1);
      w = __byte_perm(w, p, sel1);
      p = __shfl_xor_sync(0xffffffffu, w, 2);
      w = __byte_perm(w, p, sel2);
      *reinterpret_cast<uint32_t*>(q_row + (4 * j + r) * group_threads) = w;
    }
  }
}

template <bool kQuant>
int launch_heads(const void* X, int64_t rows, int64_t n_heads, int64_t head_dim, int64_t ld, const float* pre,
                 float clip, uint8_t* q_out, float* step_out, float* y_out, cudaStream_t stream) {
  if (rows < 0 || n_heads <= 0 || head_dim <= 0) return SMOOTHROT_INVALID_ARG;
  if (!(n_heads == 8 || n_heads == 16 || n_heads == 32 || n_heads == 64) ||
      !(head_dim == 64 || head_dim == 128 || head_dim == 256))
    return SMOOTHROT_UNSUPPORTED_K;
  if (rows == 0) return SMOOTHROT_OK;
  const int64_t K = n_heads * head_dim;
  if (X == nullptr || ld < K || rows > 0x7fffffffLL) return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X) || (ld % 8) != 0 || (pre != nullptr && !aligned16(pre))) return SMOOTHROT_BAD_ALIGNMENT;
  const bool low = kQuant && (7.0f / clip >= 8.49f);
  const float rs = float(1.0 / sqrt(double(n_heads)));
  const int groups = kHeadsThreads / int(head_dim / 2);
  const int ctas_per_sm = n_heads <= 32 ? 2 : 1;
  int64_t grid = (rows + groups - 1) / groups;
  const int64_t cap = int64_t(device_sm_count()) * ctas_per_sm;
  if (grid > cap) grid = cap;
  auto launch = [&](auto kern) {
    kern<<<unsigned(grid), kHeadsThreads, 0, stream>>>(static_cast<const __half*>(X), ld, int(rows), pre, low, rs, clip,
                                                      q_out, step_out, y_out);
    count_launch();
    return launch_status();
  };
  auto pick = [&](auto nh_tag) {
    constexpr int NH = decltype(nh_tag)::value;
    switch (int(head_dim)) {
      case 64: return launch(heads_kernel<NH, 64, kQuant>);
      case 128: return launch(heads_kernel<NH, 128, kQuant>);
      default: return launch(heads_kernel<NH, 256, kQuant>);
    }
  };
  switch (int(n_heads)) {
    case 8: return pick(std::integral_constant<int, 8>{});
    case 16: return pick(std::integral_constant<int, 16>{});
    case 32: return pick(std::integral_constant<int, 32>{});
    default: return pick(std::integral_constant<int, 64>{});
  }
}

}  // namespace
}  // namespace smoothrot

extern "C" {

int smoothrot_quant_act_heads(const void* X_f16, int64_t M, int64_t n_heads, int64_t head_dim, int64_t ldx,
                              const float* pre, float clip_a, uint8_t* Xq_out, float* dx_out, void* stream) {
  if (!(clip_a > 0.0f) || clip_a > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (M > 0 && (Xq_out == nullptr || dx_out == nullptr)) return SMOOTHROT_INVALID_ARG;
  if (M > 0 && !smoothrot::aligned16(Xq_out)) return SMOOTHROT_BAD_ALIGNMENT;
  return smoothrot::launch_heads<true>(X_f16, M, n_heads, head_dim, ldx, pre, clip_a, Xq_out, dx_out, nullptr,
                                       static_cast<cudaStream_t>(stream));
}

int smoothrot_debug_hadamard_heads(const void* X_f16, int64_t M, int64_t n_heads, int64_t head_dim, int64_t ldx,
                                   const float* pre, float* Y_f32, void* stream) {
  if (M > 0 && Y_f32 == nullptr) return SMOOTHROT_INVALID_ARG;
  if (M > 0 && !smoothrot::aligned16(Y_f32)) return SMOOTHROT_BAD_ALIGNMENT;
  return smoothrot::launch_heads<false>(X_f16, M, n_heads, head_dim, ldx, pre, 1.0f, nullptr, nullptr, Y_f32,
                                        static_cast<cudaStream_t>(stream));
}

}  // extern "C"
