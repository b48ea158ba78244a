// Weight quantization with the clip-ratio search of the paper's weight quantizer
// (Experimental settings, "Quantization": per-channel symmetric 4-bit weights, each clip ratio
// being the candidate with the least squared quantization error).
//
// Offline path, built for clarity rather than speed: the rows are rotated by the same kernels
// as smoothrot_fuse_weights (through the fp32 export) into the caller's workspace, then one CTA
// per row tries every ratio of the grid  1, 1 - d, ..., lowest  on the fp32 row held in shared
// memory: Eq. 1's symmetric quantizer with step = fp32(ratio * max|w^|) / 7 (fp32 decisions),
// squared error accumulated in fp64 in a fixed order, first minimum kept.
#include "common.cuh"

namespace smoothrot {

constexpr int kSearchThreads = 256;

__device__ __forceinline__ double block_sum(double v, double* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double total = 0.0;
#pragma unroll
  for (int w = 0; w < kSearchThreads / 32; ++w) total += red[w];
  __syncthreads();
  return total;
}

__global__ void __launch_bounds__(kSearchThreads)
clip_search_kernel(const float* __restrict__ rotated, int64_t row0, int K, double lowest, int count,
                   uint8_t* __restrict__ q_out, float* __restrict__ step_out, int32_t* __restrict__ best_out) {
  extern __shared__ __align__(16) float row[];
  __shared__ double red[kSearchThreads / 32];
  __shared__ float red_max[kSearchThreads / 32];
  const int tid = threadIdx.x;
  const int64_t m = row0 + blockIdx.x;
  const float* src = rotated + int64_t(blockIdx.x) * K;

  float amax = 0.0f;
  for (int j = tid; j < K; j += kSearchThreads) {
    const float v = src[j];
    row[j] = v;
    amax = fmaxf(amax, fabsf(v));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((tid & 31) == 0) red_max[tid >> 5] = amax;
  __syncthreads();
  amax = red_max[0];
#pragma unroll
  for (int w = 1; w < kSearchThreads / 32; ++w) amax = fmaxf(amax, red_max[w]);

  double best_err = 0.0;
  float best_step = 1.0f;
  int best = 0;
  for (int i = 0; i < count; ++i) {
    // the grid in fp64, rounded to fp32: 1 - i * (1 - lowest) / (count - 1)
    const float ratio = count > 1 ? float(1.0 - double(i) * (1.0 - lowest) / double(count - 1)) : 1.0f;
    const float step = amax == 0.0f ? 1.0f : __fdiv_rn(__fmul_rn(ratio, amax), 7.0f);
    double err = 0.0;
    for (int j = tid; j < K; j += kSearchThreads) {
      const float v = row[j];
      const float q = fminf(fmaxf(rintf(__fdiv_rn(v, step)), -8.0f), 7.0f);
      const double d = double(v) - double(q) * double(step);
      err = fma(d, d, err);
    }
    err = block_sum(err, red);
    if (i == 0 || err < best_err) {   // every thread holds the same sums: the choice is uniform
      best_err = err;
      best_step = step;
      best = i;
    }
  }
  if (tid == 0) {
    step_out[m] = best_step;
    if (best_out != nullptr) best_out[m] = best;
  }
  uint32_t* q = reinterpret_cast<uint32_t*>(q_out + m * int64_t(K / 2));
  for (int c = tid; c < K / 8; c += kSearchThreads) {
    uint32_t word = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float t = rintf(__fdiv_rn(row[c * 8 + i], best_step));
      t = fminf(fmaxf(t, -8.0f), 7.0f);
      word |= (uint32_t(int(t)) & 0xFu) << (4 * i);
    }
    q[c] = word;
  }
}

}  // namespace smoothrot

extern "C" {

size_t smoothrot_fuse_weights_search_workspace_bytes(int64_t N, int64_t K) {
  if (N <= 0 || K <= 0) return 0;
  // the rotated fp32 rows; a smaller workspace (a multiple of one row) makes the call work in slices
  return size_t(N) * size_t(K) * sizeof(float);
}

int smoothrot_fuse_weights_search(const void* W_f16, int64_t N, int64_t K, int64_t ldw, const float* pre,
                                  float lowest_ratio, int ratio_count, uint8_t* Wq_out, float* dw_out,
                                  int32_t* best_out, void* workspace, size_t workspace_bytes, void* stream) {
  using namespace smoothrot;
  if (N < 0 || K <= 0) return SMOOTHROT_INVALID_ARG;
  int base = 0, n = 0, logn = 0;
  if (!split_order(K, &base, &n, &logn)) return SMOOTHROT_UNSUPPORTED_K;
  if (!(lowest_ratio > 0.0f) || lowest_ratio > 1.0f || ratio_count < 1 || ratio_count > 1024)
    return SMOOTHROT_INVALID_ARG;
  if (N == 0) return SMOOTHROT_OK;
  if (W_f16 == nullptr || Wq_out == nullptr || dw_out == nullptr || ldw < K) return SMOOTHROT_INVALID_ARG;
  if (!aligned16(W_f16) || ldw % 8 != 0 || !aligned16(Wq_out)) return SMOOTHROT_BAD_ALIGNMENT;
  const size_t row_bytes = size_t(K) * sizeof(float);
  if (workspace == nullptr || workspace_bytes < row_bytes) return SMOOTHROT_WORKSPACE_TOO_SMALL;
  if (!aligned16(workspace)) return SMOOTHROT_BAD_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto kern = clip_search_kernel;
  if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), int(row_bytes)))
    return SMOOTHROT_CUDA_ERROR;
  const int64_t slice = int64_t(workspace_bytes / row_bytes) < N ? int64_t(workspace_bytes / row_bytes) : N;
  const __half* W = static_cast<const __half*>(W_f16);
  float* rotated = static_cast<float*>(workspace);
  for (int64_t r0 = 0; r0 < N; r0 += slice) {
    const int64_t rows = N - r0 < slice ? N - r0 : slice;
    const int rc = smoothrot_debug_hadamard(W + r0 * ldw, rows, K, ldw, pre, rotated, stream);
    if (rc != SMOOTHROT_OK) return rc;
    kern<<<unsigned(rows), kSearchThreads, row_bytes, st>>>(rotated, r0, int(K), double(lowest_ratio), ratio_count,
                                                             Wq_out, dw_out, best_out);
    count_launch();
    if (launch_status() != SMOOTHROT_OK) return SMOOTHROT_CUDA_ERROR;
  }
  return SMOOTHROT_OK;
}

}  // extern "C"
