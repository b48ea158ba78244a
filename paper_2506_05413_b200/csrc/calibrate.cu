// Scale calibration of libsmoothrot:  s_j = max|X_j|^alpha / max|W_j|^(1 - alpha).
//
// column_absmax_kernel folds a batch of rows into a running per-channel
// maximum (fp16 magnitudes are exact in fp32, and non-negative floats order
// like their bit patterns, so an integer atomicMax keeps the result
// independent of the order in which rows arrive).  finalize_scales_kernel
// evaluates the formula in fp64 and writes s and the two diagonals derived
// from it.
#include "common.cuh"

namespace smoothrot {

std::atomic<int64_t> g_launches{0};

constexpr int kAbsmaxChunks = 128;     // 8-channel chunks per CTA (x dimension of the block)
constexpr int kAbsmaxRowLanes = 4;     // threads that share a chunk and split the rows (y dimension)
constexpr int kAbsmaxRowsPerCta = 64;

__device__ __forceinline__ void absmax_fold(uint4& best, const uint4& v) {
  // |x| as fp16 bit patterns: clear the sign bits, then a packed unsigned max
  // on the 16-bit lanes orders the magnitudes (NaNs aside).
  best.x = __vmaxu2(best.x, v.x & 0x7fff7fffu);
  best.y = __vmaxu2(best.y, v.y & 0x7fff7fffu);
  best.z = __vmaxu2(best.z, v.z & 0x7fff7fffu);
  best.w = __vmaxu2(best.w, v.w & 0x7fff7fffu);
}

__global__ void __launch_bounds__(kAbsmaxChunks * kAbsmaxRowLanes)
column_absmax_kernel(const __half* __restrict__ X, int64_t rows, int64_t K, int64_t ld,
                     float* __restrict__ amax) {
  __shared__ uint4 part[kAbsmaxRowLanes][kAbsmaxChunks];
  const int64_t c8 = int64_t(blockIdx.x) * kAbsmaxChunks + threadIdx.x;  // 8-channel chunk
  const bool live = c8 * 8 < K;
  const int64_t r0 = int64_t(blockIdx.y) * kAbsmaxRowsPerCta + threadIdx.y;
  const int64_t r1 = min(rows, int64_t(blockIdx.y + 1) * kAbsmaxRowsPerCta);
  uint4 best = make_uint4(0u, 0u, 0u, 0u);
  if (live) {
    const __half* col = X + c8 * 8;
    int64_t r = r0;
    // eight independent 16-byte loads in flight per thread
    for (; r + 7 * kAbsmaxRowLanes < r1; r += 8 * kAbsmaxRowLanes) {
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        v[u] = __ldg(reinterpret_cast<const uint4*>(col + (r + u * kAbsmaxRowLanes) * ld));
#pragma unroll
      for (int u = 0; u < 8; ++u) absmax_fold(best, v[u]);
    }
    for (; r < r1; r += kAbsmaxRowLanes)
      absmax_fold(best, __ldg(reinterpret_cast<const uint4*>(col + r * ld)));
  }
  part[threadIdx.y][threadIdx.x] = best;
  __syncthreads();
  if (threadIdx.y != 0 || !live) return;
#pragma unroll
  for (int y = 1; y < kAbsmaxRowLanes; ++y) absmax_fold(best, part[y][threadIdx.x]);
  const __half2* h = reinterpret_cast<const __half2*>(&best);
  int* out = reinterpret_cast<int*>(amax + c8 * 8);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h[i]);
    // non-negative floats order like their bit patterns
    atomicMax(out + 2 * i, __float_as_int(f.x));
    atomicMax(out + 2 * i + 1, __float_as_int(f.y));
  }
}

__global__ void finalize_scales_kernel(const float* __restrict__ amax, float* __restrict__ s_io, int64_t K,
                                       double alpha, const float* __restrict__ d,
                                       float* __restrict__ pre_w, float* __restrict__ pre_x) {
  const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (j >= K) return;
  const double eps = 1e-5;
  const double a = fmax(double(amax[j]), eps);
  const double w = fmax(double(s_io[j]), eps);   // s_io holds max|W_j| on entry
  const double s64 = fmax(pow(a, alpha) / pow(w, 1.0 - alpha), eps);
  const float s = float(s64);
  s_io[j] = s;
  if (d != nullptr) {
    const float dj = d[j];
    if (pre_w != nullptr) pre_w[j] = s * dj;
    if (pre_x != nullptr) pre_x[j] = __fdiv_rn(dj, s);
  }
}

static void launch_absmax(const __half* X, int64_t rows, int64_t K, int64_t ld, float* amax, cudaStream_t st) {
  dim3 grid(unsigned((K / 8 + kAbsmaxChunks - 1) / kAbsmaxChunks),
            unsigned((rows + kAbsmaxRowsPerCta - 1) / kAbsmaxRowsPerCta));
  dim3 block(kAbsmaxChunks, kAbsmaxRowLanes);
  column_absmax_kernel<<<grid, block, 0, st>>>(X, rows, K, ld, amax);
  count_launch();
}

}  // namespace smoothrot

extern "C" {

int smoothrot_calibrate(const void* X_f16, int64_t T, int64_t K, int64_t ldx, const void* W_f16, int64_t N,
                        int64_t ldw, float alpha, int finalize, float* amax_inout, float* s_out,
                        const float* d, float* pre_w_out, float* pre_x_out, void* stream) {
  using namespace smoothrot;
  if (T < 0 || K <= 0 || amax_inout == nullptr) return SMOOTHROT_INVALID_ARG;
  if (K % 8 != 0) return SMOOTHROT_UNSUPPORTED_K;
  if (T > 0 && (X_f16 == nullptr || ldx < K)) return SMOOTHROT_INVALID_ARG;
  if (T > 0 && (!aligned16(X_f16) || ldx % 8 != 0)) return SMOOTHROT_BAD_ALIGNMENT;
  if (!aligned16(amax_inout)) return SMOOTHROT_BAD_ALIGNMENT;
  if (T > 0x7fffffffLL * kAbsmaxRowsPerCta / 65535) return SMOOTHROT_INVALID_ARG;
  if (finalize) {
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return SMOOTHROT_INVALID_ARG;
    if (N <= 0 || W_f16 == nullptr || s_out == nullptr || ldw < K) return SMOOTHROT_INVALID_ARG;
    if (!aligned16(W_f16) || ldw % 8 != 0 || !aligned16(s_out)) return SMOOTHROT_BAD_ALIGNMENT;
    if ((N + kAbsmaxRowsPerCta - 1) / kAbsmaxRowsPerCta > 65535) return SMOOTHROT_INVALID_ARG;
  }
  if ((T + kAbsmaxRowsPerCta - 1) / kAbsmaxRowsPerCta > 65535) return SMOOTHROT_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (T > 0) launch_absmax(static_cast<const __half*>(X_f16), T, K, ldx, amax_inout, st);
  if (finalize) {
    if (cudaMemsetAsync(s_out, 0, size_t(K) * sizeof(float), st) != cudaSuccess) return SMOOTHROT_CUDA_ERROR;
    launch_absmax(static_cast<const __half*>(W_f16), N, K, ldw, s_out, st);
    const int threads = 256;
    finalize_scales_kernel<<<unsigned((K + threads - 1) / threads), threads, 0, st>>>(
        amax_inout, s_out, K, double(alpha), d, pre_w_out, pre_x_out);
    count_launch();
  }
  return launch_status();
}

const char* smoothrot_status_string(int status) {
  switch (status) {
    case SMOOTHROT_OK: return "ok";
    case SMOOTHROT_INVALID_ARG: return "invalid argument";
    case SMOOTHROT_UNSUPPORTED_K: return "unsupported K (need 2^p, 7<=p<=13, or 28*2^p, 3<=p<=9)";
    case SMOOTHROT_BAD_ALIGNMENT: return "pointer or leading dimension not aligned";
    case SMOOTHROT_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SMOOTHROT_CUDA_ERROR: return "CUDA error";
    case SMOOTHROT_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case SMOOTHROT_STATIC_SCRATCH_EXCEEDED:
      return "shape needs more split-K scratch than the library's built-in array holds";
    default: return "unknown status";
  }
}

int64_t smoothrot_launch_count(void) { return smoothrot::g_launches.load(); }

}  // extern "C"
