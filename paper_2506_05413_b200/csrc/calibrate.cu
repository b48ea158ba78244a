// Scale calibration of libsmoothrot:  s_j = max|X_j|^alpha / max|W_j|^(1 - alpha).
//
// column_absmax_kernel folds a batch of rows into a running per-channel
// maximum (fp16 magnitudes are exact in fp32, and non-negative floats order
// like their bit patterns, so an integer atomicMax keeps the result
// independent of the order in which rows arrive).  finalize_scales_kernel
// evaluates the formula in fp64 (as 2^(alpha log2 a - (1 - alpha) log2 w)) and writes s and the two diagonals derived
// from it.
#include "common.cuh"

namespace smoothrot {

std::atomic<int64_t> g_launches{0};

constexpr int kAbsmaxChunks = 32;      // 8-channel chunks per CTA (x dimension of the block): one warp = 512 bytes of a row
constexpr int kAbsmaxRowLanes = 16;    // threads that share a chunk and split the rows (y dimension)
constexpr int kAbsmaxCtasPerSm = 1;    // the grid is sized to fill the machine once, whatever the row count

__device__ __forceinline__ uint32_t absmax_fold2(uint32_t best, uint32_t v) {
  // max(best, |v|) on both fp16 lanes: clear the sign bits, then the native packed fp16 maximum
  // (exact on magnitudes; NaNs aside)
  uint32_t m;
  asm("max.f16x2 %0, %1, %2;" : "=r"(m) : "r"(best), "r"(v & 0x7fff7fffu));
  return m;
}

__device__ __forceinline__ void absmax_fold(uint4& best, const uint4& v) {
  best.x = absmax_fold2(best.x, v.x);
  best.y = absmax_fold2(best.y, v.y);
  best.z = absmax_fold2(best.z, v.z);
  best.w = absmax_fold2(best.w, v.w);
}

// Folds rows r0, r0 + step, ... (< rows) of one 8-channel chunk into `best`.  A ring of eight
// 16-byte loads stays in flight: each value is folded and its register refilled eight rows ahead.
__device__ __forceinline__ void absmax_rows(uint4& best, const __half* col, int64_t ld, int r0, int step, int rows) {
  constexpr int kDepth = 8;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  const uint4* p = reinterpret_cast<const uint4*>(col + int64_t(r0) * ld);   // row r0 of this chunk
  const int64_t hop = int64_t(step) * ld / 8;                                 // one step of rows, in 16-byte units
  uint4 v[kDepth];
#pragma unroll
  for (int u = 0; u < kDepth; ++u) v[u] = r0 + u * step < rows ? __ldg(p + u * hop) : zero;
#pragma unroll 1
  for (int r = r0; r < rows; r += kDepth * step) {
    p += kDepth * hop;
#pragma unroll
    for (int u = 0; u < kDepth; ++u) {
      absmax_fold(best, v[u]);
      v[u] = r + (u + kDepth) * step < rows ? __ldg(p + u * hop) : zero;
    }
  }
}

// Reduces the row lanes of a CTA and merges the result into out[c8 * 8 ...] with integer atomicMax.
__device__ __forceinline__ void absmax_merge(uint4 best, uint4 (*part)[kAbsmaxChunks], int64_t c8, bool live,
                                             float* __restrict__ out) {
  part[threadIdx.y][threadIdx.x] = best;
  __syncthreads();
  if (threadIdx.y == 0 && live) {
#pragma unroll 4
    for (int y = 1; y < kAbsmaxRowLanes; ++y) absmax_fold(best, part[y][threadIdx.x]);
    const __half2* h = reinterpret_cast<const __half2*>(&best);
    int* o = reinterpret_cast<int*>(out + c8 * 8);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(h[i]);
      // non-negative floats order like their bit patterns; zero never raises the maximum
      if (f.x != 0.0f) atomicMax(o + 2 * i, __float_as_int(f.x));
      if (f.y != 0.0f) atomicMax(o + 2 * i + 1, __float_as_int(f.y));
    }
  }
  __syncthreads();
}

// One launch covers the calibration batch X [T x K] (blockIdx.z = 0, into amax) and, when W is
// given, the weights W [N x K] (blockIdx.z = 1, into wmax).  blockIdx.x picks a slab of 256
// channels, blockIdx.y a set of rows (row lanes of all CTAs of a slab interleave).
__global__ void __launch_bounds__(kAbsmaxChunks * kAbsmaxRowLanes)
column_absmax_kernel(const __half* __restrict__ X, int T, int64_t ldx, float* __restrict__ amax,
                     const __half* __restrict__ W, int N, int64_t ldw, float* __restrict__ wmax, int64_t K) {
  __shared__ uint4 part[kAbsmaxRowLanes][kAbsmaxChunks];
  const bool second = blockIdx.z != 0;
  const __half* src = second ? W : X;
  const int rows = second ? N : T;
  const int64_t ld = second ? ldw : ldx;
  float* out = second ? wmax : amax;
  if (src == nullptr || rows <= 0) return;   // uniform over the CTA
  const int64_t c8 = int64_t(blockIdx.x) * kAbsmaxChunks + threadIdx.x;  // 8-channel chunk
  const bool live = c8 * 8 < K;
  const int r0 = int(blockIdx.y) * kAbsmaxRowLanes + int(threadIdx.y);
  const int step = int(gridDim.y) * kAbsmaxRowLanes;
  uint4 best = make_uint4(0u, 0u, 0u, 0u);
  if (live) absmax_rows(best, src + c8 * 8, ld, r0, step, rows);
  absmax_merge(best, part, c8, live, out);
}

__global__ void finalize_scales_kernel(const float* __restrict__ amax, float* __restrict__ s_io, int64_t K,
                                       double alpha, const float* __restrict__ d,
                                       float* __restrict__ pre_w, float* __restrict__ pre_x) {
  const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (j >= K) return;
  const double eps = 1e-5;
  const double a = fmax(double(amax[j]), eps);
  const double w = fmax(double(s_io[j]), eps);   // s_io holds max|W_j| on entry
  // a^alpha / w^(1 - alpha) through base-2 logarithms, all in fp64 (error far below one fp32 ulp)
  const double s64 = fmax(exp2(alpha * log2(a) - (1.0 - alpha) * log2(w)), eps);
  const float s = float(s64);
  s_io[j] = s;
  if (d != nullptr) {
    const float dj = d[j];
    if (pre_w != nullptr) pre_w[j] = s * dj;
    if (pre_x != nullptr) pre_x[j] = __fdiv_rn(dj, s);
  }
}

static void launch_absmax(const __half* X, int64_t T, int64_t ldx, float* amax, const __half* W, int64_t N,
                          int64_t ldw, float* wmax, int64_t K, cudaStream_t st) {
  const int64_t slabs = (K / 8 + kAbsmaxChunks - 1) / kAbsmaxChunks;
  const int64_t most_rows = T > N ? T : N;
  int64_t row_sets = int64_t(device_sm_count()) * kAbsmaxCtasPerSm / slabs;   // rounded down: one wave, no tail
  const int64_t useful = (most_rows + kAbsmaxRowLanes - 1) / kAbsmaxRowLanes;   // beyond this, CTAs would idle
  if (row_sets > useful) row_sets = useful;
  if (row_sets < 1) row_sets = 1;
  const dim3 grid(static_cast<unsigned>(slabs), static_cast<unsigned>(row_sets), W != nullptr ? 2u : 1u);
  dim3 block(kAbsmaxChunks, kAbsmaxRowLanes);
  column_absmax_kernel<<<grid, block, 0, st>>>(X, int(T), ldx, amax, W, int(N), ldw, wmax, K);
  count_launch();
}

}  // namespace smoothrot

extern "C" {

int smoothrot_calibrate(const void* X_f16, int64_t T, int64_t K, int64_t ldx, const void* W_f16, int64_t N,
                        int64_t ldw, float alpha, int finalize, float* amax_inout, float* s_out,
                        const float* d, float* pre_w_out, float* pre_x_out, void* stream) {
  using namespace smoothrot;
  if (T < 0 || K <= 0 || amax_inout == nullptr) return SMOOTHROT_INVALID_ARG;
  if (T > 0x3fffffffLL || N > 0x3fffffffLL) return SMOOTHROT_INVALID_ARG;
  if (K % 8 != 0) return SMOOTHROT_UNSUPPORTED_K;
  if (T > 0 && (X_f16 == nullptr || ldx < K)) return SMOOTHROT_INVALID_ARG;
  if (T > 0 && (!aligned16(X_f16) || ldx % 8 != 0)) return SMOOTHROT_BAD_ALIGNMENT;
  if (!aligned16(amax_inout)) return SMOOTHROT_BAD_ALIGNMENT;
  if (finalize) {
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return SMOOTHROT_INVALID_ARG;
    if (N <= 0 || W_f16 == nullptr || s_out == nullptr || ldw < K) return SMOOTHROT_INVALID_ARG;
    if (!aligned16(W_f16) || ldw % 8 != 0 || !aligned16(s_out)) return SMOOTHROT_BAD_ALIGNMENT;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __half* X = T > 0 ? static_cast<const __half*>(X_f16) : nullptr;
  if (finalize) {
    // s_out collects max|W_j| first (it must start at zero), then receives s
    if (cudaMemsetAsync(s_out, 0, size_t(K) * sizeof(float), st) != cudaSuccess) return SMOOTHROT_CUDA_ERROR;
    launch_absmax(X, T, ldx, amax_inout, static_cast<const __half*>(W_f16), N, ldw, s_out, K, st);
    const int threads = 128;
    finalize_scales_kernel<<<unsigned((K + threads - 1) / threads), threads, 0, st>>>(
        amax_inout, s_out, K, double(alpha), d, pre_w_out, pre_x_out);
    count_launch();
  } else if (T > 0) {
    launch_absmax(X, T, ldx, amax_inout, nullptr, 0, 0, nullptr, K, st);
  }
  return launch_status();
}

const char* smoothrot_status_string(int status) {
  switch (status) {
    case SMOOTHROT_OK: return "ok";
    case SMOOTHROT_INVALID_ARG: return "invalid argument";
    case SMOOTHROT_UNSUPPORTED_K: return "unsupported K (need 2^p, 7<=p<=13, or 12*2^p, 20*2^p, 28*2^p, 3<=p<=10)";
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
