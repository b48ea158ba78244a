// Shared host-side helpers of libsmoothrot (argument checks, launch counting).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "smoothrot.h"

namespace smoothrot {

// Number of kernels launched by the library (reported by smoothrot_launch_count).
extern std::atomic<int64_t> g_launches;

inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

inline int ilog2(int64_t v) {
  int l = 0;
  while ((int64_t(1) << l) < v) ++l;
  return l;
}

// K = base * n with base 1 (Walsh, n = 2^p, 7 <= p <= 13) or base 12, 20 or 28
// (Paley x Walsh, n = 2^p, 3 <= p <= 10).  Returns false if K is neither.
inline bool split_order(int64_t K, int* base, int* n, int* logn) {
  if (is_pow2(K)) {
    int l = ilog2(K);
    if (l < 7 || l > 13) return false;
    *base = 1; *n = int(K); *logn = l;
    return true;
  }
  // 4 * odd * 2^p with odd in {3, 5, 7}: the odd part of K decides the Paley factor (12, 20 or 28)
  for (int b : {28, 20, 12}) {
    if (K > 0 && K % b == 0 && is_pow2(K / b)) {
      int l = ilog2(K / b);
      if (l < 3 || l > 10) return false;
      *base = b; *n = int(K / b); *logn = l;
      return true;
    }
  }
  return false;
}

// Number of SMs of the current device (148 on B200); cached after the first query.
inline int device_sm_count() {
  static std::atomic<int> cached{0};
  int n = cached.load(std::memory_order_relaxed);
  if (n > 0) return n;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
    return 148;
  cached.store(n, std::memory_order_relaxed);
  return n;
}

// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link libcuda).
#ifdef CUDA_VERSION
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline TensorMapEncodeFn tensor_map_encoder() {
  static std::atomic<TensorMapEncodeFn> cached{nullptr};
  TensorMapEncodeFn fn = cached.load(std::memory_order_acquire);
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<TensorMapEncodeFn>(ptr);
      cached.store(fn, std::memory_order_release);
    }
  }
  return fn;
}
#endif

// Raises a kernel's dynamic shared-memory limit: one runtime call per kernel, device and size, then a
// table look-up (the runtime call costs a microsecond or so on every eager launch otherwise).
inline bool allow_dynamic_smem(const void* kern, int bytes) {
  struct Entry {
    const void* kern;
    int dev;
    int bytes;
  };
  static std::mutex mu;
  static std::vector<Entry> done;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : done)
      if (e.kern == kern && e.dev == dev && e.bytes >= bytes) return true;
  }
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  std::lock_guard<std::mutex> lock(mu);
  done.push_back(Entry{kern, dev, bytes});
  return true;
}

inline int launch_status() {
  return cudaGetLastError() == cudaSuccess ? SMOOTHROT_OK : SMOOTHROT_CUDA_ERROR;
}

}  // namespace smoothrot
