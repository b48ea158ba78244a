// W4A4 GEMM of libsmoothrot:  acc[m][n] = sum_k Xq[m][k] Wq[n][k]  on packed
// 4-bit codes, with the dequantization  Y = fp16(acc * dx[m] * dw[n])  fused
// into the epilogue (Eq. 2's product on Eq. 1's integer codes, then Eq. 1's
// dequantizer on both factors).
//
// sm_100a has no 4-bit integer MMA, so the codes are widened to int8 on the
// way to the tensor core:
//
//   TMA (cp.async.bulk.tensor, 64-byte swizzle) brings 64 packed bytes per
//   row and k-block into shared memory;
//   "widen" warps read 16 packed bytes and write two 16-byte int8 vectors
//   (w & 0xF0F0F0F0 and (w << 4) & 0xF0F0F0F0: each byte lane is 16 * code in
//   two's complement, no sign extension needed) into the 128-byte-swizzled
//   K-major layout tcgen05.mma reads.  Both operands get the same permutation
//   of k inside a k-block, which a dot product does not see;
//   one thread issues tcgen05.mma.kind::i8 (128 x BN x 32) with the int32
//   accumulator in tensor memory; accumulators are 256 * acc, exact, and
//   |256 * acc| <= K * 128 * 128 < 2^31 for K <= 65536;
//   four epilogue warps read the accumulator with tcgen05.ld, shift by 8,
//   scale and store, while the next tile's main loop runs on the other half
//   of tensor memory.
//
// The kernels are persistent (one CTA per SM, tiles handed out round-robin).
// Shapes with M >= 256 and N >= 256 run the two-CTA kernel further down, which
// keeps the token operand in tensor memory instead of shared memory.
// For M <= 128 tokens the roles of the operands are swapped (output channels on
// the 128-row MMA axis, tokens on the N axis) and K is split across CTAs;
// the int32 partial sums are added inside a thread-block cluster, or go to the
// caller's workspace where a second kernel adds them and dequantizes.
// For up to 32 tokens (64 with small weight matrices) none of this machinery
// pays: a small kernel streams the weights with plain loads and forms the
// products with the warp-level integer MMA (see the decode kernel near the end).
//
// Every wait on an mbarrier is bounded in wall time; a wait that runs out
// sets a device status word, raises a CTA-wide abort flag and the kernel
// winds down normally.
#include <cuda.h>

#include "common.cuh"
#include "decode.cuh"

// defined with the row transform kernels: their timeout word
extern "C" int smoothrot_rotate_status_word(int* value, int clear);
// defined with the row transform kernels: the limit of their bounded waits
extern "C" int smoothrot_rotate_set_wait_limit_ns(uint64_t ns);

namespace smoothrot {
namespace gemm {

constexpr int kBM = 128;            // MMA M: rows of the A side per tile
constexpr int kPackedRow = 64;      // packed bytes per row and k-block
constexpr int kWideRow = 128;       // int8 bytes per row and k-block (= codes per k-block)
constexpr int kWidenWarps = 8;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 32 * (2 + kWidenWarps + kEpiWarps);
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s
constexpr unsigned long long kDrainNs = 50000ull;           // pause before leaving after a timeout

__device__ int g_device_status = 0;
// Limit of every bounded wait of these kernels, in nanoseconds (a test shortens it).
__device__ unsigned long long g_wait_limit_ns = kWaitLimitNs;

enum TimeoutSite { kSiteProducer = 1, kSiteWidenFull = 2, kSiteWidenEmpty = 3, kSiteMmaAcc = 4,
                   kSiteMmaWide = 5, kSiteEpilogue = 6, kSiteProbe = 7 };

template <int BN>
struct Tile {
  static constexpr int kWideStages = BN >= 256 ? 2 : (BN >= 128 ? 3 : 4);
  static constexpr int kPackedStages = BN >= 256 ? 4 : (BN >= 128 ? 4 : 6);
  static constexpr int kWideA = kBM * kWideRow, kWideB = BN * kWideRow;
  static constexpr int kPackedA = kBM * kPackedRow, kPackedB = BN * kPackedRow;
  // kPackedB may be below 1024 bytes (BN = 16): round stage parts up to 1024 so
  // that every tile base keeps the alignment the swizzle patterns assume.
  static constexpr int kPackedBPad = (kPackedB + 1023) / 1024 * 1024;
  static constexpr int kWideBPad = (kWideB + 1023) / 1024 * 1024;
  static constexpr int kWideStageBytes = kWideA + kWideBPad;
  static constexpr int kPackedStageBytes = kPackedA + kPackedBPad;
  static constexpr int kNumBarriers = 2 * kWideStages + 2 * kPackedStages + 4;
  static constexpr int kSmemBytes = 1024 /*alignment slack*/ + kWideStages * kWideStageBytes +
                                    kPackedStages * kPackedStageBytes + kNumBarriers * 8 + 16;
  static constexpr int kTmemCols = (2 * BN) < 32 ? 32 : 2 * BN;  // two accumulators, power of two
};

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Waits for the barrier phase with the given parity, at most g_wait_limit_ns (2 s unless a test
// has shortened it).
// Returns false if the wait ran out or another role of this CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int site) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 63u) == 0u) {
      if (*abort_flag != 0) return false;
      if (global_ns() - t0 > g_wait_limit_ns) {
        *abort_flag = 1;
        atomicCAS(&g_device_status, 0, site);
        return false;
      }
    }
  }
}

// Wind-down after a timeout: copies and tensor-core operations this CTA started may still be on
// their way into its shared and tensor memory.  Every thread pauses long enough for them to land
// (they complete in microseconds once issued) before the CTA gives its memory back.
__device__ __forceinline__ void drain_after_abort(volatile int* abort_flag) {
  if (*abort_flag == 0) return;
  const unsigned long long t0 = global_ns();
  while (global_ns() - t0 < kDrainNs) __nanosleep(1000);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of
// 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t smem_addr) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return (uint64_t(hi) << 32) | lo;
}

// Instruction descriptor: int8 x int8 -> int32, both operands K-major, M = 128.
__host__ __device__ constexpr uint32_t make_idesc_i8(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(kBM >> 4) << 24);
}

// ---------------------------------------------------------------------------
// Kernel parameters
// ---------------------------------------------------------------------------
struct Params {
  int rows_a, rows_b;     // valid rows of the A-side and B-side matrices
  int tiles_a, tiles_b;   // tile counts
  int kblocks;            // K / 128
  int splits;             // k-splits (1 = none)
  int cluster_reduce;     // the k-splits of a tile form a thread-block cluster and add up in shared memory
  int swapped;            // 0: A side = tokens (Xq), B side = channels (Wq); 1: the reverse
  int M, N;               // logical output shape
  const float* dx;        // [M]
  const float* dw;        // [N]
  __half* Y;              // [M x ldy] (direct dequantized output) or nullptr
  int64_t ldy;
  int32_t* acc_out;       // [splits][M][N] int32 (debug export or split-K partials) or nullptr
};

// Writes 32 consecutive accumulator columns [c0, c0 + 32) of A-side row `a`.
template <int NCOLS>
__device__ __forceinline__ void store_columns(const Params& p, int a, int b0, int split, const uint32_t* r) {
  if (a >= p.rows_a) return;
  if (!p.swapped) {
    const int m = a;
    if (p.Y != nullptr) {
      const float sx = __ldg(p.dx + m);
      __half* y = p.Y + int64_t(m) * p.ldy + b0;
#pragma unroll
      for (int j = 0; j < NCOLS; j += 8) {
        if (b0 + j + 8 <= p.rows_b) {
          const float4 w0 = __ldg(reinterpret_cast<const float4*>(p.dw + b0 + j));
          const float4 w1 = __ldg(reinterpret_cast<const float4*>(p.dw + b0 + j + 4));
          const float ws[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
          uint4 out;
          __half2* h = reinterpret_cast<__half2*>(&out);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float v0 = float(int32_t(r[j + 2 * q]) >> 8) * (sx * ws[2 * q]);
            const float v1 = float(int32_t(r[j + 2 * q + 1]) >> 8) * (sx * ws[2 * q + 1]);
            h[q] = __floats2half2_rn(v0, v1);
          }
          *reinterpret_cast<uint4*>(y + j) = out;
        }
      }
    } else {
      int32_t* o = p.acc_out + (int64_t(split) * p.M + m) * p.N + b0;
#pragma unroll
      for (int j = 0; j < NCOLS; j += 4) {
        if (b0 + j + 4 <= p.rows_b) {
          int4 v = make_int4(int32_t(r[j]) >> 8, int32_t(r[j + 1]) >> 8, int32_t(r[j + 2]) >> 8,
                             int32_t(r[j + 3]) >> 8);
          *reinterpret_cast<int4*>(o + j) = v;
        }
      }
    }
  } else {
    const int n = a;  // output channel; columns are tokens
    if (p.Y != nullptr) {
      const float sw = __ldg(p.dw + n);
#pragma unroll
      for (int j = 0; j < NCOLS; ++j) {
        const int m = b0 + j;
        if (m < p.rows_b) {
          const float v = float(int32_t(r[j]) >> 8) * (__ldg(p.dx + m) * sw);
          p.Y[int64_t(m) * p.ldy + n] = __float2half_rn(v);
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < NCOLS; ++j) {
        const int m = b0 + j;
        if (m < p.rows_b) p.acc_out[(int64_t(split) * p.M + m) * p.N + n] = int32_t(r[j]) >> 8;
      }
    }
  }
}

// ---------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
w4a4_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const Params p) {
  using T = Tile<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);

  const uint32_t wide_base = base;
  const uint32_t packed_base = wide_base + T::kWideStages * T::kWideStageBytes;
  const uint32_t bar_base = packed_base + T::kPackedStages * T::kPackedStageBytes;
  // barrier order: wide_full[WS], wide_empty[WS], pk_full[PS], pk_empty[PS], acc_full[2], acc_empty[2]
  auto wide_full = [&](int s) { return bar_base + 8u * s; };
  auto wide_empty = [&](int s) { return bar_base + 8u * (T::kWideStages + s); };
  auto pk_full = [&](int s) { return bar_base + 8u * (2 * T::kWideStages + s); };
  auto pk_empty = [&](int s) { return bar_base + 8u * (2 * T::kWideStages + T::kPackedStages + s); };
  auto acc_full = [&](int s) { return bar_base + 8u * (2 * T::kWideStages + 2 * T::kPackedStages + s); };
  auto acc_empty = [&](int s) { return bar_base + 8u * (2 * T::kWideStages + 2 * T::kPackedStages + 2 + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + (bar_base - base) + 8 * T::kNumBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < T::kWideStages; ++s) {
      mbar_init(wide_full(s), kWidenWarps);
      mbar_init(wide_empty(s), 1);
    }
    for (int s = 0; s < T::kPackedStages; ++s) {
      mbar_init(pk_full(s), 1);
      mbar_init(pk_empty(s), kWidenWarps);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(acc_full(s), 1);
      mbar_init(acc_empty(s), kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(uint32_t(T::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int total_tiles = p.tiles_a * p.tiles_b * p.splits;
  const int kb_per_split = p.kblocks / p.splits;  // host guarantees divisibility

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int ta = tile % p.tiles_a;
        const int rest = tile / p.tiles_a;
        const int tb = rest % p.tiles_b;
        const int split = rest / p.tiles_b;
        const int kb0 = split * kb_per_split;
        for (int kb = kb0; kb < kb0 + kb_per_split; ++kb, ++it) {
          const int s = it % T::kPackedStages;
          const uint32_t ph = (it / T::kPackedStages) & 1u;
          if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag, kSiteProducer)) { ok = false; break; }
          mbar_expect_tx(pk_full(s), uint32_t(T::kPackedA + T::kPackedB));
          const uint32_t dst = packed_base + s * T::kPackedStageBytes;
          tma_load_2d(dst, &map_a, pk_full(s), kb * kPackedRow, ta * kBM);
          tma_load_2d(dst + T::kPackedA, &map_b, pk_full(s), kb * kPackedRow, tb * BN);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_i8(BN);
      uint32_t it = 0, local_tile = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++local_tile) {
        const int ab = local_tile & 1;
        const uint32_t aph = (local_tile >> 1) & 1u;
        if (!mbar_wait(acc_empty(ab), aph ^ 1u, abort_flag, kSiteMmaAcc)) break;
        tcgen05_fence_after();
        const uint32_t tmem_d = tmem_base + uint32_t(ab * BN);
        for (int kb = 0; kb < kb_per_split; ++kb, ++it) {
          const int s = it % T::kWideStages;
          const uint32_t ph = (it / T::kWideStages) & 1u;
          if (!mbar_wait(wide_full(s), ph, abort_flag, kSiteMmaWide)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t a_addr = wide_base + s * T::kWideStageBytes;
          const uint64_t da = make_desc_sw128(a_addr);
          const uint64_t db = make_desc_sw128(a_addr + T::kWideA);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) {
            // 32 int8 = 32 bytes further along K inside the swizzle atom: +2 in 16-byte units
            mma_i8(tmem_d, da + uint64_t(2 * k4), db + uint64_t(2 * k4), idesc, (kb > 0 || k4 > 0) ? 1u : 0u);
          }
          tcgen05_commit(wide_empty(s));
        }
        if (ok) tcgen05_commit(acc_full(ab));
      }
    }
  } else if (warp < 2 + kWidenWarps) {
    // ------------------------------------------------------------ widen warps
    const int w = warp - 2;
    const int r = lane & 7;    // row inside an 8-row group
    const int c = lane >> 3;   // 16-byte chunk of the packed row (0..3)
    constexpr int kGroupsA = kBM / 8;
    constexpr int kGroups = (kBM + BN) / 8;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < kb_per_split; ++kb, ++it) {
        const int ps = it % T::kPackedStages;
        const uint32_t pph = (it / T::kPackedStages) & 1u;
        const int ws = it % T::kWideStages;
        const uint32_t wph = (it / T::kWideStages) & 1u;
        if (!mbar_wait(pk_full(ps), pph, abort_flag, kSiteWidenFull)) { ok = false; break; }
        if (!mbar_wait(wide_empty(ws), wph ^ 1u, abort_flag, kSiteWidenEmpty)) { ok = false; break; }
        const uint32_t pk = packed_base + ps * T::kPackedStageBytes;
        const uint32_t wd = wide_base + ws * T::kWideStageBytes;
#pragma unroll 2
        for (int g = w; g < kGroups; g += kWidenWarps) {
          // operand-local row and the two tile bases
          const bool is_b = g >= kGroupsA;
          const int row = (is_b ? g - kGroupsA : g) * 8 + r;
          const uint32_t src = (is_b ? pk + T::kPackedA : pk) + row * kPackedRow + ((c ^ ((row >> 1) & 3)) << 4);
          const uint32_t dst_row = (is_b ? wd + T::kWideA : wd) + row * kWideRow;
          uint32_t x0, x1, x2, x3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3) : "r"(src) : "memory");
          const uint32_t lo_dst = dst_row + (((2 * c) ^ (row & 7)) << 4);
          const uint32_t hi_dst = dst_row + (((2 * c + 1) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(lo_dst), "r"((x0 << 4) & 0xF0F0F0F0u), "r"((x1 << 4) & 0xF0F0F0F0u),
                         "r"((x2 << 4) & 0xF0F0F0F0u), "r"((x3 << 4) & 0xF0F0F0F0u) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(hi_dst), "r"(x0 & 0xF0F0F0F0u), "r"(x1 & 0xF0F0F0F0u),
                         "r"(x2 & 0xF0F0F0F0u), "r"(x3 & 0xF0F0F0F0u) : "memory");
        }
        fence_proxy_async();   // make the generic-proxy stores visible to the tensor core
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(wide_full(ws));
          mbar_arrive(pk_empty(ps));
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int e = warp & 3;  // tensor-memory lane quadrant this warp may read
    uint32_t local_tile = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++local_tile) {
      const int ta = tile % p.tiles_a;
      const int rest = tile / p.tiles_a;
      const int tb = rest % p.tiles_b;
      const int split = rest / p.tiles_b;
      const int ab = local_tile & 1;
      const uint32_t aph = (local_tile >> 1) & 1u;
      if (!mbar_wait(acc_full(ab), aph, abort_flag, kSiteEpilogue)) break;
      tcgen05_fence_after();
      const int a = ta * kBM + e * 32 + lane;
      const uint32_t taddr = tmem_base + (uint32_t(e * 32) << 16) + uint32_t(ab * BN);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t regs[32];
        tmem_load32(taddr + c0, regs);
        tmem_wait_ld();
        store_columns<32>(p, a, tb * BN + c0, split, regs);
        __syncwarp();
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(ab));
    }
  }

  drain_after_abort(abort_flag);
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"(uint32_t(T::kTmemCols)) : "memory");
  }
}

// ---------------------------------------------------------------------------
// Two-CTA kernel for prefill shapes.  A cluster of two CTAs (one SM pair)
// computes one 256 x 256 output tile with tcgen05.mma.cta_group::2: each CTA
// holds its own 128 rows of the A side and stages HALF of the B side (128 of
// the 256 output channels); the tensor cores of both SMs read the two B
// halves, so per SM the widen work and the operand reads of B are halved.
// The MMA is issued by one thread of the leader CTA (cluster rank 0).
//
// Barriers that collect arrivals from both CTAs (full, acc_empty) live in the
// leader; the peer's warps arrive on them through the cluster shared window.
// Barriers that release work in both CTAs (empty, acc_full) are signalled by
// tcgen05.commit with a two-CTA multicast mask.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// Arrival on a barrier of the other CTA of the pair.  The data this signals
// (int8 tiles in the arriving CTA's own shared memory, already fenced for the
// async proxy; accumulator reads already fenced with tcgen05.fence) is consumed
// by tensor-core work on the arriving CTA's own SM, so the default CTA-scope
// release is enough; a cluster-scope release here stalls every arriving warp
// for well over a thousand cycles per k-block.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(mask)
      : "memory");
}
// int8 x int8 -> int32, K-major operands, M = 256 over the CTA pair.
__host__ __device__ constexpr uint32_t make_idesc_i8_pair(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(256 >> 4) << 24);
}

// ---------------------------------------------------------------------------
// The token operand lives in tensor memory.
//
// Shared-memory bandwidth (128 bytes per clock and SM, shared by TMA writes,
// the widen warps and the tensor core's operand reads) is what bounds the
// kernels above.  Here the A side (128 token rows per CTA) never goes back to
// shared memory after it was widened: "A-widen" warps read the packed rows
// that TMA delivered, widen them in registers and write them with tcgen05.st
// into a ring of slots in tensor memory, from where tcgen05.mma takes its A
// operand.  Only the B side (each CTA's half of the 256 output channels) is
// widened into shared memory.  Per 128-deep k-block a CTA then moves
// 16 KB (A: TMA write + read) + 48 KB (B: TMA write, read, int8 write,
// tensor-core read) through shared memory, against 96 KB before.
//
// Tensor memory: columns [0, 256) hold the one 128 x 256 int32 accumulator,
// columns [256, 256 + 32 * kStages) the A ring (a k-block of a row is 128 int8
// = 32 columns).  With a single accumulator the epilogue cannot overlap the
// next tile's MMAs; it drains the accumulator into a shared-memory staging
// area as fp16 (releasing tensor memory as soon as the last tcgen05.ld has
// returned) and TMA stores write the staged tile to Y asynchronously.
// ---------------------------------------------------------------------------
struct PairT {
  static constexpr int kBN = 256;      // output channels per pair tile
  static constexpr int kHalfN = 128;   // B-side rows staged by each CTA
  static constexpr int kStages = 5;    // int8 B stages in shared memory = A slots in tensor memory
  static constexpr int kPackedStages = 4;
  static constexpr int kPackedA = kBM * kPackedRow, kPackedB = kHalfN * kPackedRow;
  static constexpr int kPackedStageBytes = kPackedA + kPackedB;
  static constexpr int kWideB = kHalfN * kWideRow;
  static constexpr int kOutBoxBytes = 32 * 128;              // 32 rows x 64 fp16
  static constexpr int kOutBytes = kEpiWarps * 4 * kOutBoxBytes;  // 128 rows x 256 fp16
  static constexpr int kDwBytes = kEpiWarps * kBN * 4;         // per epilogue warp: the tile's 256 weight steps
  static constexpr int kNumBarriers = 2 * kStages + 2 * kPackedStages + 2;
  static constexpr int kSmemBytes = 1024 + kStages * kWideB + kPackedStages * kPackedStageBytes + kOutBytes +
                                    kDwBytes + kNumBarriers * 8 + 16;
  static constexpr int kTmemCols = 512;
  static constexpr int kAccCols = 256;
  // Two sets of widen warps take the k-blocks in turn (even / odd), so that a warp has two
  // k-block periods for its chain of waits, loads and stores; per k-block 4 A-widen warps (one
  // per tensor-memory lane quadrant) and 4 B-widen warps are at work.
  static constexpr int kWidenSets = 2;
  static constexpr int kAWidenWarps = 4 * kWidenSets, kBWidenWarps = 4 * kWidenSets;
  static constexpr int kArrivalsPerStage = 8;   // 4 A-widen + 4 B-widen warps per CTA and k-block
  static constexpr int kThreads = 32 * (2 + kAWidenWarps + kBWidenWarps + kEpiWarps);
  static_assert(kAccCols + 32 * kStages <= kTmemCols, "A ring does not fit tensor memory");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ void mma_i8_pair_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The odd codes of a packed word as int8 lanes (16 * code).  Volatile on purpose: the
// instruction needs the loaded word, so the warp cannot go past it (to the arrival that hands the
// packed stage back to the TMA producer) while the shared-memory load is still in flight.
__device__ __forceinline__ uint32_t high_nibbles_now(uint32_t packed) {
  uint32_t r;
  asm volatile("and.b32 %0, %1, 0xF0F0F0F0;" : "=r"(r) : "r"(packed));
  return r;
}

// 32 consecutive 32-bit columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_store32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until the shared-memory sources of all earlier bulk stores of this thread have been read.
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairT::kThreads, 1)
w4a4_gemm_pair_tmem_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                           const __grid_constant__ CUtensorMap map_y, const Params p) {
  using T = PairT;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);

  const uint32_t wide_base = base;                                             // int8 B stages
  const uint32_t packed_base = wide_base + T::kStages * T::kWideB;             // packed A + B stages
  const uint32_t out_base = packed_base + T::kPackedStages * T::kPackedStageBytes;  // fp16 output staging
  const uint32_t dw_base = out_base + T::kOutBytes;                            // weight steps of the current tile
  const uint32_t bar_base = dw_base + T::kDwBytes;
  // full[s]: A slot s written in both CTAs' tensor memory and B stage s written in both CTAs' shared
  // memory (collected in the leader); empty[s]: the MMAs that read them have completed (both CTAs).
  auto full = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (T::kStages + s); };
  auto pk_full = [&](int s) { return bar_base + 8u * (2 * T::kStages + s); };
  auto pk_empty = [&](int s) { return bar_base + 8u * (2 * T::kStages + T::kPackedStages + s); };
  const uint32_t acc_full = bar_base + 8u * (2 * T::kStages + 2 * T::kPackedStages);
  const uint32_t acc_empty = acc_full + 8u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + (bar_base - base) + 8 * T::kNumBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < T::kStages; ++s) {
      mbar_init(full(s), 2 * T::kArrivalsPerStage);   // widen warps of both CTAs (used in the leader only)
      mbar_init(empty(s), 1);
    }
    for (int s = 0; s < T::kPackedStages; ++s) {
      mbar_init(pk_full(s), 1);
      mbar_init(pk_empty(s), T::kArrivalsPerStage);
    }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 2 * kEpiWarps);     // epilogue warps of both CTAs (used in the leader only)
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(uint32_t(T::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_a_ring = tmem_base + uint32_t(T::kAccCols);

  // a unit of work is (tile, k-split); with k-splits the int32 partial sums go to the workspace
  const int tiles_ab = p.tiles_a * p.tiles_b;
  const int total_tiles = tiles_ab * p.splits;
  const int first_tile = blockIdx.x >> 1;
  const int tile_step = gridDim.x >> 1;
  const int kblocks = p.kblocks / p.splits;   // host guarantees divisibility

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (each CTA, own rows)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
        const int ta = (tile % tiles_ab) % p.tiles_a;
        const int tb = (tile % tiles_ab) / p.tiles_a;
        const int kb0 = (tile / tiles_ab) * kblocks;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % T::kPackedStages;
          const uint32_t ph = (it / T::kPackedStages) & 1u;
          if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag, kSiteProducer)) { ok = false; break; }
          mbar_expect_tx(pk_full(s), uint32_t(T::kPackedA + T::kPackedB));
          const uint32_t dst = packed_base + s * T::kPackedStageBytes;
          tma_load_2d(dst, &map_a, pk_full(s), (kb0 + kb) * kPackedRow, ta * 256 + int(rank) * kBM);
          tma_load_2d(dst + T::kPackedA, &map_b, pk_full(s), (kb0 + kb) * kPackedRow,
                      tb * T::kBN + int(rank) * T::kHalfN);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = make_idesc_i8_pair(T::kBN);
      uint32_t it = 0, local_tile = 0;
      bool ok = true;
      for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++local_tile) {
        if (!mbar_wait(acc_empty, (local_tile & 1u) ^ 1u, abort_flag, kSiteMmaAcc)) break;
        tcgen05_fence_after();
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % T::kStages;
          const uint32_t ph = (it / T::kStages) & 1u;
          if (!mbar_wait(full(s), ph, abort_flag, kSiteMmaWide)) { ok = false; break; }
          tcgen05_fence_after();
          const uint64_t db = make_desc_sw128(wide_base + s * T::kWideB);
          const uint32_t ta_addr = tmem_a_ring + uint32_t(s * 32);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)   // 32 int8 of K: 8 columns of A, 32 bytes of B's swizzle atom
            mma_i8_pair_ts(tmem_base, ta_addr + uint32_t(8 * k4), db + uint64_t(2 * k4), idesc,
                           (kb > 0 || k4 > 0) ? 1u : 0u);
          tcgen05_commit_pair(empty(s));
        }
        if (ok) tcgen05_commit_pair(acc_full);
      }
    }
  } else if (warp < 2 + T::kAWidenWarps) {
    // ------------------------------------------------------------ A-widen warps: packed rows -> tensor memory
    const int q = warp & 3;               // tensor-memory lane quadrant this warp may write
    const uint32_t set = uint32_t(warp - 2) >> 2;   // which k-blocks this warp takes
    const int row = q * 32 + lane;        // A row inside the CTA's 128 = tensor-memory lane
    const uint32_t sw = uint32_t((row >> 1) & 3);
    uint32_t it = 0;
    bool ok = true;
    for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
      for (int kb = 0; kb < kblocks; ++kb, ++it) {
        const int ps = it % T::kPackedStages;
        const uint32_t pph = (it / T::kPackedStages) & 1u;
        const int s = it % T::kStages;
        const uint32_t sph = (it / T::kStages) & 1u;
        if ((it % T::kWidenSets) != set) continue;
        if (!mbar_wait(pk_full(ps), pph, abort_flag, kSiteWidenFull)) { ok = false; break; }
        const uint32_t src = packed_base + ps * T::kPackedStageBytes + row * kPackedRow;
        uint32_t x[16];
#pragma unroll
        for (int c = 0; c < 4; ++c)
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(x[4 * c]), "=r"(x[4 * c + 1]), "=r"(x[4 * c + 2]), "=r"(x[4 * c + 3])
                       : "r"(src + ((uint32_t(c) ^ sw) << 4)) : "memory");
        // Same order of k inside a k-block as the B side: per 32 packed codes, the 16 even codes
        // (low nibbles) first, then the 16 odd codes.
        uint32_t r[32];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            r[8 * c + i] = (x[4 * c + i] << 4) & 0xF0F0F0F0u;
            r[8 * c + 4 + i] = high_nibbles_now(x[4 * c + i]);
          }
        }
        // the packed stage is in registers (the instructions above have consumed every loaded
        // word): give it back to the producer before waiting for a slot
        __syncwarp();
        if (lane == 0) mbar_arrive(pk_empty(ps));
        if (!mbar_wait(empty(s), sph ^ 1u, abort_flag, kSiteWidenEmpty)) { ok = false; break; }
        tcgen05_fence_after();
        tmem_store32(tmem_a_ring + (uint32_t(q * 32) << 16) + uint32_t(s * 32), r);
        tmem_wait_st();
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (leader) mbar_arrive(full(s));
          else mbar_arrive_cluster(map_to_cta(full(s), 0));
        }
      }
    }
  } else if (warp < 2 + T::kAWidenWarps + T::kBWidenWarps) {
    // ------------------------------------------------------------ B-widen warps: packed rows -> int8 tile
    const int w = (warp - 2 - T::kAWidenWarps) & 3;
    const uint32_t set = uint32_t(warp - 2 - T::kAWidenWarps) >> 2;   // which k-blocks this warp takes
    const int r = lane & 7;
    const int c = lane >> 3;
    constexpr int kGroups = T::kHalfN / 8;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
      for (int kb = 0; kb < kblocks; ++kb, ++it) {
        const int ps = it % T::kPackedStages;
        const uint32_t pph = (it / T::kPackedStages) & 1u;
        const int s = it % T::kStages;
        const uint32_t sph = (it / T::kStages) & 1u;
        if ((it % T::kWidenSets) != set) continue;
        if (!mbar_wait(pk_full(ps), pph, abort_flag, kSiteWidenFull)) { ok = false; break; }
        const uint32_t pk = packed_base + ps * T::kPackedStageBytes + T::kPackedA;
        const uint32_t wd = wide_base + s * T::kWideB;
        constexpr int kPerWarp = kGroups / 4;
        uint32_t x[kPerWarp][4];
#pragma unroll
        for (int u = 0; u < kPerWarp; ++u) {
          const int row = (w + u * 4) * 8 + r;
          const uint32_t src = pk + row * kPackedRow + ((c ^ ((row >> 1) & 3)) << 4);
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(x[u][0]), "=r"(x[u][1]), "=r"(x[u][2]), "=r"(x[u][3]) : "r"(src) : "memory");
        }
        uint32_t hi[kPerWarp][4];
#pragma unroll
        for (int u = 0; u < kPerWarp; ++u) {
#pragma unroll
          for (int i = 0; i < 4; ++i) hi[u][i] = high_nibbles_now(x[u][i]);
        }
        // the packed stage is in registers (every loaded word has been consumed above): give it
        // back to the producer before waiting for a stage
        __syncwarp();
        if (lane == 0) mbar_arrive(pk_empty(ps));
        if (!mbar_wait(empty(s), sph ^ 1u, abort_flag, kSiteWidenEmpty)) { ok = false; break; }
#pragma unroll
        for (int u = 0; u < kPerWarp; ++u) {
          const int row = (w + u * 4) * 8 + r;
          const uint32_t dst_row = wd + row * kWideRow;
          const uint32_t lo_dst = dst_row + (((2 * c) ^ (row & 7)) << 4);
          const uint32_t hi_dst = dst_row + (((2 * c + 1) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(lo_dst), "r"((x[u][0] << 4) & 0xF0F0F0F0u), "r"((x[u][1] << 4) & 0xF0F0F0F0u),
                         "r"((x[u][2] << 4) & 0xF0F0F0F0u), "r"((x[u][3] << 4) & 0xF0F0F0F0u) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(hi_dst), "r"(hi[u][0]), "r"(hi[u][1]), "r"(hi[u][2]), "r"(hi[u][3]) : "memory");
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          if (leader) mbar_arrive(full(s));
          else mbar_arrive_cluster(map_to_cta(full(s), 0));
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps (each CTA, own 128 rows)
    const int q = warp & 3;               // tensor-memory lane quadrant this warp may read
    const uint32_t out_warp = out_base + uint32_t(q) * uint32_t(4 * T::kOutBoxBytes);
    const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16);
    const uint32_t dw_warp = dw_base + uint32_t(q) * uint32_t(T::kBN * 4);
    uint32_t local_tile = 0;
    for (int tile = first_tile; tile < total_tiles; tile += tile_step, ++local_tile) {
      const int ta = (tile % tiles_ab) % p.tiles_a;
      const int tb = (tile % tiles_ab) / p.tiles_a;
      const int split = tile / tiles_ab;
      const int row0 = ta * 256 + int(rank) * kBM + q * 32;
      const int a = row0 + lane;
      float sx = 0.0f;
      if (p.Y != nullptr) {
        // fetch the scales while the tile is still being accumulated: this warp's copy of the
        // tile's 256 weight steps goes to shared memory, the token step stays in a register
        const int n = tb * T::kBN + lane * 8;
        float4 w0 = make_float4(0.f, 0.f, 0.f, 0.f), w1 = w0;
        if (n + 8 <= p.rows_b) {
          w0 = __ldg(reinterpret_cast<const float4*>(p.dw + n));
          w1 = __ldg(reinterpret_cast<const float4*>(p.dw + n + 4));
        }
        if (a < p.rows_a) sx = __ldg(p.dx + a) * 0.00390625f;   // accumulators are 256 * acc
        float4* dst = reinterpret_cast<float4*>(smem + (dw_warp - base)) + lane * 2;
        dst[0] = w0;
        dst[1] = w1;
        __syncwarp();
      }
      if (!mbar_wait(acc_full, local_tile & 1u, abort_flag, kSiteEpilogue)) break;
      tcgen05_fence_after();
      if (p.Y != nullptr) {
        // the staging boxes of the previous tile must have been read by their TMA stores
        if (lane == 0) tma_store_wait_read();
        __syncwarp();
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
          const uint32_t box = out_warp + uint32_t(cb * T::kOutBoxBytes);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t regs[32];
            tmem_load32(taddr + uint32_t(cb * 64 + h * 32), regs);
            tmem_wait_ld();
            if (cb == 3 && h == 1) {
              // the accumulator is in registers or staged: hand tensor memory back to the MMA warp
              tcgen05_fence_before();
              __syncwarp();
              if (lane == 0) {
                if (leader) mbar_arrive(acc_empty);
                else mbar_arrive_cluster(map_to_cta(acc_empty, 0));
              }
            }
            const int n0 = cb * 64 + h * 32;   // column inside the tile
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              const float4* wsrc = reinterpret_cast<const float4*>(smem + (dw_warp - base)) + (n0 + 8 * jj) / 4;
              const float4 w0 = wsrc[0], w1 = wsrc[1];
              const float ws[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
              uint32_t o[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float v0 = float(int32_t(regs[8 * jj + 2 * e])) * (sx * ws[2 * e]);
                const float v1 = float(int32_t(regs[8 * jj + 2 * e + 1])) * (sx * ws[2 * e + 1]);
                const __half2 hv = __floats2half2_rn(v0, v1);
                o[e] = *reinterpret_cast<const uint32_t*>(&hv);
              }
              const uint32_t chunk = uint32_t(h * 4 + jj) ^ uint32_t(lane & 7);   // 128-byte swizzle of the store map
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                           ::"r"(box + uint32_t(lane) * 128u + (chunk << 4)), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3])
                           : "memory");
            }
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            const int x = tb * T::kBN + cb * 64;
            if (x < p.rows_b && row0 < p.rows_a) tma_store_2d(&map_y, box, x, row0);   // TMA clips the ragged edges
          }
        }
        if (lane == 0) tma_store_commit();
      } else {
        // int32 accumulators (partial sums of a k-split, or the test export): plain stores
#pragma unroll 1
        for (int c0 = 0; c0 < T::kBN; c0 += 32) {
          uint32_t regs[32];
          tmem_load32(taddr + uint32_t(c0), regs);
          tmem_wait_ld();
          store_columns<32>(p, a, tb * T::kBN + c0, split, regs);
          __syncwarp();
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (leader) mbar_arrive(acc_empty);
          else mbar_arrive_cluster(map_to_cta(acc_empty, 0));
        }
      }
    }
    if (lane == 0) tma_store_wait_all();
  }

  // A CTA that gave up tells its peer, which would otherwise wait for its own limit (the peer is
  // still resident: it cannot pass the cluster barrier below before this CTA arrives there).
  if (*abort_flag != 0)
    asm volatile("st.shared::cluster.u32 [%0], %1;"
                 ::"r"(map_to_cta(smem_u32(const_cast<const int*>(abort_flag)), rank ^ 1u)), "r"(1u) : "memory");
  drain_after_abort(abort_flag);
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs are done with both halves of tensor memory
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"(uint32_t(T::kTmemCols)) : "memory");
  }
}

// ---------------------------------------------------------------------------
// Weight-streaming kernel for up to 128 tokens per tile (short prompts, batched decode beyond
// the reach of the decode kernel).
//
// The layer is then bound by the one pass over the packed weights, so the
// kernel is built around that stream: output channels sit on the 128-row MMA
// axis (operand A), the tokens on the N axis (BN = 128; narrower tiles are supported by the
// template but lost to this one or to the decode kernel on every shape measured), K is split
// across CTAs so that every SM streams.  As in the two-CTA kernel the streamed
// operand never returns to shared memory: TMA delivers 64 packed bytes per
// weight row and k-block, four A-widen warps (one per tensor-memory lane
// quadrant) widen them in registers and tcgen05.st them into a ring of slots
// in tensor memory, and the MMA takes A from there.  Only the token tile
// (BN x 128 bytes per k-block) is widened into shared memory.  Per k-block a
// CTA moves 16 KB of weight bytes through shared memory (TMA write + one read)
// instead of 40 KB.  One CTA computes one (channel tile, k-split) and leaves;
// two CTAs fit an SM (<= 256 tensor-memory columns each), which hides the fill
// and drain of the short pipelines.  Partial sums of a split go to the
// workspace as int32 and splitk_reduce_kernel adds them and dequantizes.
// ---------------------------------------------------------------------------
template <int BN>
struct Stream {
  static_assert(BN == 32 || BN == 64 || BN == 128, "token tile");
  static constexpr int kStages = BN <= 64 ? 6 : 4;       // A slots in tensor memory = token stages in shared memory
  static constexpr int kPackedStages = 6;
  static constexpr int kPackedA = kBM * kPackedRow;      // 8 KB of weights
  static constexpr int kPackedB = BN * kPackedRow;
  static constexpr int kPackedBPad = (kPackedB + 1023) / 1024 * 1024;
  static constexpr int kPackedStageBytes = kPackedA + kPackedBPad;
  static constexpr int kWideB = BN * kWideRow;
  static constexpr int kWideBPad = (kWideB + 1023) / 1024 * 1024;
  // with the 128-token tile two sets of widen warps take the k-blocks in turn
  static constexpr int kSets = BN >= 128 ? 2 : 1;
  static constexpr int kBPerSet = BN >= 128 ? 4 : (BN >= 64 ? 2 : 1);
  static constexpr int kAWidenWarps = 4 * kSets, kBWidenWarps = kBPerSet * kSets;
  static constexpr int kArrivals = 4 + kBPerSet;          // per k-block
  static constexpr int kThreads = 32 * (2 + kAWidenWarps + kBWidenWarps + kEpiWarps);
  static constexpr int kNumBarriers = 2 * kStages + 2 * kPackedStages + 1;
  static constexpr int kSmemBytes = 1024 + kStages * kWideBPad + kPackedStages * kPackedStageBytes +
                                    kNumBarriers * 8 + 16;
  static constexpr int kTmemCols = 256;                  // accumulator (BN columns) + A ring (32 per slot)
  static constexpr int kAccCols = BN;
  static constexpr int kRingCol = BN <= 64 ? 64 : 128;   // the A ring starts here
  static_assert(kRingCol + 32 * kStages <= kTmemCols && kAccCols <= kRingCol, "tensor-memory budget");
};

__device__ __forceinline__ void mma_i8_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

template <int BN>
__global__ void __launch_bounds__(Stream<BN>::kThreads, BN >= 128 ? 1 : 2)
w4a4_gemm_stream_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                        const Params p) {
  using T = Stream<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);

  const uint32_t wide_base = base;                                            // int8 token stages
  const uint32_t packed_base = wide_base + T::kStages * T::kWideBPad;         // packed weights + tokens
  const uint32_t bar_base = packed_base + T::kPackedStages * T::kPackedStageBytes;
  auto full = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (T::kStages + s); };
  auto pk_full = [&](int s) { return bar_base + 8u * (2 * T::kStages + s); };
  auto pk_empty = [&](int s) { return bar_base + 8u * (2 * T::kStages + T::kPackedStages + s); };
  const uint32_t acc_full = bar_base + 8u * (2 * T::kStages + 2 * T::kPackedStages);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + (bar_base - base) + 8 * T::kNumBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < T::kStages; ++s) {
      mbar_init(full(s), T::kArrivals);
      mbar_init(empty(s), 1);
    }
    for (int s = 0; s < T::kPackedStages; ++s) {
      mbar_init(pk_full(s), 1);
      mbar_init(pk_empty(s), T::kArrivals);
    }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(uint32_t(T::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_a_ring = tmem_base + uint32_t(T::kRingCol);

  // this CTA's work: channel tile ta, token tile tb, k-split
  // (the k-splits of a tile are neighbours in blockIdx.x, so that they can form a cluster)
  const int split = blockIdx.x % p.splits;
  const int tile = blockIdx.x / p.splits;
  const int ta = tile % p.tiles_a;
  const int tb = tile / p.tiles_a;
  const int kb_count = p.kblocks / p.splits;   // host guarantees divisibility
  const int kb0 = split * kb_count;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int it = 0; it < kb_count; ++it) {
        const int s = it % T::kPackedStages;
        const uint32_t ph = uint32_t(it / T::kPackedStages) & 1u;
        if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag, kSiteProducer)) break;
        mbar_expect_tx(pk_full(s), uint32_t(T::kPackedA + T::kPackedB));
        const uint32_t dst = packed_base + s * T::kPackedStageBytes;
        tma_load_2d(dst, &map_a, pk_full(s), (kb0 + it) * kPackedRow, ta * kBM);
        tma_load_2d(dst + T::kPackedA, &map_b, pk_full(s), (kb0 + it) * kPackedRow, tb * BN);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_i8(BN);
      bool ok = true;
      for (int it = 0; it < kb_count; ++it) {
        const int s = it % T::kStages;
        const uint32_t ph = uint32_t(it / T::kStages) & 1u;
        if (!mbar_wait(full(s), ph, abort_flag, kSiteMmaWide)) { ok = false; break; }
        tcgen05_fence_after();
        const uint64_t db = make_desc_sw128(wide_base + s * T::kWideBPad);
        const uint32_t ta_addr = tmem_a_ring + uint32_t(s * 32);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
          mma_i8_ts(tmem_base, ta_addr + uint32_t(8 * k4), db + uint64_t(2 * k4), idesc, (it > 0 || k4 > 0) ? 1u : 0u);
        tcgen05_commit(empty(s));
      }
      if (ok) tcgen05_commit(acc_full);
    }
  } else if (warp < 2 + T::kAWidenWarps) {
    // ------------------------------------------------------------ A-widen warps: packed weight rows -> tensor memory
    const int q = warp & 3;
    const int set = (warp - 2) >> 2;
    const int row = q * 32 + lane;
    const uint32_t sw = uint32_t((row >> 1) & 3);
    for (int it = set; it < kb_count; it += T::kSets) {
      const int ps = it % T::kPackedStages;
      const uint32_t pph = uint32_t(it / T::kPackedStages) & 1u;
      const int s = it % T::kStages;
      const uint32_t sph = uint32_t(it / T::kStages) & 1u;
      if (!mbar_wait(pk_full(ps), pph, abort_flag, kSiteWidenFull)) break;
      const uint32_t src = packed_base + ps * T::kPackedStageBytes + row * kPackedRow;
      uint32_t x[16];
#pragma unroll
      for (int c = 0; c < 4; ++c)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(x[4 * c]), "=r"(x[4 * c + 1]), "=r"(x[4 * c + 2]), "=r"(x[4 * c + 3])
                     : "r"(src + ((uint32_t(c) ^ sw) << 4)) : "memory");
      uint32_t r[32];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          r[8 * c + i] = (x[4 * c + i] << 4) & 0xF0F0F0F0u;
          r[8 * c + 4 + i] = high_nibbles_now(x[4 * c + i]);
        }
      }
      // every loaded word has been consumed: the packed stage can go back to the producer
      __syncwarp();
      if (lane == 0) mbar_arrive(pk_empty(ps));
      if (!mbar_wait(empty(s), sph ^ 1u, abort_flag, kSiteWidenEmpty)) break;
      tcgen05_fence_after();
      tmem_store32(tmem_a_ring + (uint32_t(q * 32) << 16) + uint32_t(s * 32), r);
      tmem_wait_st();
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(full(s));
    }
  } else if (warp < 2 + T::kAWidenWarps + T::kBWidenWarps) {
    // ------------------------------------------------------------ B-widen warps: packed token rows -> int8 tile
    const int w = (warp - 2 - T::kAWidenWarps) % T::kBPerSet;
    const int set = (warp - 2 - T::kAWidenWarps) / T::kBPerSet;
    const int r = lane & 7;
    const int c = lane >> 3;
    constexpr int kGroups = BN / 8;
    for (int it = set; it < kb_count; it += T::kSets) {
      const int ps = it % T::kPackedStages;
      const uint32_t pph = uint32_t(it / T::kPackedStages) & 1u;
      const int s = it % T::kStages;
      const uint32_t sph = uint32_t(it / T::kStages) & 1u;
      if (!mbar_wait(pk_full(ps), pph, abort_flag, kSiteWidenFull)) break;
      if (!mbar_wait(empty(s), sph ^ 1u, abort_flag, kSiteWidenEmpty)) break;
      const uint32_t pk = packed_base + ps * T::kPackedStageBytes + T::kPackedA;
      const uint32_t wd = wide_base + s * T::kWideBPad;
#pragma unroll
      for (int g = w; g < kGroups; g += T::kBPerSet) {
        const int row = g * 8 + r;
        const uint32_t src = pk + row * kPackedRow + ((c ^ ((row >> 1) & 3)) << 4);
        const uint32_t dst_row = wd + row * kWideRow;
        uint32_t x0, x1, x2, x3;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3) : "r"(src) : "memory");
        const uint32_t lo_dst = dst_row + (((2 * c) ^ (row & 7)) << 4);
        const uint32_t hi_dst = dst_row + (((2 * c + 1) ^ (row & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(lo_dst), "r"((x0 << 4) & 0xF0F0F0F0u), "r"((x1 << 4) & 0xF0F0F0F0u),
                       "r"((x2 << 4) & 0xF0F0F0F0u), "r"((x3 << 4) & 0xF0F0F0F0u) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(hi_dst), "r"(x0 & 0xF0F0F0F0u), "r"(x1 & 0xF0F0F0F0u),
                       "r"(x2 & 0xF0F0F0F0u), "r"(x3 & 0xF0F0F0F0u) : "memory");
      }
      // the stores above consumed the loaded words, so the packed stage is free as well
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(full(s));
        mbar_arrive(pk_empty(ps));
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int e = warp & 3;
    if (mbar_wait(acc_full, 0u, abort_flag, kSiteEpilogue)) {
      tcgen05_fence_after();
      const int a = ta * kBM + e * 32 + lane;
      const uint32_t taddr = tmem_base + (uint32_t(e * 32) << 16);
      if (p.cluster_reduce) {
        // this split's partial sums, token-major [BN][128] int32, over the int8 token stages
        // (every MMA that read them has completed)
        const uint32_t dst = wide_base + uint32_t(e * 32 + lane) * 4u;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t regs[32];
          tmem_load32(taddr + uint32_t(c0), regs);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst + uint32_t(c0 + j) * 512u), "r"(regs[j]) : "memory");
        }
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t regs[32];
          tmem_load32(taddr + uint32_t(c0), regs);
          tmem_wait_ld();
          store_columns<32>(p, a, tb * BN + c0, split, regs);
          __syncwarp();
        }
      }
    }
  }

  drain_after_abort(abort_flag);
  tcgen05_fence_before();
  __syncthreads();
  if (p.cluster_reduce) {
    // The CTAs of a cluster hold the partial sums of one tile for their k-splits.  Each CTA
    // adds up a slice of 128 / splits channels over all of them, read through the cluster's
    // shared-memory window, and writes the finished outputs.
    cluster_sync_all();
    const int slice = kBM / p.splits;              // 16, 32 or 64 channels
    const int tokens = min(BN, p.rows_b - tb * BN);
    const int n_local0 = split * slice;
    const int quads = slice / 4;                   // a thread adds up 4 consecutive channels of one token
    for (int idx = threadIdx.x; idx < tokens * quads; idx += T::kThreads) {
      const int mi = idx / quads;                  // token inside the tile
      const int nl = n_local0 + (idx % quads) * 4; // first channel inside the tile
      const uint32_t off = wide_base + uint32_t(mi * kBM + nl) * 4u;
      int4 part[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        part[r] = make_int4(0, 0, 0, 0);
        if (r < p.splits)
          asm volatile("ld.shared::cluster.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(part[r].x), "=r"(part[r].y), "=r"(part[r].z), "=r"(part[r].w)
                       : "r"(map_to_cta(off, uint32_t(r))) : "memory");
      }
      int sum[4] = {0, 0, 0, 0};
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        sum[0] += part[r].x; sum[1] += part[r].y; sum[2] += part[r].z; sum[3] += part[r].w;
      }
      const int n = ta * kBM + nl;
      const int m = tb * BN + mi;
      if (n < p.rows_a) {                          // channel counts are multiples of 8: all four or none
        if (p.Y != nullptr) {
          const float sx = __ldg(p.dx + m);
          const float4 sw = __ldg(reinterpret_cast<const float4*>(p.dw + n));
          const __half2 h0 = __floats2half2_rn(float(sum[0] >> 8) * (sx * sw.x), float(sum[1] >> 8) * (sx * sw.y));
          const __half2 h1 = __floats2half2_rn(float(sum[2] >> 8) * (sx * sw.z), float(sum[3] >> 8) * (sx * sw.w));
          uint2 out;
          out.x = *reinterpret_cast<const uint32_t*>(&h0);
          out.y = *reinterpret_cast<const uint32_t*>(&h1);
          *reinterpret_cast<uint2*>(p.Y + int64_t(m) * p.ldy + n) = out;
        } else {
          *reinterpret_cast<int4*>(p.acc_out + int64_t(m) * p.N + n) =
              make_int4(sum[0] >> 8, sum[1] >> 8, sum[2] >> 8, sum[3] >> 8);
        }
      }
    }
    cluster_sync_all();   // nobody leaves while its shared memory may still be read
  }
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"(uint32_t(T::kTmemCols)) : "memory");
  }
}

// Sums the split-K partials and applies the dequantization (or writes the int32 sum).
// A thread owns 8 consecutive output channels of one token (N is a multiple of 8).
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const int32_t* __restrict__ part, int splits, int M, int N,
                     const float* __restrict__ dx, const float* __restrict__ dw,
                     __half* __restrict__ Y, int64_t ldy, int32_t* __restrict__ acc_out) {
  const int n8 = N >> 3;
  const int64_t idx = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= int64_t(M) * n8) return;
  const int m = int(idx / n8);
  const int n = int(idx - int64_t(m) * n8) * 8;
  const int64_t plane = int64_t(M) * N;
  const int4* src = reinterpret_cast<const int4*>(part + int64_t(m) * N + n);
  int4 s0 = make_int4(0, 0, 0, 0), s1 = s0;
  for (int s = 0; s < splits; ++s) {
    const int4 a = __ldcs(src), b = __ldcs(src + 1);   // read once: keep the partials out of the way in L2
    s0.x += a.x; s0.y += a.y; s0.z += a.z; s0.w += a.w;
    s1.x += b.x; s1.y += b.y; s1.z += b.z; s1.w += b.w;
    src += plane / 4;
  }
  if (Y != nullptr) {
    const float sx = __ldg(dx + m);
    const float4 w0 = __ldg(reinterpret_cast<const float4*>(dw + n));
    const float4 w1 = __ldg(reinterpret_cast<const float4*>(dw + n + 4));
    uint4 out;
    __half2* h = reinterpret_cast<__half2*>(&out);
    h[0] = __floats2half2_rn(float(s0.x) * (sx * w0.x), float(s0.y) * (sx * w0.y));
    h[1] = __floats2half2_rn(float(s0.z) * (sx * w0.z), float(s0.w) * (sx * w0.w));
    h[2] = __floats2half2_rn(float(s1.x) * (sx * w1.x), float(s1.y) * (sx * w1.y));
    h[3] = __floats2half2_rn(float(s1.z) * (sx * w1.z), float(s1.w) * (sx * w1.w));
    *reinterpret_cast<uint4*>(Y + int64_t(m) * ldy + n) = out;
  } else {
    int4* o = reinterpret_cast<int4*>(acc_out + int64_t(m) * N + n);
    o[0] = s0;
    o[1] = s1;
  }
}

// ---------------------------------------------------------------------------
// Decode kernel for few tokens (M <= 8 * NT, NT = 1, 2, 4, 8 token tiles).
//
// With a handful of tokens the layer is one pass over the packed weights and nothing else,
// and the tensor-memory kernels spend more time on their set-up (cluster launch, tensor-memory
// allocation, barrier chains, a reduction over k-splits) than on the stream.  This kernel has
// no set-up at all: a CTA of 8 warps owns 16 * RG weight rows, its warps take the rows'
// 64-byte chunks in turn (a split of K inside the CTA), and every lane loads 16 bytes of two
// weight rows and 16 bytes of one token's codes straight from global memory.  The products
// are formed by the warp-level integer MMA (16 rows x 8 tokens x 32 codes per instruction),
// used here as a dot-product engine for a kernel that is bound by HBM: its operands are the
// same 16 * code int8 words as above (low nibbles and high nibbles of a packed word go to
// different k slots of the instruction, for weights and tokens alike, and a dot product does
// not care about the order of its terms).  Sums are int32 (256 * acc), added over the warps in
// shared memory in a fixed order: exact, and identical from run to run.
// ---------------------------------------------------------------------------
// NT: token tiles of 8 (M <= 8 * NT); RG: row groups of 16 per CTA; U: chunks per batch and warp (two
// batches are in flight); WARPS: warps per CTA, which split K between them.
template <int NT, int RG, int U>
struct DecodeBatch {
  uint4 w[U][RG][2];
  uint4 x[U][NT];
};

template <int NT, int RG, int U, int WARPS>
__device__ __forceinline__ void decode_load(DecodeBatch<NT, RG, U>& b, const uint8_t* const (&wrow)[RG][2],
                                            const uint8_t* const (&xrow)[NT], const bool (&xvalid)[NT], int c0,
                                            int chunks) {
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int cc = c0 + u * WARPS;
    const bool on = cc < chunks;
#pragma unroll
    for (int rg = 0; rg < RG; ++rg)
#pragma unroll
      for (int h = 0; h < 2; ++h) b.w[u][rg][h] = on ? load_stream_16(wrow[rg][h] + cc * 64) : zero;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) b.x[u][nt] = (on && xvalid[nt]) ? load_keep_16(xrow[nt] + cc * 64) : zero;
  }
}

template <int NT, int RG, int U>
__device__ __forceinline__ void decode_accumulate(const DecodeBatch<NT, RG, U>& b, int (&c)[RG][NT][4]) {
#pragma unroll
  for (int u = 0; u < U; ++u) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t b0[NT], b1[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const uint32_t xw = word_of(b.x[u][nt], i);
        b0[nt] = even_codes_x16(xw);
        b1[nt] = odd_codes_x16(xw);
      }
#pragma unroll
      for (int rg = 0; rg < RG; ++rg) {
        const uint32_t wa = word_of(b.w[u][rg][0], i), wb = word_of(b.w[u][rg][1], i);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
          mma_s8_16x8x32(c[rg][nt], even_codes_x16(wa), even_codes_x16(wb), odd_codes_x16(wa), odd_codes_x16(wb),
                         b0[nt], b1[nt]);
      }
    }
  }
}

template <int NT, int RG, int U, int WARPS, bool PIPE>
__global__ void __launch_bounds__(WARPS * 32)
w4a4_decode_kernel(const uint8_t* __restrict__ Xq, const uint8_t* __restrict__ Wq, int M, int N, int K,
                   const float* __restrict__ dx, const float* __restrict__ dw, __half* __restrict__ Y, int64_t ldy,
                   int32_t* __restrict__ acc_out) {
  constexpr int kOutputs = RG * NT * 128;          // outputs of the CTA, tokens past M included
  constexpr int kPerThread = (kOutputs + WARPS * 32 - 1) / (WARPS * 32);
  __shared__ int red[WARPS][kOutputs];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int row_base = blockIdx.x * (16 * RG);
  const int chunks = K / 128;                    // 64-byte chunks of a packed row
  const int64_t row_bytes = K / 2;

  // a row past the end repeats the last one, a token past the end contributes zeros
  const uint8_t* wrow[RG][2];
#pragma unroll
  for (int rg = 0; rg < RG; ++rg)
#pragma unroll
    for (int h = 0; h < 2; ++h)
      wrow[rg][h] = Wq + int64_t(min(row_base + rg * 16 + h * 8 + g, N - 1)) * row_bytes + t * 16;
  const uint8_t* xrow[NT];
  bool xvalid[NT];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    xvalid[nt] = nt * 8 + g < M;
    xrow[nt] = Xq + int64_t(min(nt * 8 + g, M - 1)) * row_bytes + t * 16;
  }

  DecodeBatch<NT, RG, U> cur;
  decode_load<NT, RG, U, WARPS>(cur, wrow, xrow, xvalid, warp, chunks);

  // the scales of this thread's outputs arrive while the weights stream
  float scale[kPerThread];
#pragma unroll
  for (int j = 0; j < kPerThread; ++j) {
    const int o = threadIdx.x + j * WARPS * 32;
    const int tile = o >> 7, i = o & 127;
    const int m = (tile % NT) * 8 + (i >> 4);
    const int n = row_base + (tile / NT) * 16 + (i & 15);
    scale[j] = (Y != nullptr && o < kOutputs && m < M && n < N) ? __ldg(dx + m) * __ldg(dw + n) : 0.0f;
  }

  int c[RG][NT][4];
#pragma unroll
  for (int rg = 0; rg < RG; ++rg)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) c[rg][nt][i] = 0;

  if constexpr (PIPE) {                  // long rows: the next batch is on its way during the MMAs
    DecodeBatch<NT, RG, U> nxt;
    for (int c0 = warp; c0 < chunks; c0 += WARPS * U) {
      const int c1 = c0 + WARPS * U;
      if (c1 < chunks) decode_load<NT, RG, U, WARPS>(nxt, wrow, xrow, xvalid, c1, chunks);
      decode_accumulate<NT, RG, U>(cur, c);
      cur = nxt;
    }
  } else {                               // short rows: one batch (or few) per warp, more CTAs per SM instead
    for (int c0 = warp; c0 < chunks; c0 += WARPS * U) {
      if (c0 != warp) decode_load<NT, RG, U, WARPS>(cur, wrow, xrow, xvalid, c0, chunks);
      decode_accumulate<NT, RG, U>(cur, c);
    }
  }

  // lane (g, t) holds rows g and g + 8, tokens 2t and 2t + 1 of every 16 x 8 tile; tiles are
  // laid out token-major in shared memory so that the final stores run along the channels
#pragma unroll
  for (int rg = 0; rg < RG; ++rg)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      int* tile = &red[warp][(rg * NT + nt) * 128];
      tile[(2 * t) * 16 + g] = c[rg][nt][0];
      tile[(2 * t + 1) * 16 + g] = c[rg][nt][1];
      tile[(2 * t) * 16 + g + 8] = c[rg][nt][2];
      tile[(2 * t + 1) * 16 + g + 8] = c[rg][nt][3];
    }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < kPerThread; ++j) {
    const int o = threadIdx.x + j * WARPS * 32;
    if (o < kOutputs) {
      int sum = 0;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) sum += red[w][o];
      sum >>= 8;                                   // the sums are 256 * acc, exactly
      const int tile = o >> 7, i = o & 127;
      const int m = (tile % NT) * 8 + (i >> 4);
      const int n = row_base + (tile / NT) * 16 + (i & 15);
      if (m < M && n < N) {
        if (Y != nullptr)
          Y[int64_t(m) * ldy + n] = __float2half_rn(float(sum) * scale[j]);
        else
          acc_out[int64_t(m) * N + n] = sum;
      }
    }
  }
}

template <int NT, int RG, int U, int WARPS, bool PIPE>
static int launch_decode(const uint8_t* Xq, const uint8_t* Wq, int M, int N, int K, const float* dx, const float* dw,
                         __half* Y, int64_t ldy, int32_t* acc_out, cudaStream_t st) {
  const int grid = (N + 16 * RG - 1) / (16 * RG);
  w4a4_decode_kernel<NT, RG, U, WARPS, PIPE><<<grid, WARPS * 32, 0, st>>>(Xq, Wq, M, N, K, dx, dw, Y, ldy, acc_out);
  count_launch();
  return launch_status();
}

// Test probe: one warp waits, through the same bounded wait as the kernels above, on an mbarrier
// that nobody ever arrives on.  The wait runs out after g_wait_limit_ns, records kSiteProbe in the
// status word and the kernel returns normally.
__global__ void wait_expiry_probe_kernel() {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int abort_word;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  volatile int* abort_flag = &abort_word;
  (void)mbar_wait(bar, 0u, abort_flag, kSiteProbe);
  drain_after_abort(abort_flag);
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
struct Plan {
  bool gemv;      // few tokens: the decode kernel
  bool swapped;
  bool pair;      // two-CTA kernel, 256 x 256 pair tiles
  bool cluster;   // the k-splits of a tile form a cluster and add up in shared memory (no workspace)
  int bn;
  int splits;
};

// Number of SMs of the current device, remembered per device.
static int sm_count() {
  constexpr int kSlots = 64;
  static std::atomic<int> cached[kSlots];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kSlots) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

constexpr int kPairSplitMinBlocks = 32;   // k-blocks per split below which the extra pass over the partial sums costs more than it saves

// Clusters of `size` CTAs of the streaming kernel that the device runs at the same time.  A cluster
// stays inside one GPC, so large clusters leave SMs unused: 148 / 74 / 33 / 15 clusters of
// 1 / 2 / 4 / 8 on B200.  Asked of the runtime once per device; a conservative guess without one.
static int active_clusters(int size) {
  constexpr int kSlots = 64;
  static std::atomic<int> cached[kSlots][4];
  const int idx = size >= 8 ? 3 : size >= 4 ? 2 : size >= 2 ? 1 : 0;
  const int guess = size <= 1 ? sm_count() : sm_count() / size * 7 / 8;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kSlots) return guess;
  int n = cached[dev][idx].load(std::memory_order_relaxed);
  if (n > 0) return n;
  auto kern = w4a4_gemm_stream_kernel<128>;
  n = 0;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Stream<128>::kSmemBytes) == cudaSuccess) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(size * 32), 1, 1);
    cfg.blockDim = dim3(unsigned(Stream<128>::kThreads), 1, 1);
    cfg.dynamicSmemBytes = size_t(Stream<128>::kSmemBytes);
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = unsigned(size);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) n = 0;
  }
  if (n <= 0) {
    (void)cudaGetLastError();
    return guess;
  }
  cached[dev][idx].store(n, std::memory_order_relaxed);
  return n;
}

// How the streaming kernel would split K for this shape.
struct StreamPlan {
  int splits;
  bool cluster;
  int ctas;
};

static StreamPlan plan_stream(int64_t M, int64_t N, int kblocks) {
  const int tiles = int((N + kBM - 1) / kBM) * int((M + 127) / 128);
  const int slots = sm_count();   // one CTA of the streaming kernel per SM
  // as many k-splits as keep all CTAs in one wave (a second wave costs a second fill and drain:
  // 128 tokens x 6144 channels took 24 us with 4 splits in two waves, 17 us with 2 splits in one)
  int want = slots / tiles;
  if (want < 1) want = 1;
  // Workspace path: the largest divisor of kblocks that does not exceed `want` and leaves >= 4
  // k-blocks per split.  Cluster path: the same among 1, 2, 4, 8 (portable cluster sizes that
  // divide the 128 channels of a tile), as long as the device runs that many clusters at once.
  // The cluster path needs no workspace and no second kernel, so it is taken unless the workspace
  // path offers at least four times the CTAs while the cluster path would leave more than half
  // of the machine idle.
  int splits = 1, csplits = 1;
  for (int s = 1; s <= kblocks && s <= want; ++s)
    if (kblocks % s == 0 && kblocks / s >= 4) splits = s;
  for (int s = 2; s <= 8 && s <= want; s *= 2)
    if (kblocks % s == 0 && kblocks / s >= 4 && tiles <= active_clusters(s)) csplits = s;
  StreamPlan sp{};
  if (splits >= 4 * csplits && 2 * csplits * tiles < slots) {
    sp.cluster = false;
    sp.splits = splits;
  } else {
    sp.cluster = csplits > 1;
    sp.splits = csplits;
  }
  sp.ctas = tiles * sp.splits;
  return sp;
}

static Plan make_plan(int64_t M, int64_t N, int64_t K) {
  Plan pl{};
  const int kblocks = int(K / kWideRow);
  // The decode kernel (no tiles, no k-splits, no workspace) up to 32 tokens, and up to 64 where the
  // weights are small enough that the tokens' codes, which every CTA reads from L2, do not dominate.
  if (M <= 32 || (M <= 64 && N * K <= (int64_t(1) << 25))) {
    pl.gemv = true;
    pl.splits = 1;
    return pl;
  }
  // The two-CTA kernel works on 256 x 256 tiles, one per SM pair; with few tiles and a long K two
  // k-splits per tile put twice as many pairs to work (partial sums through the workspace).
  const int64_t pair_tiles = ((M + 255) / 256) * ((N + 255) / 256);
  const int pairs = sm_count() / 2;
  const int pair_splits =
      (2 * pair_tiles <= pairs && kblocks % 2 == 0 && kblocks / 2 >= kPairSplitMinBlocks) ? 2 : 1;
  const StreamPlan sp = plan_stream(M, N, kblocks);
  bool to_stream;
  if (N < 256) {
    // no pair tiles: the streaming kernel up to 512 tokens, the one-CTA kernel beyond
    to_stream = M <= 512;
  } else {
    // Between the two, the estimated time decides (microseconds, fitted to graph-replay timings of
    // 72 shapes with 96..768 tokens on B200: a fixed part and a cost per k-block and wave).
    const int64_t pair_waves = (pair_tiles * pair_splits + pairs - 1) / pairs;
    const double pair_us = 10.2 + 0.35 * double(kblocks / pair_splits) * double(pair_waves) + (pair_splits > 1 ? 5.8 : 0.0);
    const int64_t stream_waves = (sp.ctas + sm_count() - 1) / sm_count();
    const double stream_us = (sp.cluster ? 10.7 : (sp.splits > 1 ? 16.7 : 15.6)) +
                             0.32 * double(kblocks / sp.splits) * double(stream_waves);
    to_stream = stream_us < pair_us;
  }
  if (!to_stream) {
    pl.swapped = false;
    pl.pair = N >= 256;
    pl.bn = N > 64 ? 128 : 64;   // of the one-CTA kernel that serves N < 256
    pl.splits = pl.pair ? pair_splits : 1;
    return pl;
  }
  pl.swapped = true;
  pl.bn = 128;   // narrower token tiles were slower than this one on every shape they served
  pl.cluster = sp.cluster;
  pl.splits = sp.splits;
  return pl;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// A tensor map is a pure function of (address, shape, box); the last few are kept so that repeated
// eager calls on the same buffers (a layer called once per step) do not encode them again.
template <typename Build>
static bool cached_map(CUtensorMap* map, int kind, const void* ptr, int64_t d0, int64_t d1, int64_t d2, Build build) {
  struct Entry {
    int kind;
    const void* ptr;
    int64_t d0, d1, d2;
    CUtensorMap map;
  };
  constexpr int kEntries = 16;
  static std::mutex mu;
  static Entry table[kEntries];
  static int filled = 0, next = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < filled; ++i) {
      const Entry& e = table[i];
      if (e.kind == kind && e.ptr == ptr && e.d0 == d0 && e.d1 == d1 && e.d2 == d2) {
        *map = e.map;
        return true;
      }
    }
  }
  if (!build(map)) return false;
  std::lock_guard<std::mutex> lock(mu);
  table[next] = Entry{kind, ptr, d0, d1, d2, *map};
  next = (next + 1) % kEntries;
  if (filled < kEntries) ++filled;
  return true;
}

// 2-D map over a packed matrix [rows x K/2] bytes, box = 64 bytes x box_rows, 64-byte swizzle.
static bool make_map(CUtensorMap* map, const uint8_t* ptr, int64_t rows, int64_t K, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  return cached_map(map, 0, ptr, rows, K, box_rows, [&](CUtensorMap* out) {
    const cuuint64_t dims[2] = {cuuint64_t(K / 2), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(K / 2)};
    const cuuint32_t box[2] = {cuuint32_t(kPackedRow), cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  });
}

// 2-D map over the fp16 output [M x ldy], box = 64 columns x 32 rows, 128-byte swizzle (TMA stores).
static bool make_map_y(CUtensorMap* map, __half* Y, int64_t M, int64_t N, int64_t ldy) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  return cached_map(map, 1, Y, M, N, ldy, [&](CUtensorMap* out) {
    const cuuint64_t dims[2] = {cuuint64_t(N), cuuint64_t(M)};
    const cuuint64_t strides[1] = {cuuint64_t(ldy) * sizeof(__half)};
    const cuuint32_t box[2] = {64, 32};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
  });
}

// Raises a kernel's dynamic shared-memory limit; once per kernel, device and process.  kTag tells
// the kernels apart (several share one function type, so the type alone would not).
template <int kTag, typename Kern>
static bool allow_smem(Kern kern, int bytes) {
  constexpr int kSlots = 64;
  static std::atomic<int> done[kSlots];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kSlots) dev = kSlots - 1;
  if (done[dev].load(std::memory_order_acquire) >= bytes) return true;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  done[dev].store(bytes, std::memory_order_release);
  return true;
}

template <int BN>
static int launch_stream(const CUtensorMap& ma, const CUtensorMap& mb, const Params& p, cudaStream_t st) {
  auto kern = w4a4_gemm_stream_kernel<BN>;
  if (!allow_smem<1000 + BN>(kern, Stream<BN>::kSmemBytes)) return SMOOTHROT_CUDA_ERROR;
  const int total = p.tiles_a * p.tiles_b * p.splits;   // one CTA per (channel tile, token tile, k-split)
  if (p.cluster_reduce) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(total), 1, 1);
    cfg.blockDim = dim3(unsigned(Stream<BN>::kThreads), 1, 1);
    cfg.dynamicSmemBytes = size_t(Stream<BN>::kSmemBytes);
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = unsigned(p.splits);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, ma, mb, p) != cudaSuccess) {
      (void)cudaGetLastError();
      return SMOOTHROT_CUDA_ERROR;
    }
    count_launch();
    return launch_status();
  }
  kern<<<total, Stream<BN>::kThreads, Stream<BN>::kSmemBytes, st>>>(ma, mb, p);
  count_launch();
  return launch_status();
}

template <int BN>
static int launch_tile(const CUtensorMap& ma, const CUtensorMap& mb, const Params& p, cudaStream_t st) {
  auto kern = w4a4_gemm_kernel<BN>;
  if (!allow_smem<2000 + BN>(kern, Tile<BN>::kSmemBytes)) return SMOOTHROT_CUDA_ERROR;
  const int total = p.tiles_a * p.tiles_b * p.splits;
  const int grid = total < sm_count() ? total : sm_count();
  kern<<<grid, kThreads, Tile<BN>::kSmemBytes, st>>>(ma, mb, p);
  count_launch();
  return launch_status();
}

static int launch_splitk_reduce(const void* workspace, int splits, int64_t M, int64_t N, const float* dx,
                                const float* dw, __half* Y, int64_t ldy, int32_t* acc_out, cudaStream_t st) {
  const int64_t total = M * (N / 8);
  const int threads = 256;
  splitk_reduce_kernel<<<unsigned((total + threads - 1) / threads), threads, 0, st>>>(
      static_cast<const int32_t*>(workspace), splits, int(M), int(N), dx, dw, Y, ldy, acc_out);
  count_launch();
  return launch_status();
}

// Argument checks shared by every entry point of the layer.  Returns SMOOTHROT_OK with *empty set
// when there is nothing to compute.
static int check_args(const uint8_t* Xq, const float* dx, int64_t M, const uint8_t* Wq, const float* dw, int64_t N,
                      int64_t K, const __half* Y, int64_t ldy, const int32_t* acc_out, bool* empty) {
  *empty = false;
  if (M < 0 || N < 0 || K <= 0) return SMOOTHROT_INVALID_ARG;
  if (K % kWideRow != 0 || K > 65536) return SMOOTHROT_UNSUPPORTED_K;
  if (N % 8 != 0) return SMOOTHROT_INVALID_ARG;
  if (M == 0 || N == 0) {
    *empty = true;
    return SMOOTHROT_OK;
  }
  if (M > 0x7fffffffLL / 2 || N > 0x7fffffffLL / 2) return SMOOTHROT_INVALID_ARG;
  if (Xq == nullptr || Wq == nullptr) return SMOOTHROT_INVALID_ARG;
  if (!aligned16(Xq) || !aligned16(Wq)) return SMOOTHROT_BAD_ALIGNMENT;
  if (Y != nullptr) {
    if (dx == nullptr || dw == nullptr || ldy < N) return SMOOTHROT_INVALID_ARG;
    if (!aligned16(Y) || ldy % 8 != 0 || !aligned16(dw)) return SMOOTHROT_BAD_ALIGNMENT;
  } else {
    if (acc_out == nullptr) return SMOOTHROT_INVALID_ARG;
    if (!aligned16(acc_out)) return SMOOTHROT_BAD_ALIGNMENT;
  }
  return SMOOTHROT_OK;
}

static int run(const uint8_t* Xq, const float* dx, int64_t M, const uint8_t* Wq, const float* dw, int64_t N,
               int64_t K, __half* Y, int64_t ldy, int32_t* acc_out, void* workspace, size_t workspace_bytes,
               cudaStream_t st) {
  bool empty = false;
  const int args_rc = check_args(Xq, dx, M, Wq, dw, N, K, Y, ldy, acc_out, &empty);
  if (args_rc != SMOOTHROT_OK || empty) return args_rc;
  Plan pl = make_plan(M, N, K);
  size_t need = (pl.splits > 1 && !pl.cluster) ? size_t(pl.splits) * size_t(M) * size_t(N) * sizeof(int32_t) : 0;
  if (pl.pair && need > 0 && (workspace == nullptr || workspace_bytes < need)) {
    // the two-CTA kernel splits K only to fill idle SM pairs: without the workspace it runs unsplit
    pl.splits = 1;
    need = 0;
  }
  if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return SMOOTHROT_WORKSPACE_TOO_SMALL;
  if (need > 0 && !aligned16(workspace)) return SMOOTHROT_BAD_ALIGNMENT;

  if (pl.gemv) {
    // Short rows fit one batch of loads per warp, and many small CTAs per SM keep the memory system
    // busy; long rows (K > 4096) want the double-buffered loop, and with two token tiles the codes of
    // the tokens are worth sharing between two row groups.
    int32_t* out32 = Y ? nullptr : acc_out;
    const int m = int(M), n = int(N), k = int(K);
#define SR_DECODE(NT, RG, U, W, P) launch_decode<NT, RG, U, W, P>(Xq, Wq, m, n, k, dx, dw, Y, ldy, out32, st)
    if (M <= 8) return K > 4096 ? SR_DECODE(1, 1, 4, 8, true) : SR_DECODE(1, 1, 4, 8, false);
    if (M <= 16) return K > 4096 ? SR_DECODE(2, 2, 2, 16, true) : SR_DECODE(2, 1, 4, 8, false);
    if (M <= 32) return N >= 8192 ? SR_DECODE(4, 2, 1, 8, true) : SR_DECODE(4, 1, 2, 8, false);
    return SR_DECODE(8, 1, 1, 8, false);
#undef SR_DECODE
  }
  Params p{};
  p.swapped = pl.swapped ? 1 : 0;
  const uint8_t* a_ptr = pl.swapped ? Wq : Xq;
  const uint8_t* b_ptr = pl.swapped ? Xq : Wq;
  p.rows_a = int(pl.swapped ? N : M);
  p.rows_b = int(pl.swapped ? M : N);
  p.tiles_a = (p.rows_a + kBM - 1) / kBM;
  p.tiles_b = (p.rows_b + pl.bn - 1) / pl.bn;
  p.kblocks = int(K / kWideRow);
  p.splits = pl.splits;
  p.cluster_reduce = pl.cluster ? 1 : 0;
  p.M = int(M);
  p.N = int(N);
  p.dx = dx;
  p.dw = dw;
  p.ldy = ldy;
  if (pl.splits > 1 && !pl.cluster) {
    p.Y = nullptr;
    p.acc_out = static_cast<int32_t*>(workspace);
  } else {
    p.Y = Y;
    p.acc_out = Y ? nullptr : acc_out;
  }
  CUtensorMap ma, mb;
  if (pl.pair) {
    p.tiles_a = (p.rows_a + 255) / 256;
    p.tiles_b = (p.rows_b + PairT::kBN - 1) / PairT::kBN;
    if (!make_map(&ma, a_ptr, p.rows_a, K, kBM) || !make_map(&mb, b_ptr, p.rows_b, K, PairT::kHalfN))
      return SMOOTHROT_CUDA_ERROR;
    CUtensorMap my = ma;   // only read by the kernel when Y is written
    if (p.Y != nullptr && !make_map_y(&my, p.Y, M, N, ldy)) return SMOOTHROT_CUDA_ERROR;
    auto kern = w4a4_gemm_pair_tmem_kernel;
    if (!allow_smem<3000>(kern, PairT::kSmemBytes)) return SMOOTHROT_CUDA_ERROR;
    const int total = p.tiles_a * p.tiles_b * pl.splits;
    const int pairs = sm_count() / 2;
    const int grid = 2 * (total < pairs ? total : pairs);
    kern<<<grid, PairT::kThreads, PairT::kSmemBytes, st>>>(ma, mb, my, p);
    count_launch();
    const int rc = launch_status();
    if (rc != SMOOTHROT_OK || pl.splits == 1) return rc;
    return launch_splitk_reduce(workspace, pl.splits, M, N, dx, dw, Y, ldy, acc_out, st);
  }
  if (!make_map(&ma, a_ptr, p.rows_a, K, kBM) || !make_map(&mb, b_ptr, p.rows_b, K, pl.bn))
    return SMOOTHROT_CUDA_ERROR;
  int rc;
  if (pl.swapped) {
    rc = launch_stream<128>(ma, mb, p, st);
  } else
  rc = pl.bn == 128 ? launch_tile<128>(ma, mb, p, st) : launch_tile<64>(ma, mb, p, st);
  if (rc != SMOOTHROT_OK) return rc;
  if (pl.splits > 1 && !pl.cluster) rc = launch_splitk_reduce(workspace, pl.splits, M, N, dx, dw, Y, ldy, acc_out, st);
  return rc;
}

// ---------------------------------------------------------------------------
// Built-in scratch for smoothrot_linear_static_scratch: split-K partial sums
// for callers that have no way to provide a workspace of their own.  The array
// is part of the loaded module, so every device that loads the library holds
// these bytes until the process exits.
// ---------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = size_t(SMOOTHROT_STATIC_SCRATCH_BYTES);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::atomic<void*> g_static_scratch_addr[kMaxDevices];

// Device address of g_static_scratch on the current device.  In host code the
// array's name is only a handle for the runtime; the address a kernel can use
// has to be asked for, once per device, with that device current.
static int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SMOOTHROT_CUDA_ERROR;
  void* p = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    void* sym = nullptr;
    if (cudaGetSymbolAddress(&sym, g_static_scratch) != cudaSuccess || sym == nullptr) {
      (void)cudaGetLastError();
      return SMOOTHROT_CUDA_ERROR;
    }
    g_static_scratch_addr[dev].store(sym, std::memory_order_release);
    p = sym;
  }
  *out = p;
  return SMOOTHROT_OK;
}

}  // namespace gemm
}  // namespace smoothrot

extern "C" {

int smoothrot_linear_static_scratch(const uint8_t* Xq, const float* dx, int64_t M, const uint8_t* Wq,
                                    const float* dw, int64_t N, int64_t K, void* Y_f16, int64_t ldy,
                                    void* stream) {
  using namespace smoothrot::gemm;
  if (M > 0 && N > 0 && Y_f16 == nullptr) return SMOOTHROT_INVALID_ARG;
  // the same argument checks, in the same order, as smoothrot_linear: only a valid call can be
  // refused for its size
  bool empty = false;
  const int args_rc = check_args(Xq, dx, M, Wq, dw, N, K, static_cast<const __half*>(Y_f16), ldy, nullptr, &empty);
  if (args_rc != SMOOTHROT_OK || empty) return args_rc;
  size_t need = smoothrot_workspace_bytes(M, N, K);
  if (need > kStaticScratchBytes) {
    // prefill shapes split K only as an optimisation and run without scratch memory as well
    if (M <= 0 || N <= 0 || K <= 0 || !make_plan(M, N, K).pair) return SMOOTHROT_STATIC_SCRATCH_EXCEEDED;
    need = 0;
  }
  void* scratch = nullptr;
  if (need > 0) {
    const int rc = static_scratch_address(&scratch);
    if (rc != SMOOTHROT_OK) return rc;
  }
  // Every partial sum the reduction reads is written by the GEMM kernel of the
  // same call, so nothing left in the array by an earlier call is ever read
  // and nothing has to be cleared.
  return run(Xq, dx, M, Wq, dw, N, K, static_cast<__half*>(Y_f16), ldy, nullptr, scratch,
             need > 0 ? kStaticScratchBytes : 0, static_cast<cudaStream_t>(stream));
}

int smoothrot_debug_set_wait_limit_ns(uint64_t ns) {
  const unsigned long long v = ns == 0 ? smoothrot::gemm::kWaitLimitNs : static_cast<unsigned long long>(ns);
  if (cudaMemcpyToSymbol(smoothrot::gemm::g_wait_limit_ns, &v, sizeof(v)) != cudaSuccess) return SMOOTHROT_CUDA_ERROR;
  return smoothrot_rotate_set_wait_limit_ns(ns);
}

int smoothrot_debug_wait_expiry(void* stream) {
  smoothrot::gemm::wait_expiry_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>();
  smoothrot::count_launch();
  return smoothrot::launch_status();
}

const char* smoothrot_linear_plan_name(int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0 || K % smoothrot::gemm::kWideRow != 0) return "none";
  const smoothrot::gemm::Plan pl = smoothrot::gemm::make_plan(M, N, K);
  if (pl.gemv) return "w4a4_decode_kernel";
  if (pl.swapped) return pl.cluster ? "w4a4_gemm_stream_kernel (k-splits in a cluster)"
                                    : (pl.splits > 1 ? "w4a4_gemm_stream_kernel + splitk_reduce_kernel"
                                                     : "w4a4_gemm_stream_kernel");
  if (pl.pair) return pl.splits > 1 ? "w4a4_gemm_pair_tmem_kernel + splitk_reduce_kernel" : "w4a4_gemm_pair_tmem_kernel";
  return "w4a4_gemm_kernel";
}

size_t smoothrot_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0 || K % smoothrot::gemm::kWideRow != 0) return 0;
  const smoothrot::gemm::Plan pl = smoothrot::gemm::make_plan(M, N, K);
  return (pl.splits > 1 && !pl.cluster) ? size_t(pl.splits) * size_t(M) * size_t(N) * sizeof(int32_t) : 0;
}

int smoothrot_linear(const uint8_t* Xq, const float* dx, int64_t M, const uint8_t* Wq, const float* dw,
                     int64_t N, int64_t K, void* Y_f16, int64_t ldy, void* workspace, size_t workspace_bytes,
                     void* stream) {
  if (M > 0 && N > 0 && Y_f16 == nullptr) return SMOOTHROT_INVALID_ARG;
  return smoothrot::gemm::run(Xq, dx, M, Wq, dw, N, K, static_cast<__half*>(Y_f16), ldy, nullptr, workspace,
                              workspace_bytes, static_cast<cudaStream_t>(stream));
}

int smoothrot_debug_gemm_i32(const uint8_t* Xq, int64_t M, const uint8_t* Wq, int64_t N, int64_t K,
                             int32_t* acc, void* workspace, size_t workspace_bytes, void* stream) {
  if (M > 0 && N > 0 && acc == nullptr) return SMOOTHROT_INVALID_ARG;
  return smoothrot::gemm::run(Xq, nullptr, M, Wq, nullptr, N, K, nullptr, 0, acc, workspace, workspace_bytes,
                              static_cast<cudaStream_t>(stream));
}

int smoothrot_device_status(int* status_host, int clear) {
  if (status_host == nullptr) return SMOOTHROT_INVALID_ARG;
  int v = 0, rot = 0;
  if (cudaMemcpyFromSymbol(&v, smoothrot::gemm::g_device_status, sizeof(int)) != cudaSuccess)
    return SMOOTHROT_CUDA_ERROR;
  if (smoothrot_rotate_status_word(&rot, clear) != SMOOTHROT_OK) return SMOOTHROT_CUDA_ERROR;
  *status_host = v != 0 ? v : rot;
  if (clear && v != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(smoothrot::gemm::g_device_status, &zero, sizeof(int)) != cudaSuccess)
      return SMOOTHROT_CUDA_ERROR;
  }
  return SMOOTHROT_OK;
}

}  // extern "C"
