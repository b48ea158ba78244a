// Row transform kernels of libsmoothrot:  v = (x * pre) H / sqrt(K)  followed by
// per-row symmetric 4-bit quantization and packing (two codes per byte).
//
// Serves three entry points: smoothrot_quant_act (online activation path),
// smoothrot_fuse_weights (offline weight path, same map with another diagonal
// and clip ratio) and smoothrot_debug_hadamard (the rotation alone, fp32 out).
//
// Kernels
//   rotate_generic_kernel   any supported K; one CTA per row, the row lives in
//                           shared memory as fp32, butterflies three bits at a
//                           time, the order-12, -20 or -28 factor by a table product.
//   walsh4096_kernel        K = 4096: 64 threads per row, 64 values per thread,
//                           6 + 6 butterfly stages in registers around one
//                           shared-memory transpose, codes assembled with warp
//                           shuffles so that every global access is coalesced.
//   paley512_kernel         K = 14336 = 28 x 512: see below.
#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "rowquant.cuh"

namespace smoothrot {

// ---------------------------------------------------------------------------
// Order-28 Hadamard matrix, Paley construction I over GF(27).
// GF(27) = GF(3)[x]/(x^3 + 2x + 1); element (c0, c1, c2) has index c0 + 3 c1 + 9 c2.
// ---------------------------------------------------------------------------
struct Gf27 {
  int c0, c1, c2;
};

__host__ __device__ constexpr Gf27 gf_from_index(int e) { return Gf27{e % 3, (e / 3) % 3, e / 9}; }
__host__ __device__ constexpr int gf_to_index(Gf27 v) { return v.c0 + 3 * v.c1 + 9 * v.c2; }

__host__ __device__ constexpr Gf27 gf_diff(Gf27 a, Gf27 b) {
  return Gf27{(a.c0 - b.c0 + 3) % 3, (a.c1 - b.c1 + 3) % 3, (a.c2 - b.c2 + 3) % 3};
}

// Product modulo x^3 + 2x + 1:  x^3 = x + 2 and x^4 = x^2 + 2x over GF(3).
__host__ __device__ constexpr Gf27 gf_prod(Gf27 a, Gf27 b) {
  int p0 = a.c0 * b.c0;
  int p1 = a.c0 * b.c1 + a.c1 * b.c0;
  int p2 = a.c0 * b.c2 + a.c1 * b.c1 + a.c2 * b.c0;
  int p3 = a.c1 * b.c2 + a.c2 * b.c1;
  int p4 = a.c2 * b.c2;
  return Gf27{(p0 + 2 * p3) % 3, (p1 + p3 + 2 * p4) % 3, (p2 + p4) % 3};
}

// Quadratic character by Euler's criterion: e^((27-1)/2) is 1 on squares, -1 otherwise.
__host__ __device__ constexpr int gf_character(int e) {
  if (e == 0) return 0;
  Gf27 base = gf_from_index(e);
  Gf27 acc = Gf27{1, 0, 0};
  for (int i = 0; i < 13; ++i) acc = gf_prod(acc, base);
  return gf_to_index(acc) == 1 ? 1 : -1;
}

// H28[r][c]: first row all +1, first column +1 then -1, core I + chi(r - c).
__host__ __device__ constexpr int paley28_entry(int r, int c) {
  if (r == 0) return 1;
  if (c == 0) return -1;
  if (r == c) return 1;
  return gf_character(gf_to_index(gf_diff(gf_from_index(r - 1), gf_from_index(c - 1))));
}

struct Paley28Table {
  float v[28][28];
};

constexpr Paley28Table make_paley28_table() {
  Paley28Table t{};
  for (int r = 0; r < 28; ++r)
    for (int c = 0; c < 28; ++c) t.v[r][c] = float(paley28_entry(r, c));
  return t;
}

__constant__ Paley28Table c_paley28 = make_paley28_table();

// Orders 12 and 20: Paley construction I over the prime fields GF(11) and GF(19), elements
// 0..q-1 in natural order, same border as above.  (Widths 12 * 2^p and 20 * 2^p; an addition,
// the paper's models need 2^p and 28 * 2^p only.)
__host__ __device__ constexpr int prime_character(int e, int q) {
  e = ((e % q) + q) % q;
  if (e == 0) return 0;
  int acc = 1;                                 // Euler's criterion: e^((q-1)/2) mod q
  for (int i = 0; i < (q - 1) / 2; ++i) acc = (acc * e) % q;
  return acc == 1 ? 1 : -1;
}

__host__ __device__ constexpr int paley_prime_entry(int q, int r, int c) {
  if (r == 0) return 1;
  if (c == 0) return -1;
  if (r == c) return 1;
  return prime_character((r - 1) - (c - 1), q);
}

template <int kOrder>
struct PaleyTable {
  float v[kOrder][kOrder];
};

template <int kOrder>
constexpr PaleyTable<kOrder> make_paley_prime_table() {
  PaleyTable<kOrder> t{};
  for (int r = 0; r < kOrder; ++r)
    for (int c = 0; c < kOrder; ++c) t.v[r][c] = float(paley_prime_entry(kOrder - 1, r, c));
  return t;
}

__constant__ PaleyTable<12> c_paley12 = make_paley_prime_table<12>();
__constant__ PaleyTable<20> c_paley20 = make_paley_prime_table<20>();

// ---------------------------------------------------------------------------
// Small device helpers
// ---------------------------------------------------------------------------
__device__ __forceinline__ void unpack8_f16(const uint4& raw, float* f) {
  const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// SiLU(g) * u, the gated product of Fig. 2, in fp32 with the library exponential and an IEEE
// division (a few ulp).  Large |g| is safe: exp(-g) = inf gives g / inf = -0, exp(-g) = 0 gives g.
__device__ __forceinline__ float glu_product(float g, float u) {
  return __fdiv_rn(g, 1.0f + expf(-g)) * u;
}

// ---------------------------------------------------------------------------
// Generic kernel: one CTA per row.
// ---------------------------------------------------------------------------
constexpr int kGenericThreads = 256;

template <int kOrder>
__device__ __forceinline__ void base_product(float* row, const float (&table)[kOrder][kOrder], int n, int tid) {
  for (int b = tid; b < n; b += kGenericThreads) {
    float xin[kOrder], yv[kOrder];
#pragma unroll
    for (int a = 0; a < kOrder; ++a) xin[a] = row[a * n + b];
#pragma unroll
    for (int c = 0; c < kOrder; ++c) {
      float acc = 0.0f;
#pragma unroll
      for (int a = 0; a < kOrder; ++a) acc = fmaf(xin[a], table[a][c], acc);
      yv[c] = acc;
    }
#pragma unroll
    for (int c = 0; c < kOrder; ++c) row[c * n + b] = yv[c];
  }
  __syncthreads();
}

template <bool kQuant, bool kGlu>
__global__ void __launch_bounds__(kGenericThreads)
rotate_generic_kernel(const __half* __restrict__ X, int64_t ldx, const __half* __restrict__ U, int64_t ldu,
                      int K, int base, int n, int logn,
                      const float* __restrict__ pre, float inv_sqrt_k, float clip,
                      uint8_t* __restrict__ q_out, float* __restrict__ step_out,
                      float* __restrict__ y_out) {
  extern __shared__ __align__(16) float row[];
  __shared__ float red[kGenericThreads / 32];
  const int tid = threadIdx.x;
  const int64_t m = blockIdx.x;
  const __half* x = X + m * ldx;

  for (int c = tid; c < K / 8; c += kGenericThreads) {
    uint4 raw = *reinterpret_cast<const uint4*>(x + c * 8);
    float f[8];
    unpack8_f16(raw, f);
    if (kGlu) {   // X holds the gate rows, U the up rows
      const uint4 raw_u = *reinterpret_cast<const uint4*>(U + m * ldu + c * 8);
      float u[8];
      unpack8_f16(raw_u, u);
#pragma unroll
      for (int i = 0; i < 8; ++i) f[i] = glu_product(f[i], u[i]);
    }
    if (pre != nullptr) {
#pragma unroll
      for (int i = 0; i < 8; ++i) f[i] *= pre[c * 8 + i];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) row[c * 8 + i] = f[i];
  }
  __syncthreads();

  // Walsh butterflies on the low `logn` index bits, up to three bits per pass.
  for (int s = 0; s < logn; s += 3) {
    const int nb = min(3, logn - s);
    const int cnt = 1 << nb;
    const int groups = K >> nb;
    for (int v = tid; v < groups; v += kGenericThreads) {
      const int lo = v & ((1 << s) - 1);
      const int hi = v >> s;
      const int idx0 = lo | (hi << (s + nb));
      float e[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) e[i] = (i < cnt) ? row[idx0 + (i << s)] : 0.0f;
#pragma unroll
      for (int h = 1; h < 8; h <<= 1) {
        if (h < cnt) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if ((i & h) == 0) {
              float a = e[i], b = e[i + h];
              e[i] = a + b;
              e[i + h] = a - b;
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (i < cnt) row[idx0 + (i << s)] = e[i];
    }
    __syncthreads();
  }

  // Paley factor on the slow index a of j = a * n + b:  y[a'] = sum_a x[a] H[a][a'].
  if (base == 28) base_product<28>(row, c_paley28.v, n, tid);
  else if (base == 20) base_product<20>(row, c_paley20.v, n, tid);
  else if (base == 12) base_product<12>(row, c_paley12.v, n, tid);

  if (!kQuant) {
    float* y = y_out + m * int64_t(K);
    for (int j = tid; j < K; j += kGenericThreads) y[j] = row[j] * inv_sqrt_k;
    return;
  }

  float amax = 0.0f;
  for (int j = tid; j < K; j += kGenericThreads) {
    float v = row[j] * inv_sqrt_k;
    row[j] = v;
    amax = fmaxf(amax, fabsf(v));
  }
  amax = warp_max(amax);
  if ((tid & 31) == 0) red[tid >> 5] = amax;
  __syncthreads();
  amax = red[0];
#pragma unroll
  for (int w = 1; w < kGenericThreads / 32; ++w) amax = fmaxf(amax, red[w]);
  const float step = step_from_absmax(amax, clip);
  if (tid == 0) step_out[m] = step;

  uint32_t* q = reinterpret_cast<uint32_t*>(q_out + m * int64_t(K / 2));
  for (int c = tid; c < K / 8; c += kGenericThreads) {
    uint32_t word = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float t = rintf(__fdiv_rn(row[c * 8 + i], step));
      t = fminf(fmaxf(t, -8.0f), 7.0f);
      word |= (uint32_t(int(t)) & 0xFu) << (4 * i);
    }
    q[c] = word;
  }
}

// ---------------------------------------------------------------------------
// K = 4096.  Persistent kernel: one CTA per SM, kW4096Groups (10) row groups of
// 64 threads (two warps) each; a group walks over rows  m, m + stride, ...
//
// The next row of a group is fetched by a bulk asynchronous copy
// (cp.async.bulk, completion on an mbarrier) into the group's transpose tile as
// soon as the tile has been read back (midway through the current row), so that
// loads stay in flight while the second half of the row's arithmetic runs.
//
// Index bits of a row position j (12 bits):  i = j[0:3), t = j[3:9), g = j[9:12).
//   phase 1  thread t reads the eight 16-byte chunks (g, t): values (g, i);
//            butterflies on the bits of i and g (6 stages, in registers).
//   transpose through shared memory: [t][g*8+i], row pitch 68 floats.
//   phase 2  thread (g, i) holds the 64 values over t; butterflies on the six
//            bits of t.  1/sqrt(4096) = 2^-6 is folded into the step size (exact).
//   absmax over the row, step size, rounding by the 1.5 * 2^23 trick, then the
//   codes travel between the lanes of a row group so that each lane ends up
//   with whole 32-bit words of packed output.
// ---------------------------------------------------------------------------
constexpr int kW4096Groups = 10;
constexpr int kW4096Threads = kW4096Groups * 64;
constexpr int kW4096Pitch = 68;  // floats per t-row in shared memory (64 + 4 pad)
constexpr int kW4096PreBytes = 4096 * 4;
constexpr int kW4096TileBytes = 64 * kW4096Pitch * 4;
constexpr int kW4096InBytes = 4096 * 2;
constexpr int kW4096GroupBytes = kW4096TileBytes;   // the next row lands in the tile's first 8 KB
constexpr int kW4096SmemBytes = kW4096PreBytes + kW4096Groups * kW4096GroupBytes + kW4096Groups * 8 + kW4096Groups * 4;
constexpr unsigned long long kLoadWaitLimitNs = 2000000000ull;  // 2 s

// Set when a bounded wait for a row copy ran out (read by smoothrot_device_status).
__device__ int g_rotate_status = 0;
// Limit of the bounded waits of the row kernels in nanoseconds (a test shortens it).
__device__ unsigned long long g_rotate_wait_limit_ns = kLoadWaitLimitNs;

__device__ __forceinline__ void group_barrier(int group) {
  asm volatile("bar.sync %0, 64;" ::"r"(group + 1) : "memory");
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool row_copy_done(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Waits (bounded) until the bulk copy that was started on `bar` has landed.
__device__ __forceinline__ bool wait_row_copy(uint32_t bar, uint32_t parity) {
  if (row_copy_done(bar, parity)) return true;
  unsigned long long t0;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (uint32_t spin = 1;; ++spin) {
    if (row_copy_done(bar, parity)) return true;
    if ((spin & 255u) == 0u) {
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (now - t0 > g_rotate_wait_limit_ns) {
        atomicCAS(&g_rotate_status, 0, 16);
        return false;
      }
    }
  }
}

// Starts the copy of one row (bytes, a multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void start_row_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Walsh butterflies on 2 * NP values held as NP pairs (pair k = values 2k, 2k+1).
// The stage inside a pair is scalar; every other stage works on whole pairs.
template <int NP>
__device__ __forceinline__ void butterflies_pairs(f32x2* v) {
#pragma unroll
  for (int k = 0; k < NP; ++k) {
    float a, b;
    unpack2(v[k], a, b);
    v[k] = pack2(a + b, a - b);
  }
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

// The stage inside each pair with instructions that stay where they are written: they consume
// every value just loaded from shared memory, so that the loads have completed before the code
// that follows (a barrier, then a bulk copy into the same memory) can run.
template <int NP>
__device__ __forceinline__ void butterflies_first_stage_in_place(f32x2* v) {
#pragma unroll
  for (int k = 0; k < NP; ++k) {
    float a, b, s, d;
    unpack2(v[k], a, b);
    asm volatile("add.f32 %0, %1, %2;" : "=f"(s) : "f"(a), "f"(b));
    asm volatile("sub.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    v[k] = pack2(s, d);
  }
}

// The remaining stages (between pairs) of butterflies_pairs.
template <int NP>
__device__ __forceinline__ void butterflies_between_pairs(f32x2* v) {
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

// kLowClamp: the general two-sided clamp, needed when the row maximum can reach 8.5 steps or more
// (clip ratios <= 7/8.5); otherwise only the code +8 can occur out of range and is fixed on the bytes.
template <bool kQuant, bool kHasPre, bool kLowClamp>
__global__ void __launch_bounds__(kW4096Threads, 1)
walsh4096_kernel(const __half* __restrict__ X, int64_t ldx, int64_t M,
                 const float* __restrict__ pre, float clip,
                 uint8_t* __restrict__ q_out, float* __restrict__ step_out,
                 float* __restrict__ y_out) {
  // shared memory: [pre: 4096 fp32][per group: transpose tile, also the landing place of the next row]
  //                [per group: mbarrier][per group: flag]
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ float red[kW4096Groups][2];
  const int group = threadIdx.x >> 6;
  const int t = threadIdx.x & 63;
  const int lane = threadIdx.x & 31;
  float* spre = reinterpret_cast<float*>(smem_raw);
  uint8_t* gbase = smem_raw + kW4096PreBytes + group * kW4096GroupBytes;
  float* tile = reinterpret_cast<float*>(gbase);
  const uint32_t inbuf = smem_addr(gbase);   // the input row shares the tile
  const uint32_t bar = smem_addr(smem_raw + kW4096PreBytes + kW4096Groups * kW4096GroupBytes + group * 8);
  volatile int* lost = reinterpret_cast<volatile int*>(smem_raw + kW4096PreBytes + kW4096Groups * kW4096GroupBytes +
                                                         kW4096Groups * 8) + group;

  if (kHasPre) {
    // the diagonal's 16-byte unit i = (g, t, half) goes to (g, half, t): the two units a thread reads
    // per chunk are then 1 KB apart and the lanes of a warp read consecutive units (no bank conflicts)
    for (int i = threadIdx.x; i < 1024; i += kW4096Threads)
      reinterpret_cast<float4*>(spre)[(i & ~127) | ((i & 1) << 6) | ((i >> 1) & 63)] =
          __ldg(reinterpret_cast<const float4*>(pre) + i);
  }
  if (t == 0) {
    *lost = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // rows of this group: blockIdx.x + gridDim.x * (group + kW4096Groups * k)
  const int64_t stride = int64_t(gridDim.x) * kW4096Groups;
  int64_t m = int64_t(blockIdx.x) + int64_t(gridDim.x) * group;
  if (t == 0 && m < M) start_row_copy(inbuf, X + m * ldx, kW4096InBytes, bar);
  uint32_t parity = 0;

  for (; m < M; m += stride) {
  // Every thread waits (bounded) for the row; a copy that never lands marks the group as lost and
  // the group leaves together after its next barrier.
  if (!wait_row_copy(bar, parity)) *lost = 1;
  parity ^= 1u;

  // The values stay unnormalised until the end: 1/sqrt(4096) = 2^-6 is exact,
  // so it is folded into the step size (or applied at the fp32 store).
  f32x2 v[32];
  {
    uint4 raw[8];
#pragma unroll
    for (int g = 0; g < 8; ++g)
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(raw[g].x), "=r"(raw[g].y), "=r"(raw[g].z), "=r"(raw[g].w)
                   : "r"(inbuf + uint32_t(g * 1024 + t * 16)) : "memory");
    group_barrier(group);   // the whole row is in registers: the tile can take the transposed values
    if (*lost != 0) break;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const uint32_t* h = reinterpret_cast<const uint32_t*>(&raw[g]);
      float4 p0, p1;
      if (kHasPre) {
        p0 = reinterpret_cast<const float4*>(spre)[g * 128 + t];
        p1 = reinterpret_cast<const float4*>(spre)[g * 128 + 64 + t];
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        f32x2 val = half2_to_f32x2(h[k]);   // on the FMA pipe; cvt.f32.f16 would queue on the conversion unit
        if (kHasPre) {
          const f32x2 pp = k == 0 ? pack2(p0.x, p0.y) : k == 1 ? pack2(p0.z, p0.w)
                         : k == 2 ? pack2(p1.x, p1.y) : pack2(p1.z, p1.w);
          val = mul2(val, pp);
        }
        v[g * 4 + k] = val;
      }
    }
  }
  butterflies_pairs<32>(v);  // value index = g * 8 + i: bits of i, then bits of g

  // transpose: thread t writes its 64 values as one padded row
  {
    float4* dst = reinterpret_cast<float4*>(tile + t * kW4096Pitch);
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float4 o;
      unpack2(v[2 * c], o.x, o.y);
      unpack2(v[2 * c + 1], o.z, o.w);
      dst[c] = o;
    }
  }
  group_barrier(group);
  // thread gi = t now owns position (g, i) = (t >> 3, t & 7) for all 64 values of the t-bits
#pragma unroll
  for (int u = 0; u < 32; ++u) v[u] = pack2(tile[(2 * u) * kW4096Pitch + t], tile[(2 * u + 1) * kW4096Pitch + t]);
  butterflies_first_stage_in_place<32>(v);   // every loaded value has been consumed
  group_barrier(group);                       // the tile is free: fetch the next row into it
  if (t == 0 && m + stride < M) start_row_copy(inbuf, X + (m + stride) * ldx, kW4096InBytes, bar);
  butterflies_between_pairs<32>(v);

  const int gi_g = t >> 3, gi_i = t & 7;
  if (!kQuant) {
    float* y = y_out + m * 4096;
#pragma unroll
    for (int u = 0; u < 32; ++u) {
      float a, b;
      unpack2(v[u], a, b);
      y[gi_g * 512 + (2 * u) * 8 + gi_i] = a * 0.015625f;
      y[gi_g * 512 + (2 * u + 1) * 8 + gi_i] = b * 0.015625f;
    }
    group_barrier(group);   // the tile is reused by the next row
    continue;
  }

  float am[4] = {0.0f, 0.0f, 0.0f, 0.0f};   // four chains: the maximum is not one long dependency
#pragma unroll
  for (int u = 0; u < 32; ++u) {
    float a, b;
    unpack2(v[u], a, b);
    am[u & 3] = fmaxf(fmaxf(am[u & 3], fabsf(a)), fabsf(b));
  }
  float amax = warp_max(fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])));
  if (lane == 0) red[group][t >> 5] = amax;
  group_barrier(group);
  amax = fmaxf(red[group][0], red[group][1]) * 0.015625f;   // now the absmax of the normalised row
  const float step = step_from_absmax(amax, clip);
  if (t == 0) step_out[m] = step;
  const float inv = __frcp_rn(step) * 0.015625f;            // 1/step for unnormalised values (exact scaling)
  const f32x2 inv2 = pack2(inv, inv);

  // Round to nearest even and bias by 8: the low byte of the float's bit
  // pattern is code + 8 in [0, 15].
  const float kMagic = 12582912.0f + 8.0f;  // 1.5 * 2^23 + 8
  const f32x2 magic2 = pack2(kMagic, kMagic);
  uint32_t spread[16];                      // four codes per word, one per byte
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    uint32_t r[4];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      float q0, q1;
      unpack2(fma2(v[2 * c + k], inv2, magic2), q0, q1);
      if (kLowClamp) {
        q0 = fmaxf(fminf(q0, 12582912.0f + 15.0f), 12582912.0f);
        q1 = fmaxf(fminf(q1, 12582912.0f + 15.0f), 12582912.0f);
      }
      r[2 * k] = __float_as_uint(q0);
      r[2 * k + 1] = __float_as_uint(q1);
    }
    const uint32_t lo = __byte_perm(r[0], r[1], 0x0040);  // bytes: r0.b0, r1.b0
    const uint32_t hi = __byte_perm(r[2], r[3], 0x0040);
    uint32_t four = __byte_perm(lo, hi, 0x5410);
    // Without the clamp above the row maximum sits below 8.5 steps, so a byte is code + 8 in
    // [0, 16]; the one value out of range, 16 (code +8), comes down to 15: subtract bit 4 of each byte.
    if (!kLowClamp) four -= (four >> 4) & 0x01010101u;
    spread[c] = four;
  }
  // Lanes 2p and 2p+1 hold the even and odd position of each byte.  The even
  // lane finishes the words with even c, the odd lane those with odd c.
  const bool odd = (gi_i & 1) != 0;
  uint32_t word[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint32_t give = odd ? spread[2 * c] : spread[2 * c + 1];
    const uint32_t keep = odd ? spread[2 * c + 1] : spread[2 * c];
    const uint32_t got = __shfl_xor_sync(0xffffffffu, give, 1);
    const uint32_t lo_n = odd ? got : keep;   // even position -> low nibble
    const uint32_t hi_n = odd ? keep : got;
    word[c] = (lo_n | (hi_n << 4)) ^ 0x88888888u;  // offset binary -> two's complement
  }
  // word[c] of lane (g, i) holds, for u = 4 * (2c + odd) + k (k = byte), the
  // output byte at  g * 256 + u * 4 + (i >> 1).  A 4 x 4 byte transpose among
  // the lanes i>>1 = 0..3 turns these into aligned 32-bit words.
  const int r = gi_i >> 1;
  const uint32_t sel1 = (r & 1) ? 0x3715u : 0x6240u;  // step 1 selector (own = a, partner = b)
  const uint32_t sel2 = (r & 2) ? 0x3276u : 0x5410u;  // step 2 selector
  uint32_t* q = reinterpret_cast<uint32_t*>(q_out + m * 2048);
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    uint32_t w = word[c];
    uint32_t p = __shfl_xor_sync(0xffffffffu, w, 2);
    // r even: [own.k0, p.k0, own.k2, p.k2];  r odd: [p.k1, own.k1, p.k3, own.k3]
    w = __byte_perm(w, p, sel1);
    p = __shfl_xor_sync(0xffffffffu, w, 4);
    // r < 2: [own.b0, own.b1, p.b0, p.b1];  r >= 2: [p.b2, p.b3, own.b2, own.b3]
    w = __byte_perm(w, p, sel2);
    const int u = 4 * (2 * c + (odd ? 1 : 0)) + r;
    q[gi_g * 64 + u] = w;
  }
  }  // rows of this group
}

}  // namespace smoothrot
#include "walsh4096_tc.cuh"
namespace smoothrot {

// ---------------------------------------------------------------------------
// K = 14336 = 28 x 512  (index j = a * 512 + b; H = kron(H28, H512)).
// Persistent kernel, one CTA per SM with kP512Groups row groups of 224 threads;
// rows are prefetched by bulk asynchronous copies as in the K = 4096 kernel.
//
//   step 1  a thread takes the two columns b = 2bp, 2bp + 1 and applies the
//           order-28 factor to them: it reads the 28 fp16 pairs (a, b) from
//           the input buffer four rows a at a time, multiplies by `pre`, and
//           accumulates the 28 outputs.  Four inputs meet an output with one
//           of 8 sign patterns (up to a global sign), so the 8 pattern sums
//           are formed once per group of four (12 packed operations) and each
//           output takes one add or subtract per group: about 4.5 packed
//           operations per value instead of 13.5.
//           The result goes to the fp32 row [28][512] in shared memory.
//   step 2  thread (a, j), a < 28, j < 8, takes the eight 32-byte chunks
//           j, j + 8, ... of row a: 64 values covering b bits {0,1,2} and
//           {6,7,8}; six butterfly stages in registers, results back in
//           place; then the same 8 lanes re-read the row as 64 consecutive
//           values each (chunks 8j .. 8j+7) and do the stages on b bits
//           {3,4,5}, again in registers.
//   absmax over the row, step size, rounding; a thread's 64 consecutive codes
//   are eight 32-bit words of output, written as two 16-byte stores.
// 1/sqrt(14336) is folded into the step size and the reciprocal.
// ---------------------------------------------------------------------------
constexpr int kP512Groups = 2;
constexpr int kP512GroupThreads = 224;   // 28 rows a x 8 lanes: step 2 uses every thread
constexpr int kP512Threads = kP512Groups * kP512GroupThreads;
constexpr int kP512K = 28 * 512;
constexpr int kP512PreBytes = kP512K * 4;
constexpr int kP512InBytes = kP512K * 2;
constexpr int kP512RowBytes = kP512K * 4;
constexpr int kP512GroupBytes = kP512InBytes + kP512RowBytes;
constexpr int kP512SmemBytes = kP512PreBytes + kP512Groups * kP512GroupBytes + kP512Groups * 8 + kP512Groups * 4;
static_assert(kP512SmemBytes <= 227 * 1024, "shared memory budget of the K = 14336 kernel");

// For inputs 4g .. 4g+3 and output c: which of the 8 pattern sums, and whether it is added.
// Pattern sums (first input always +):  0 ++++  1 ++--  2 +-+-  3 +--+  4 +++-  5 ++-+  6 +-++  7 +---
struct Paley28Plan {
  unsigned char index[7][28];
  bool add[7][28];
};

__host__ __device__ constexpr Paley28Plan make_paley28_plan() {
  Paley28Plan p{};
  for (int g = 0; g < 7; ++g) {
    for (int c = 0; c < 28; ++c) {
      const int s0 = paley28_entry(4 * g, c), s1 = paley28_entry(4 * g + 1, c);
      const int s2 = paley28_entry(4 * g + 2, c), s3 = paley28_entry(4 * g + 3, c);
      // relative signs with respect to the first input
      const int r1 = s1 * s0, r2 = s2 * s0, r3 = s3 * s0;
      int idx = 0;
      if (r1 > 0 && r2 > 0 && r3 > 0) idx = 0;
      else if (r1 > 0 && r2 < 0 && r3 < 0) idx = 1;
      else if (r1 < 0 && r2 > 0 && r3 < 0) idx = 2;
      else if (r1 < 0 && r2 < 0 && r3 > 0) idx = 3;
      else if (r1 > 0 && r2 > 0 && r3 < 0) idx = 4;
      else if (r1 > 0 && r2 < 0 && r3 > 0) idx = 5;
      else if (r1 < 0 && r2 > 0 && r3 > 0) idx = 6;
      else idx = 7;
      p.index[g][c] = static_cast<unsigned char>(idx);
      p.add[g][c] = s0 > 0;
    }
  }
  return p;
}

// Adds (or subtracts) the pattern sum the plan names for (group G, output C) to acc[C], for C = 0..27.
template <int G, int C>
struct Paley28Accumulate {
  static __device__ __forceinline__ void run(f32x2* acc, const f32x2* sums) {
    constexpr Paley28Plan plan = make_paley28_plan();
    constexpr int idx = plan.index[G][C];
    constexpr bool add = plan.add[G][C];
    if (G == 0) {
      static_assert(G != 0 || add, "the first row of the order-28 matrix is all +1");
      acc[C] = sums[idx];
    } else if (add) {
      acc[C] = add2(acc[C], sums[idx]);
    } else {
      acc[C] = sub2(acc[C], sums[idx]);
    }
    if constexpr (C + 1 < 28) Paley28Accumulate<G, C + 1>::run(acc, sums);
  }
};

// One group of four inputs (rows a = 4G .. 4G+3 of the order-28 factor) of step 1.
// With kGlu the value is SiLU(gate) * up, read from two input buffers kP512InBytes apart, and the
// diagonal comes from global memory (shared memory is taken by the second input buffer).
template <int G, bool kHasPre, bool kGlu>
__device__ __forceinline__ void paley28_group(f32x2* acc, uint32_t in_addr, const float* pre_src, int bp) {
  f32x2 x[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int a = 4 * G + q;
    uint32_t raw;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(raw) : "r"(in_addr + uint32_t(a * 1024 + bp * 4)) : "memory");
    float2 f = __half22float2(*reinterpret_cast<const __half2*>(&raw));
    if (kGlu) {
      uint32_t raw_u;
      asm volatile("ld.shared.b32 %0, [%1];"
                   : "=r"(raw_u) : "r"(in_addr + uint32_t(kP512K * 2 + a * 1024 + bp * 4)) : "memory");
      const float2 u = __half22float2(*reinterpret_cast<const __half2*>(&raw_u));
      f.x = glu_product(f.x, u.x);
      f.y = glu_product(f.y, u.y);
    }
    x[q] = pack2(f.x, f.y);
    if (kHasPre) {
      const float2 p = kGlu ? __ldg(reinterpret_cast<const float2*>(pre_src + a * 512 + bp * 2))
                            : *reinterpret_cast<const float2*>(pre_src + a * 512 + bp * 2);
      x[q] = mul2(x[q], pack2(p.x, p.y));
    }
  }
  const f32x2 p0 = add2(x[0], x[1]), m0 = sub2(x[0], x[1]);
  const f32x2 p1 = add2(x[2], x[3]), m1 = sub2(x[2], x[3]);
  f32x2 sums[8];
  sums[0] = add2(p0, p1);   // + + + +
  sums[1] = sub2(p0, p1);   // + + - -
  sums[2] = add2(m0, m1);   // + - + -
  sums[3] = sub2(m0, m1);   // + - - +
  sums[4] = add2(p0, m1);   // + + + -
  sums[5] = sub2(p0, m1);   // + + - +
  sums[6] = add2(m0, p1);   // + - + +
  sums[7] = sub2(m0, p1);   // + - - -
  Paley28Accumulate<G, 0>::run(acc, sums);
}

// Position of 16-byte unit u (0..127) inside a 2 KB row of the fp32 buffer.  The low three bits
// (the 128-byte bank group) are mixed with bits 3 and 4..6, so that 8 lanes reading units
// 2 apart (step 2a), 16 apart (step 2b) or adjacent (step 1) never meet in a bank.
__device__ __forceinline__ int p512_unit(int u) { return u ^ ((u >> 3) & 1) ^ ((u >> 4) & 7); }

__device__ __forceinline__ void group_barrier224(int group) {
  asm volatile("bar.sync %0, 224;" ::"r"(group + 1) : "memory");
}

// kGlu: the row is SiLU(gate) * up of two fp16 inputs (X = gate rows, U = up rows); the second
// input buffer takes the place of the diagonal's copy in shared memory (same total).
template <bool kQuant, bool kHasPre, bool kLowClamp, bool kGlu>
__global__ void __launch_bounds__(kP512Threads, 1)
paley512_kernel(const __half* __restrict__ X, int64_t ldx, const __half* __restrict__ U, int64_t ldu, int64_t M,
                const float* __restrict__ pre, float clip,
                uint8_t* __restrict__ q_out, float* __restrict__ step_out,
                float* __restrict__ y_out) {
  // shared memory: [pre: 14336 fp32][per group: input row fp16 | transformed row fp32][mbarriers][flags]
  // with kGlu:     [per group: gate row fp16 | up row fp16 | transformed row fp32][mbarriers][flags]
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ float red[kP512Groups][8];   // one slot per warp of a group (7 used)
  constexpr int kPreBytes = kGlu ? 0 : kP512PreBytes;
  constexpr int kInBytes = kGlu ? 2 * kP512InBytes : kP512InBytes;
  constexpr int kGroupBytes = kInBytes + kP512RowBytes;
  static_assert(kPreBytes + kP512Groups * kGroupBytes == kP512PreBytes + kP512Groups * kP512GroupBytes,
                "both layouts fill the same shared memory");
  const int group = threadIdx.x >= kP512GroupThreads ? 1 : 0;
  const int t = threadIdx.x - group * kP512GroupThreads;
  const int lane = threadIdx.x & 31;
  const float* spre = kGlu ? pre : reinterpret_cast<const float*>(smem_raw);   // where step 1 reads the diagonal
  uint8_t* gbase = smem_raw + kPreBytes + group * kGroupBytes;
  const uint32_t inbuf = smem_addr(gbase);
  float* row = reinterpret_cast<float*>(gbase + kInBytes);
  const uint32_t bar = smem_addr(smem_raw + kP512PreBytes + kP512Groups * kP512GroupBytes + group * 8);
  volatile int* lost = reinterpret_cast<volatile int*>(smem_raw + kP512PreBytes + kP512Groups * kP512GroupBytes +
                                                       kP512Groups * 8) + group;

  if (kHasPre && !kGlu) {
    for (int i = threadIdx.x; i < kP512K / 4; i += kP512Threads)
      reinterpret_cast<float4*>(smem_raw)[i] = __ldg(reinterpret_cast<const float4*>(pre) + i);
  }
  if (t == 0) {
    *lost = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // one row (or the gate and up rows) into the group's input buffer, completion on `bar`
  auto fetch_row = [&](int64_t r) {
    if (kGlu) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                   ::"r"(bar), "r"(uint32_t(2 * kP512InBytes)) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(inbuf), "l"(X + r * ldx), "r"(uint32_t(kP512InBytes)), "r"(bar) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(inbuf + uint32_t(kP512InBytes)), "l"(U + r * ldu), "r"(uint32_t(kP512InBytes)), "r"(bar)
                   : "memory");
    } else {
      start_row_copy(inbuf, X + r * ldx, kP512InBytes, bar);
    }
  };

  const int64_t stride = int64_t(gridDim.x) * kP512Groups;
  int64_t m = int64_t(blockIdx.x) + int64_t(gridDim.x) * group;
  if (t == 0 && m < M) fetch_row(m);
  uint32_t parity = 0;

  // step 2 ownership: row a of the order-28 factor, lane group j
  const int a2 = t >> 3, j2 = t & 7;

  for (; m < M; m += stride) {
    if (!wait_row_copy(bar, parity)) *lost = 1;
    parity ^= 1u;

    // ---- step 1: order-28 factor on a pair of columns; 256 pairs for 224 threads, so the
    //      first warp of the group takes a second pair
    for (int bp = t; bp < 256; bp += kP512GroupThreads) {
      f32x2 acc[28];
      paley28_group<0, kHasPre, kGlu>(acc, inbuf, spre, bp);
      paley28_group<1, kHasPre, kGlu>(acc, inbuf, spre, bp);
      paley28_group<2, kHasPre, kGlu>(acc, inbuf, spre, bp);
      paley28_group<3, kHasPre, kGlu>(acc, inbuf, spre, bp);
      paley28_group<4, kHasPre, kGlu>(acc, inbuf, spre, bp);
      paley28_group<5, kHasPre, kGlu>(acc, inbuf, spre, bp);
      paley28_group<6, kHasPre, kGlu>(acc, inbuf, spre, bp);
      // fp32 row [28][512], its 16-byte units permuted by p512_unit
      const int phys = p512_unit(bp >> 1);
#pragma unroll
      for (int c = 0; c < 28; ++c) {
        float lo, hi;
        unpack2(acc[c], lo, hi);
        *reinterpret_cast<float2*>(row + c * 512 + phys * 4 + (bp & 1) * 2) = make_float2(lo, hi);
      }
    }
    group_barrier224(group);   // input consumed, transformed row complete
    if (*lost != 0) break;
    if (t == 0 && m + stride < M) fetch_row(m + stride);

    // ---- step 2: Walsh-512 along b ------------------------------------------------------------
    f32x2 v[32];
    {
      float* arow = row + a2 * 512;
      // 2a: chunks j, j + 8, ..: b bits 0,1,2 (inside a chunk) and 6,7,8 (k), in place
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int chunk = j2 + 8 * k;
        const float4 lo4 = *reinterpret_cast<const float4*>(arow + p512_unit(2 * chunk) * 4);
        const float4 hi4 = *reinterpret_cast<const float4*>(arow + p512_unit(2 * chunk + 1) * 4);
        v[4 * k] = pack2(lo4.x, lo4.y);
        v[4 * k + 1] = pack2(lo4.z, lo4.w);
        v[4 * k + 2] = pack2(hi4.x, hi4.y);
        v[4 * k + 3] = pack2(hi4.z, hi4.w);
      }
      butterflies_pairs<32>(v);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int chunk = j2 + 8 * k;
        float4 lo4, hi4;
        unpack2(v[4 * k], lo4.x, lo4.y);
        unpack2(v[4 * k + 1], lo4.z, lo4.w);
        unpack2(v[4 * k + 2], hi4.x, hi4.y);
        unpack2(v[4 * k + 3], hi4.z, hi4.w);
        *reinterpret_cast<float4*>(arow + p512_unit(2 * chunk) * 4) = lo4;
        *reinterpret_cast<float4*>(arow + p512_unit(2 * chunk + 1) * 4) = hi4;
      }
    }
    __syncwarp();   // the 8 lanes that share row a sit in one warp
    {
      const float* arow = row + a2 * 512;
      // 2b: the 8 consecutive chunks 8 j .. 8 j + 7 (64 consecutive b): b bits 3,4,5
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int chunk = 8 * j2 + c;
        const float4 lo4 = *reinterpret_cast<const float4*>(arow + p512_unit(2 * chunk) * 4);
        const float4 hi4 = *reinterpret_cast<const float4*>(arow + p512_unit(2 * chunk + 1) * 4);
        v[4 * c] = pack2(lo4.x, lo4.y);
        v[4 * c + 1] = pack2(lo4.z, lo4.w);
        v[4 * c + 2] = pack2(hi4.x, hi4.y);
        v[4 * c + 3] = pack2(hi4.z, hi4.w);
      }
#pragma unroll
      for (int h = 4; h < 32; h <<= 1) {   // pair index = 4 * c + p: the bits of c
#pragma unroll
        for (int u = 0; u < 32; ++u) {
          if ((u & h) == 0) {
            const f32x2 x0 = v[u], x1 = v[u + h];
            v[u] = add2(x0, x1);
            v[u + h] = sub2(x0, x1);
          }
        }
      }
    }

    const float isk = 0.00835191381f;   // 1 / sqrt(14336), rounded to fp32
    if (!kQuant) {
      {
        float* y = y_out + m * kP512K + a2 * 512;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          float4 o0, o1;
          unpack2(v[4 * k], o0.x, o0.y);
          unpack2(v[4 * k + 1], o0.z, o0.w);
          unpack2(v[4 * k + 2], o1.x, o1.y);
          unpack2(v[4 * k + 3], o1.z, o1.w);
          o0.x *= isk; o0.y *= isk; o0.z *= isk; o0.w *= isk;
          o1.x *= isk; o1.y *= isk; o1.z *= isk; o1.w *= isk;
          float4* dst = reinterpret_cast<float4*>(y + (8 * j2 + k) * 8);
          dst[0] = o0;
          dst[1] = o1;
        }
      }
      group_barrier224(group);   // the row buffer is rewritten by the next row's step 1
      continue;
    }

    float amax = 0.0f;
    {
#pragma unroll
      for (int u = 0; u < 32; ++u) {
        float lo, hi;
        unpack2(v[u], lo, hi);
        amax = fmaxf(amax, fmaxf(fabsf(lo), fabsf(hi)));
      }
    }
    amax = warp_max(amax);
    if (lane == 0) red[group][t >> 5] = amax;
    group_barrier224(group);
    amax = red[group][0];
#pragma unroll
    for (int w = 1; w < 7; ++w) amax = fmaxf(amax, red[group][w]);
    amax = __fmul_rn(amax, isk);                       // absmax of the normalised row
    const float step = step_from_absmax(amax, clip);
    if (t == 0) step_out[m] = step;
    const float inv = __fmul_rn(__frcp_rn(step), isk);  // 1/step for the unnormalised values
    const f32x2 inv2 = pack2(inv, inv);
    const float kMagic = 12582912.0f + 8.0f;            // 1.5 * 2^23 + 8: low byte = code + 8
    const f32x2 magic2 = pack2(kMagic, kMagic);
    uint32_t* q = reinterpret_cast<uint32_t*>(q_out + m * (kP512K / 2)) + a2 * 64;
    uint32_t words[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      uint32_t r[8];
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        float q0, q1;
        unpack2(fma2(v[4 * k + p], inv2, magic2), q0, q1);
        if (kLowClamp) {
          q0 = fmaxf(fminf(q0, 12582912.0f + 15.0f), 12582912.0f);
          q1 = fmaxf(fminf(q1, 12582912.0f + 15.0f), 12582912.0f);
        }
        r[2 * p] = __float_as_uint(q0);
        r[2 * p + 1] = __float_as_uint(q1);
      }
      uint32_t lo4 = __byte_perm(__byte_perm(r[0], r[1], 0x0040), __byte_perm(r[2], r[3], 0x0040), 0x5410);
      uint32_t hi4 = __byte_perm(__byte_perm(r[4], r[5], 0x0040), __byte_perm(r[6], r[7], 0x0040), 0x5410);
      if (!kLowClamp) {   // bytes are code + 8 in [0, 16]: 16 comes down to 15
        lo4 -= (lo4 >> 4) & 0x01010101u;
        hi4 -= (hi4 >> 4) & 0x01010101u;
      }
      lo4 |= lo4 >> 4;    // bytes 0 and 2 now hold two codes each
      hi4 |= hi4 >> 4;
      const uint32_t word = __byte_perm(lo4, hi4, 0x6420) ^ 0x88888888u;   // offset binary -> two's complement
      words[k] = word;
    }
    uint4* dst = reinterpret_cast<uint4*>(q + 8 * j2);
    dst[0] = make_uint4(words[0], words[1], words[2], words[3]);
    dst[1] = make_uint4(words[4], words[5], words[6], words[7]);
  }  // rows of this group
}

}  // namespace smoothrot
#include "paley512_tc.cuh"
namespace smoothrot {

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
static int check_rows(const void* X, int64_t rows, int64_t K, int64_t ld, int* base, int* n, int* logn) {
  if (rows < 0 || K <= 0) return SMOOTHROT_INVALID_ARG;
  if (!split_order(K, base, n, logn)) return SMOOTHROT_UNSUPPORTED_K;
  if (rows == 0) return SMOOTHROT_OK;
  if (X == nullptr || ld < K) return SMOOTHROT_INVALID_ARG;
  if (!aligned16(X) || (ld % 8) != 0) return SMOOTHROT_BAD_ALIGNMENT;
  if (rows > 0x7fffffffLL) return SMOOTHROT_INVALID_ARG;
  return SMOOTHROT_OK;
}

// U != nullptr: X holds gate rows, U up rows, and the transformed row is SiLU(gate) * up.
template <bool kQuant>
static int launch_rotate(const void* X, int64_t rows, int64_t K, int64_t ld, const void* U, int64_t ldu,
                         const float* pre, float clip, uint8_t* q_out, float* step_out, float* y_out,
                         cudaStream_t stream) {
  int base = 0, n = 0, logn = 0;
  int rc = check_rows(X, rows, K, ld, &base, &n, &logn);
  if (rc != SMOOTHROT_OK || rows == 0) return rc;
  const bool glu = U != nullptr;
  if (glu) {
    int b2 = 0, n2 = 0, l2 = 0;
    rc = check_rows(U, rows, K, ldu, &b2, &n2, &l2);
    if (rc != SMOOTHROT_OK) return rc;
  }
  const __half* x = static_cast<const __half*>(X);
  const __half* u = static_cast<const __half*>(U);
  if (K == 4096 && !glu && pre == nullptr && rows >= 512) {
    // No diagonal: the order-128 factor of the rotation on the tensor cores (walsh4096_tc.cuh).
    // A few hundred rows or fewer finish sooner in the register kernel below (shorter set-up).
    const bool low = kQuant && (7.0f / clip >= 8.49f);
    // the rows as a [rows][32 groups][2 halves][64 values] tensor; a box = one K half of a batch's rows
    CUtensorMap xmap;
    TensorMapEncodeFn encode = tensor_map_encoder();
    if (encode == nullptr) return SMOOTHROT_CUDA_ERROR;
    const cuuint64_t dims[4] = {64, 2, 32, cuuint64_t(rows)};
    const cuuint64_t strides[3] = {128, 256, cuuint64_t(ld) * sizeof(__half)};
    const int sms = device_sm_count();
    // batches of six rows for long inputs, of four (finer granularity, shorter tail) otherwise
    const bool six = rows >= int64_t(48) * sms;
    const int tokens = six ? 6 : 4;
    const cuuint32_t box[4] = {64, 1, 32, cuuint32_t(tokens)};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<__half*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SMOOTHROT_CUDA_ERROR;
    const int64_t batches = (rows + tokens - 1) / tokens;
    const unsigned grid = unsigned(batches < sms ? batches : sms);
    if (six) {
      auto kern = low ? wtc::walsh4096_tc_kernel<kQuant, true, 6> : wtc::walsh4096_tc_kernel<kQuant, false, 6>;
      if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), wtc::Cfg<6>::kSmemBytes))
        return SMOOTHROT_CUDA_ERROR;
      kern<<<grid, wtc::Cfg<6>::kThreads, wtc::Cfg<6>::kSmemBytes, stream>>>(xmap, rows, clip, q_out, step_out, y_out);
    } else {
      auto kern = low ? wtc::walsh4096_tc_kernel<kQuant, true, 4> : wtc::walsh4096_tc_kernel<kQuant, false, 4>;
      if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), wtc::Cfg<4>::kSmemBytes))
        return SMOOTHROT_CUDA_ERROR;
      kern<<<grid, wtc::Cfg<4>::kThreads, wtc::Cfg<4>::kSmemBytes, stream>>>(xmap, rows, clip, q_out, step_out, y_out);
    }
    count_launch();
    return launch_status();
  }
  if (K == 4096 && !glu) {
    // codes below -8 can only come up when the row maximum sits at 8.5 steps or more
    const bool low = kQuant && (7.0f / clip >= 8.49f);
    auto kern = pre ? (low ? walsh4096_kernel<kQuant, true, true> : walsh4096_kernel<kQuant, true, false>)
                    : (low ? walsh4096_kernel<kQuant, false, true> : walsh4096_kernel<kQuant, false, false>);
    if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), kW4096SmemBytes))
      return SMOOTHROT_CUDA_ERROR;
    const int sms = device_sm_count();
    const unsigned grid = unsigned(rows < sms ? rows : sms);
    kern<<<grid, kW4096Threads, kW4096SmemBytes, stream>>>(x, ld, rows, pre, clip, q_out, step_out, y_out);
    count_launch();
    return launch_status();
  }
  if (K == kP512K && !glu && pre == nullptr && rows >= 256) {
    // No diagonal: the Walsh part of the rotation on the tensor cores (paley512_tc.cuh).
    const bool low = kQuant && (7.0f / clip >= 8.49f);
    // the rows as a [rows][28][8 blocks of 64][64 values] tensor; a box = one block of 64 values of the 28 rows a
    CUtensorMap xmap;
    TensorMapEncodeFn encode = tensor_map_encoder();
    if (encode == nullptr) return SMOOTHROT_CUDA_ERROR;
    const cuuint64_t dims[4] = {64, 8, 28, cuuint64_t(rows)};
    const cuuint64_t strides[3] = {128, 1024, cuuint64_t(ld) * sizeof(__half)};
    const cuuint32_t box[4] = {64, 1, 28, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<__half*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SMOOTHROT_CUDA_ERROR;
    auto kern = low ? ptc::paley512_tc_kernel<kQuant, true> : ptc::paley512_tc_kernel<kQuant, false>;
    if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), ptc::kSmemBytes))
      return SMOOTHROT_CUDA_ERROR;
    const int64_t batches = (rows + ptc::kTokens - 1) / ptc::kTokens;
    const int sms = device_sm_count();
    const unsigned grid = unsigned(batches < sms ? batches : sms);
    kern<<<grid, ptc::kThreads, ptc::kSmemBytes, stream>>>(xmap, rows, clip, q_out, step_out, y_out);
    count_launch();
    return launch_status();
  }
  if (K == kP512K) {
    const bool low = kQuant && (7.0f / clip >= 8.49f);
    auto pick = [&](auto glu_tag) {
      constexpr bool kG = decltype(glu_tag)::value;
      return pre ? (low ? paley512_kernel<kQuant, true, true, kG> : paley512_kernel<kQuant, true, false, kG>)
                 : (low ? paley512_kernel<kQuant, false, true, kG> : paley512_kernel<kQuant, false, false, kG>);
    };
    auto kern = glu ? pick(std::true_type{}) : pick(std::false_type{});
    if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), kP512SmemBytes))
      return SMOOTHROT_CUDA_ERROR;
    const int sms = device_sm_count();
    const unsigned grid = unsigned(rows < sms ? rows : sms);
    kern<<<grid, kP512Threads, kP512SmemBytes, stream>>>(x, ld, u, ldu, rows, pre, clip, q_out, step_out, y_out);
    count_launch();
    return launch_status();
  }
  const size_t smem = size_t(K) * sizeof(float);
  auto kern = glu ? rotate_generic_kernel<kQuant, true> : rotate_generic_kernel<kQuant, false>;
  if (!allow_dynamic_smem(reinterpret_cast<const void*>(kern), int(smem)))
    return SMOOTHROT_CUDA_ERROR;
  const float inv_sqrt_k = float(1.0 / sqrt(double(K)));
  kern<<<unsigned(rows), kGenericThreads, smem, stream>>>(x, ld, u, ldu, int(K), base, n, logn, pre, inv_sqrt_k, clip,
                                                           q_out, step_out, y_out);
  count_launch();
  return launch_status();
}

static int quantize_entry(const void* X, int64_t rows, int64_t K, int64_t ld, const void* U, int64_t ldu,
                          const float* pre, float clip, uint8_t* q_out, float* step_out, void* stream) {
  if (!(clip > 0.0f) || clip > 1.0f) return SMOOTHROT_INVALID_ARG;
  if (rows > 0 && (q_out == nullptr || step_out == nullptr)) return SMOOTHROT_INVALID_ARG;
  if (rows > 0 && (!aligned16(q_out) || (pre != nullptr && !aligned16(pre)))) return SMOOTHROT_BAD_ALIGNMENT;
  return launch_rotate<true>(X, rows, K, ld, U, ldu, pre, clip, q_out, step_out, nullptr,
                             static_cast<cudaStream_t>(stream));
}

}  // namespace smoothrot

extern "C" {

int smoothrot_fuse_weights(const void* W_f16, int64_t N, int64_t K, int64_t ldw, const float* pre,
                           float clip_w, uint8_t* Wq_out, float* dw_out, void* stream) {
  return smoothrot::quantize_entry(W_f16, N, K, ldw, nullptr, 0, pre, clip_w, Wq_out, dw_out, stream);
}

int smoothrot_quant_act(const void* X_f16, int64_t M, int64_t K, int64_t ldx, const float* pre,
                        float clip_a, uint8_t* Xq_out, float* dx_out, void* stream) {
  return smoothrot::quantize_entry(X_f16, M, K, ldx, nullptr, 0, pre, clip_a, Xq_out, dx_out, stream);
}

int smoothrot_quant_act_glu(const void* gate_f16, const void* up_f16, int64_t M, int64_t K, int64_t ld_gate,
                            int64_t ld_up, const float* pre, float clip_a, uint8_t* Xq_out, float* dx_out,
                            void* stream) {
  if (M > 0 && up_f16 == nullptr) return SMOOTHROT_INVALID_ARG;
  return smoothrot::quantize_entry(gate_f16, M, K, ld_gate, up_f16, ld_up, pre, clip_a, Xq_out, dx_out, stream);
}

int smoothrot_debug_hadamard(const void* X_f16, int64_t M, int64_t K, int64_t ldx, const float* pre,
                             float* Y_f32, void* stream) {
  if (M > 0 && Y_f32 == nullptr) return SMOOTHROT_INVALID_ARG;
  if (M > 0 && pre != nullptr && !smoothrot::aligned16(pre)) return SMOOTHROT_BAD_ALIGNMENT;
  return smoothrot::launch_rotate<false>(X_f16, M, K, ldx, nullptr, 0, pre, 1.0f, nullptr, nullptr, Y_f32,
                                         static_cast<cudaStream_t>(stream));
}

// Host. Timeout word of the row transform kernels on the current device (0 = none).
int smoothrot_rotate_status_word(int* value, int clear) {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, smoothrot::g_rotate_status, sizeof(int)) != cudaSuccess) return SMOOTHROT_CUDA_ERROR;
  *value = v;
  if (clear && v != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(smoothrot::g_rotate_status, &zero, sizeof(int)) != cudaSuccess) return SMOOTHROT_CUDA_ERROR;
  }
  return SMOOTHROT_OK;
}

// Host. Limit of the bounded waits of the row transform kernels on the current device
// (0 restores the default of two seconds).
int smoothrot_rotate_set_wait_limit_ns(uint64_t ns) {
  const unsigned long long v = ns == 0 ? smoothrot::kLoadWaitLimitNs : static_cast<unsigned long long>(ns);
  if (cudaMemcpyToSymbol(smoothrot::g_rotate_wait_limit_ns, &v, sizeof(v)) != cudaSuccess) return SMOOTHROT_CUDA_ERROR;
  return SMOOTHROT_OK;
}

int smoothrot_base_matrix(int order, int8_t* out_host) {
  if (out_host == nullptr || (order != 12 && order != 20 && order != 28)) return SMOOTHROT_INVALID_ARG;
  for (int r = 0; r < order; ++r)
    for (int c = 0; c < order; ++c)
      out_host[r * order + c] = int8_t(order == 28 ? smoothrot::paley28_entry(r, c)
                                                   : smoothrot::paley_prime_entry(order - 1, r, c));
  return SMOOTHROT_OK;
}

int smoothrot_paley28(int8_t* out_host) {
  if (out_host == nullptr) return SMOOTHROT_INVALID_ARG;
  for (int r = 0; r < 28; ++r)
    for (int c = 0; c < 28; ++c) out_host[r * 28 + c] = int8_t(smoothrot::paley28_entry(r, c));
  return SMOOTHROT_OK;
}

}  // extern "C"
