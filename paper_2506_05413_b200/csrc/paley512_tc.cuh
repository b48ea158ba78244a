// K = 14336 = 28 x 512 without a diagonal (the exact online Hadamard in front of the
// down-projection, Lambda^-1 absorbed by the up-projection): the Walsh part on the tensor cores.
// Included by rotate_quant.cu after the order-28 machinery and walsh4096_tc.cuh.
//
// Position j = 512 a + 256 r + 128 c + k  (a < 28, r, c in {0, 1}, k < 128) and
// H14336 = H28 (x) H2 (x) H2 (x) H128.  The factor H2(r) (x) H128(k) is a dense +-1 product of
// order 256 that takes the raw fp16 values as exact operands:
//
//     D_r[i][n] = sum_{r', k} H2[r][r'] H128[i][k] x[token][512 a + 256 r' + 128 c + k],   n = (c, token, a),
//
// two accumulators (r = 0, 1) of N = 128 columns per batch of two tokens (32 column slots per
// (c, token), 28 of them used), each the sum of sixteen tcgen05.mma (kind::f16, M = 128, K = 16)
// over four K blocks (r', half of k); the A operand is H128 or -H128, both kept in shared memory.
// TMA brings, per K block, the 28 rows (one per a) of each (c, token) into the K-major,
// 128-byte-swizzled form the tensor core reads.  Lane i of tensor memory then holds output
// (r, i) of every (a, c): the thread that reads its lane's columns of one token owns 28 x 2
// values, applies H2 over c and the order-28 factor over a in registers (the pattern-sum scheme of
// the register kernel), and the row is complete.  Row maximum over the 256 threads of a token,
// step, rounding, and packing through warp shuffles as in walsh4096_tc.cuh.
//
// Roles (640 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 4..19 epilogue: one warp per
// (token of the batch, r, tensor-memory lane quarter).
#pragma once

namespace smoothrot {
namespace ptc {

constexpr int kTokens = 2;
constexpr int kCols = 64 * kTokens;                   // columns per accumulator: (c, token, 32 slots)
constexpr int kBlockBytes = kCols * 128;              // one K block (64 values) of a batch: 16 KB
constexpr int kStageBytes = 4 * kBlockBytes;          // four K blocks: 64 KB
constexpr int kStages = 2;
constexpr int kABytes = 2 * 128 * 128 * 2;            // H128 and -H128, two K halves of 16 KB each
constexpr int kEpiWarps = 8 * kTokens;
constexpr int kThreads = 32 * (4 + kEpiWarps);
constexpr int kBarOffset = kABytes + kStages * kStageBytes;
constexpr int kNumBarriers = 2 * kStages + 4;         // full, empty per stage; acc_full[2], acc_empty[2]
constexpr int kMiscOffset = kBarOffset + 8 * kNumBarriers;
constexpr int kSmemBytes = 1024 /*alignment slack*/ + kMiscOffset + 16 + kTokens * 2 * 8 * 4;
constexpr uint32_t kIdesc = (1u << 4) | (uint32_t(kCols >> 3) << 17) | (uint32_t(128 >> 4) << 24);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of the K = 14336 tensor-core kernel");

enum Site { kSiteProducer = 21, kSiteMmaFull = 22, kSiteMmaAcc = 23, kSiteEpilogue = 24 };

// One K block q (q = 4 r' + 2 c + half) of one token: box 64 x 1 x 28 x 1 of the
// [rows][28 a][8 q][64 values] view, 28 rows of 128 bytes.
__device__ __forceinline__ void load_rows(uint32_t dst, const CUtensorMap* map, uint32_t bar, int q, int row) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(q), "r"(0), "r"(row)
      : "memory");
}

// One group of four inputs (rows a = 4G .. 4G+3) of the order-28 factor, on packed pairs held in
// registers: acc[c] (+)= sum over the four of x[a] H28[a][c].
template <int G>
__device__ __forceinline__ void paley28_registers_group(f32x2* acc, const f32x2* x) {
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

__device__ __forceinline__ void tmem_load8(uint32_t taddr, float* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
               : "r"(taddr) : "memory");
}

// Eight columns a = 8 H .. 8 H + 7 of both accumulator halves (c = 0, 1) of one token: H2 over c,
// then their share of the order-28 factor.
template <int H>
__device__ __forceinline__ void paley28_from_tmem(f32x2* acc, uint32_t taddr) {
  float x0[8], x1[8];
  tmem_load8(taddr + uint32_t(8 * H), x0);
  tmem_load8(taddr + uint32_t(kTokens * 32 + 8 * H), x1);
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  f32x2 in[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) in[k] = pack2(x0[k] + x1[k], x0[k] - x1[k]);
  paley28_registers_group<2 * H>(acc, in);
  if constexpr (H < 3) paley28_registers_group<2 * H + 1>(acc, in + 4);
}

template <bool kQuant, bool kLowClamp>
__global__ void __launch_bounds__(kThreads, 1)
paley512_tc_kernel(const __grid_constant__ CUtensorMap xmap, int64_t M, float clip,
                   uint8_t* __restrict__ q_out, float* __restrict__ step_out, float* __restrict__ y_out) {
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t dyn = smem_addr(smem_dyn);
  const uint32_t base = (dyn + 1023u) & ~1023u;
  uint8_t* smem = smem_dyn + (base - dyn);
  const uint32_t a_base = base;                  // H128: K half h at + 16 KB h; -H128 at + 32 KB
  const uint32_t b_base = base + kABytes;        // stage s at + 64 KB s; K block (r', h) at + 16 KB (2 r' + h)
  const uint32_t bar_base = base + kBarOffset;
  auto full = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
  auto acc_empty = [&](int s) { return bar_base + 8u * (2 * kStages + 2 + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kMiscOffset);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile float* red = reinterpret_cast<volatile float*>(smem + kMiscOffset + 16);   // [token slot][parity][8]

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t batches = (M + kTokens - 1) / kTokens;

  // one batch: for every K block (r', half) and (c, token) the 28 rows a, into 32-row slots
  auto issue_batch = [&](int s, int64_t b) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 ::"r"(full(s)), "r"(uint32_t(16 * 28 * 128)) : "memory");
    const uint32_t dst = b_base + uint32_t(s) * kStageBytes;
#pragma unroll
    for (int kb = 0; kb < 4; ++kb)        // kb = 2 r' + half
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int tk = 0; tk < kTokens; ++tk)
          load_rows(dst + uint32_t(kb * kBlockBytes + (c * kTokens + tk) * 32 * 128), &xmap, full(s),
                    4 * (kb >> 1) + 2 * c + (kb & 1), int(b * kTokens + tk));
  };

  // The first batch's copy goes out before anything else (it needs one barrier only and has the
  // longest latency of the set-up); the second stage is requested after the set-up barrier.
  uint32_t produced = 0;
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&xmap) : "memory");
    wtc::mbar_init(full(0), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (int64_t(blockIdx.x) < batches) {
      issue_batch(0, int64_t(blockIdx.x));
      produced = 1;
    }
    for (int s = 0; s < kStages; ++s) {
      if (s > 0) wtc::mbar_init(full(s), 1);
      wtc::mbar_init(empty(s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      wtc::mbar_init(acc_full(s), 1);
      wtc::mbar_init(acc_empty(s), kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // H128 and -H128 in the operand's form: row i = 128 bytes per K half, 16-byte unit u at u ^ (i & 7).
  // The slots 28..31 of every (c, token) are never written by TMA: zero them once (their columns
  // of the accumulators are never read, but the tensor core multiplies whatever lies there).
  for (int idx = threadIdx.x; idx < 128 * 16; idx += kThreads) {
    const int i = idx >> 4, unit = idx & 15;
    uint32_t w[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int k = unit * 8 + 2 * p;
      const uint32_t lo = (__popc(i & k) & 1) ? 0xBC00u : 0x3C00u;
      const uint32_t hi = (__popc(i & (k + 1)) & 1) ? 0xBC00u : 0x3C00u;
      w[p] = lo | (hi << 16);
    }
    const uint32_t dst = a_base + uint32_t((unit >> 3) * 16384 + i * 128 + (((unit & 7) ^ (i & 7)) << 4));
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3])
                 : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(dst + 32768u), "r"(w[0] ^ 0x80008000u), "r"(w[1] ^ 0x80008000u), "r"(w[2] ^ 0x80008000u),
                   "r"(w[3] ^ 0x80008000u) : "memory");
  }
  for (int idx = threadIdx.x; idx < kStages * 4 * 2 * kTokens * 4 * 8; idx += kThreads) {
    // (stage, K block, (c, token), pad row 28..31, 16-byte unit)
    const int unit = idx & 7, row = 28 + ((idx >> 3) & 3), slot = (idx >> 5) % (2 * kTokens);
    const int kb = (idx >> 5) / (2 * kTokens) % 4, s = (idx >> 5) / (2 * kTokens) / 4;
    const uint32_t dst = b_base + uint32_t(s * kStageBytes + kb * kBlockBytes + (slot * 32 + row) * 128 + unit * 16);
    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_addr(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = produced;
      for (int64_t b = int64_t(blockIdx.x) + int64_t(produced) * gridDim.x; b < batches; b += gridDim.x, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (it / kStages) & 1u;
        if (!wtc::mbar_wait(empty(s), ph ^ 1u, abort_flag, kSiteProducer)) break;
        issue_batch(s, b);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0;
      for (int64_t b = blockIdx.x; b < batches; b += gridDim.x, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (it / kStages) & 1u;
        const int ab = it & 1;
        const uint32_t aph = (it >> 1) & 1u;
        if (!wtc::mbar_wait(acc_empty(ab), aph ^ 1u, abort_flag, kSiteMmaAcc)) break;
        if (!wtc::mbar_wait(full(s), ph, abort_flag, kSiteMmaFull)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t b_addr = b_base + uint32_t(s) * kStageBytes;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const uint32_t tmem_d = tmem_base + uint32_t(ab * 256 + r * kCols);
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {       // kb = 2 r' + half
            const bool neg = (r == 1) && (kb >= 2);                 // H2[r][r'] = -1
            const uint32_t a_addr = a_base + uint32_t((neg ? 32768 : 0) + (kb & 1) * 16384);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t da = wtc::desc_sw128(a_addr) + uint64_t(2 * ks);
              const uint64_t db = wtc::desc_sw128(b_addr + uint32_t(kb * kBlockBytes)) + uint64_t(2 * ks);
              wtc::mma_f16(tmem_d, da, db, kIdesc, (kb > 0 || ks > 0) ? 1u : 0u);
            }
          }
        }
        wtc::commit(empty(s));
        wtc::commit(acc_full(ab));
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;                 // tensor-memory lanes 32 quarter .. + 31
    const int r = ((warp - 4) >> 2) & 1;          // which accumulator (output bit 8 of the position inside a row of 512)
    const int tk = (warp - 4) >> 3;               // token of the batch
    const int i = quarter * 32 + lane;            // output index k of the order-128 factor
    const bool odd = (i & 1) != 0;
    const int r4 = (i >> 1) & 3;
    const uint32_t sel1 = (r4 & 1) ? 0x3715u : 0x6240u;
    const uint32_t sel2 = (r4 & 2) ? 0x3276u : 0x5410u;
    const float isk = 0.00835191381f;             // 1 / sqrt(14336), rounded to fp32
    uint32_t it = 0;
    for (int64_t b = blockIdx.x; b < batches; b += gridDim.x, ++it) {
      const int ab = it & 1;
      const uint32_t aph = (it >> 1) & 1u;
      if (!wtc::mbar_wait(acc_full(ab), aph, abort_flag, kSiteEpilogue)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int64_t m = b * kTokens + tk;
      if (m < M) {
        // columns (c, token, a): c = 0 at taddr, c = 1 64 columns further; a < 28 used.
        // H2 over c, then the order-28 factor over a, on pairs (c' = 0, c' = 1); eight a at a time
        const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(ab * 256 + r * kCols + tk * 32);
        f32x2 v[28];
        paley28_from_tmem<0>(v, taddr);
        paley28_from_tmem<1>(v, taddr);
        paley28_from_tmem<2>(v, taddr);
        paley28_from_tmem<3>(v, taddr);
        // v[a] = values at positions 512 a + 256 r + 128 c' + i  for c' = 0, 1

        if (!kQuant) {
          float* y = y_out + m * 14336 + r * 256 + i;
#pragma unroll
          for (int a = 0; a < 28; ++a) {
            float lo, hi;
            unpack2(v[a], lo, hi);
            y[a * 512] = lo * isk;
            y[a * 512 + 128] = hi * isk;
          }
        } else {
          float am[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
          for (int a = 0; a < 28; ++a) {
            float lo, hi;
            unpack2(v[a], lo, hi);
            am[a & 3] = fmaxf(fmaxf(am[a & 3], fabsf(lo)), fabsf(hi));
          }
          float amax = warp_max(fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])));
          volatile float* mine = red + (tk * 2 + (it & 1)) * 8;
          if (lane == 0) mine[r * 4 + quarter] = amax;
          asm volatile("bar.sync %0, 256;" ::"r"(1 + tk) : "memory");
          amax = fmaxf(fmaxf(fmaxf(mine[0], mine[1]), fmaxf(mine[2], mine[3])),
                       fmaxf(fmaxf(mine[4], mine[5]), fmaxf(mine[6], mine[7])));
          amax = __fmul_rn(amax, isk);                        // absmax of the normalised row
          const float step = step_from_absmax(amax, clip);
          if (i == 0 && r == 0) step_out[m] = step;
          const float inv = __fmul_rn(__frcp_rn(step), isk);  // 1/step for the unnormalised values
          const f32x2 inv2 = pack2(inv, inv);
          const float kMagic = 12582912.0f + 8.0f;            // 1.5 * 2^23 + 8: low byte = code + 8
          const f32x2 magic2 = pack2(kMagic, kMagic);
          // spread word w: four codes, one per byte: a = 4 (w >> 1) + byte, c' = w & 1
          uint32_t spread[14];
#pragma unroll
          for (int g = 0; g < 7; ++g) {
            uint32_t lo4[4], hi4[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              float q0, q1;
              unpack2(fma2(v[4 * g + k], inv2, magic2), q0, q1);
              if (kLowClamp) {
                q0 = fmaxf(fminf(q0, 12582912.0f + 15.0f), 12582912.0f);
                q1 = fmaxf(fminf(q1, 12582912.0f + 15.0f), 12582912.0f);
              }
              lo4[k] = __float_as_uint(q0);
              hi4[k] = __float_as_uint(q1);
            }
            uint32_t f0 = __byte_perm(__byte_perm(lo4[0], lo4[1], 0x0040), __byte_perm(lo4[2], lo4[3], 0x0040), 0x5410);
            uint32_t f1 = __byte_perm(__byte_perm(hi4[0], hi4[1], 0x0040), __byte_perm(hi4[2], hi4[3], 0x0040), 0x5410);
            if (!kLowClamp) {   // the code +8 comes down to +7
              f0 -= (f0 >> 4) & 0x01010101u;
              f1 -= (f1 >> 4) & 0x01010101u;
            }
            spread[2 * g] = f0;
            spread[2 * g + 1] = f1;
          }
          // Lanes 2p and 2p + 1 hold the even and the odd position of each output byte: the even lane
          // finishes the spread words with c' = 0, the odd lane those with c' = 1.
          uint32_t* q = reinterpret_cast<uint32_t*>(q_out + m * 7168) + r * 32 + (odd ? 16 : 0) + (i >> 3);
#pragma unroll
          for (int g = 0; g < 7; ++g) {
            const uint32_t give = odd ? spread[2 * g] : spread[2 * g + 1];
            const uint32_t keep = odd ? spread[2 * g + 1] : spread[2 * g];
            const uint32_t got = __shfl_xor_sync(0xffffffffu, give, 1);
            const uint32_t lo_n = odd ? got : keep;   // even position -> low nibble
            const uint32_t hi_n = odd ? keep : got;
            uint32_t wd = (lo_n | (hi_n << 4)) ^ 0x88888888u;   // offset binary -> two's complement
            // byte k of wd: a = 4 g + k, c' = odd, output byte 256 a + 128 r + 64 c' + (i >> 1).  A 4 x 4
            // byte transpose among the lanes (i >> 1) & 3 = 0..3 turns these into aligned 32-bit words.
            uint32_t pw = __shfl_xor_sync(0xffffffffu, wd, 2);
            wd = __byte_perm(wd, pw, sel1);
            pw = __shfl_xor_sync(0xffffffffu, wd, 4);
            wd = __byte_perm(wd, pw, sel2);
            q[(4 * g + r4) * 64] = wd;
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) wtc::mbar_arrive(acc_empty(ab));
    }
  }

  if (*abort_flag != 0) {
    // after a timeout: give copies and tensor-core operations already started the time to land
    unsigned long long t0, now;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    do {
      __nanosleep(1000);
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
    } while (now - t0 < 50000ull);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace ptc
}  // namespace smoothrot
