// K = 4096 without a diagonal (the exact online Hadamard transform of the paper's deployment,
// where Lambda^-1 sits in the producing layer): the rotation runs on the fifth-generation tensor
// cores.  Included by rotate_quant.cu (same translation unit: it shares the status word and the
// quantizer helpers).
//
// A row of 4096 fp16 values is 32 groups of 128.  With H4096 = H32 (x) H128 (Sylvester), the
// order-128 factor inside every group is a dense +-1 product that takes the raw fp16 values as
// exact operands:
//
//     D[i][n] = sum_k H128[i][k] * x[token][128 g + k],      n = 32 * token + g,
//
// one tcgen05.mma (kind::f16, M = 128, N = 128 or 192, fp32 accumulators in tensor memory) per 16
// values of k, eight per batch of four or six tokens.  The operands never pass through registers: TMA drops the
// rows into shared memory in the K-major, 128-byte-swizzled form the tensor core reads (a row of
// the B operand = one group, 256 bytes = two swizzle atoms along K), and H128 is written once per
// CTA in the same form.  Lane i of tensor memory then holds output i of every group: a thread
// that reads its lane's 32 columns of a token (tcgen05.ld 32x32b.x32) owns the 32 values that
// the order-32 factor combines, so the remaining five butterfly stages run in its registers, in
// fp32, with no exchange at all.  Row maximum (128 threads), step, rounding and packing follow as
// in the other kernels; the codes of eight consecutive positions meet through warp shuffles.
//
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 4.. epilogue (one warp per token of a batch
// and tensor-memory lane quarter: 16 warps for batches of four rows, 24 for batches of six).
// Pipelines: 192 KB of row batches in shared memory (6 x 32 KB or 4 x 48 KB), 2 accumulators.
// Every mbarrier wait is bounded; on expiry the CTA records a code and winds down.
#pragma once

namespace smoothrot {
namespace wtc {

constexpr int kABytes = 128 * 128 * 2;           // H128 as fp16, two K halves of 16 KB

// kTokens rows per batch: N = 32 kTokens accumulator columns, one epilogue warp per token and
// tensor-memory lane quarter.  4 for short inputs (finer batches), 6 for long ones.
template <int kTokens>
struct Cfg {
  static constexpr int kCols = 32 * kTokens;
  static constexpr int kStageBytes = kTokens * 4096 * 2;          // two K halves
  static constexpr int kStages = (192 * 1024) / kStageBytes;      // batches of rows in shared memory
  static constexpr int kEpiWarps = 4 * kTokens;
  static constexpr int kThreads = 32 * (4 + kEpiWarps);
  static constexpr int kBarOffset = kABytes + kStages * kStageBytes;
  // barriers: full[kStages], empty[kStages], acc_full[2], acc_empty[2]; then tmem slot, abort flag, maxima
  static constexpr int kNumBarriers = 2 * kStages + 4;
  static constexpr int kMiscOffset = kBarOffset + 8 * kNumBarriers;
  static constexpr int kSmemBytes = 1024 /*alignment slack*/ + kMiscOffset + 16 + kTokens * 2 * 4 * 4;
  // fp16 x fp16 -> fp32, both operands K-major, M = 128, N = kCols
  static constexpr uint32_t kIdesc = (1u << 4) | (uint32_t(kCols >> 3) << 17) | (uint32_t(128 >> 4) << 24);
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of the tensor-core rotation kernel");
  static_assert(kCols % 16 == 0 && kCols <= 256 && kThreads <= 1024, "tile limits");
};

enum Site { kSiteProducer = 17, kSiteMmaFull = 18, kSiteMmaAcc = 19, kSiteEpilogue = 20 };

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Bounded wait on an mbarrier phase; false if it ran out or another role of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int site) {
  if (row_copy_done(bar, parity)) return true;
  unsigned long long t0;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (uint32_t spin = 1;; ++spin) {
    if (row_copy_done(bar, parity)) return true;
    if ((spin & 63u) == 0u) {
      if (*abort_flag != 0) return false;
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (now - t0 > g_rotate_wait_limit_ns) {
        *abort_flag = 1;
        atomicCAS(&g_rotate_status, 0, site);
        return false;
      }
    }
  }
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, groups of
// 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return (uint64_t(hi) << 32) | lo;
}

__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_load32(uint32_t taddr, float* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7]),
        "=f"(r[8]), "=f"(r[9]), "=f"(r[10]), "=f"(r[11]), "=f"(r[12]), "=f"(r[13]), "=f"(r[14]), "=f"(r[15]),
        "=f"(r[16]), "=f"(r[17]), "=f"(r[18]), "=f"(r[19]), "=f"(r[20]), "=f"(r[21]), "=f"(r[22]), "=f"(r[23]),
        "=f"(r[24]), "=f"(r[25]), "=f"(r[26]), "=f"(r[27]), "=f"(r[28]), "=f"(r[29]), "=f"(r[30]), "=f"(r[31])
      : "r"(taddr)
      : "memory");
}

// One K half (64 values of every group) of a batch of kTokens rows: box 64 x 1 x 32 x kTokens of
// the [rows][32 groups][2 halves][64 values] view, 32 KB, rows of the box = (token, group).
__device__ __forceinline__ void load_half(uint32_t dst, const CUtensorMap* map, uint32_t bar, int half, int row0) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(half), "r"(0), "r"(row0)
      : "memory");
}

// The part of the epilogue after the tensor-memory load: r[g] is the order-128 factor's output i of
// group g of one token (position 128 g + i), unnormalised; `norm` times the final value is the
// rotated entry (2^-6, times the inverse of a power-of-two scale the caller may have applied).
// Order-32 factor over g in registers, row maximum over the 128 threads that share the token
// (they meet at named barrier `barrier_id`; `mine` is their four-float exchange slot), step,
// rounding by the 1.5 * 2^23 trick, and packing: the codes of eight consecutive positions meet
// through warp shuffles.
template <bool kQuant, bool kLowClamp>
__device__ __forceinline__ void finish_token(float* r, float norm, int i, int lane, int quarter, volatile float* mine,
                                             int barrier_id, float clip, int64_t m, uint8_t* __restrict__ q_out,
                                             float* __restrict__ step_out, float* __restrict__ y_out) {
  const bool odd = (i & 1) != 0;
  const int r4 = (i >> 1) & 3;
  const uint32_t sel1 = (r4 & 1) ? 0x3715u : 0x6240u;
  const uint32_t sel2 = (r4 & 2) ? 0x3276u : 0x5410u;
  // the order-32 factor over the groups g: r[g] is position 128 g + i
  f32x2 v[16];
#pragma unroll
  for (int p = 0; p < 16; ++p) v[p] = pack2(r[2 * p] + r[2 * p + 1], r[2 * p] - r[2 * p + 1]);
  butterflies_between_pairs<16>(v);

  if (!kQuant) {
    float* y = y_out + m * 4096 + i;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      float a, c;
      unpack2(v[p], a, c);
      y[(2 * p) * 128] = a * norm;
      y[(2 * p + 1) * 128] = c * norm;
    }
    return;
  }

  float am[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
  for (int p = 0; p < 16; ++p) {
    float a, c;
    unpack2(v[p], a, c);
    am[p & 3] = fmaxf(fmaxf(am[p & 3], fabsf(a)), fabsf(c));
  }
  float amax = warp_max(fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])));
  if (lane == 0) mine[quarter] = amax;
  asm volatile("bar.sync %0, 128;" ::"r"(barrier_id) : "memory");
  amax = fmaxf(fmaxf(mine[0], mine[1]), fmaxf(mine[2], mine[3])) * norm;
  const float step = step_from_absmax(amax, clip);
  if (i == 0) step_out[m] = step;
  const float inv = __frcp_rn(step) * norm;
  const f32x2 inv2 = pack2(inv, inv);
  const float kMagic = 12582912.0f + 8.0f;  // 1.5 * 2^23 + 8: low byte = code + 8
  const f32x2 magic2 = pack2(kMagic, kMagic);
  uint32_t spread[8];                       // four codes per word, one per byte: groups 4 w .. 4 w + 3
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    uint32_t c4[4];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      float q0, q1;
      unpack2(fma2(v[2 * w + k], inv2, magic2), q0, q1);
      if (kLowClamp) {
        q0 = fmaxf(fminf(q0, 12582912.0f + 15.0f), 12582912.0f);
        q1 = fmaxf(fminf(q1, 12582912.0f + 15.0f), 12582912.0f);
      }
      c4[2 * k] = __float_as_uint(q0);
      c4[2 * k + 1] = __float_as_uint(q1);
    }
    uint32_t four = __byte_perm(__byte_perm(c4[0], c4[1], 0x0040), __byte_perm(c4[2], c4[3], 0x0040), 0x5410);
    if (!kLowClamp) four -= (four >> 4) & 0x01010101u;   // the code +8 comes down to +7
    spread[w] = four;
  }
  // Lanes 2p and 2p + 1 hold the even and the odd position of each output byte: the even lane
  // finishes the words with even w, the odd lane those with odd w.
  uint32_t* q = reinterpret_cast<uint32_t*>(q_out + m * 2048) + (i >> 3);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint32_t give = odd ? spread[2 * c] : spread[2 * c + 1];
    const uint32_t keep = odd ? spread[2 * c + 1] : spread[2 * c];
    const uint32_t got = __shfl_xor_sync(0xffffffffu, give, 1);
    const uint32_t lo_n = odd ? got : keep;   // even position -> low nibble
    const uint32_t hi_n = odd ? keep : got;
    uint32_t wd = (lo_n | (hi_n << 4)) ^ 0x88888888u;   // offset binary -> two's complement
    // byte k of wd: group 4 (2c + odd) + k, output byte 64 g + (i >> 1).  A 4 x 4 byte transpose
    // among the lanes (i >> 1) & 3 = 0..3 turns these into aligned 32-bit words.
    uint32_t pw = __shfl_xor_sync(0xffffffffu, wd, 2);
    wd = __byte_perm(wd, pw, sel1);
    pw = __shfl_xor_sync(0xffffffffu, wd, 4);
    wd = __byte_perm(wd, pw, sel2);
    const int g = 4 * (2 * c + (odd ? 1 : 0)) + r4;
    q[g * 16] = wd;
  }
}

template <bool kQuant, bool kLowClamp, int kTokens>
__global__ void __launch_bounds__(Cfg<kTokens>::kThreads, 1)
walsh4096_tc_kernel(const __grid_constant__ CUtensorMap xmap, int64_t M, float clip,
                    uint8_t* __restrict__ q_out, float* __restrict__ step_out, float* __restrict__ y_out) {
  using C = Cfg<kTokens>;
  constexpr int kStages = C::kStages, kStageBytes = C::kStageBytes, kThreads = C::kThreads;
  constexpr int kBarOffset = C::kBarOffset, kMiscOffset = C::kMiscOffset, kEpiWarps = C::kEpiWarps;
  extern __shared__ uint8_t smem_dyn[];
  const uint32_t dyn = smem_addr(smem_dyn);
  const uint32_t base = (dyn + 1023u) & ~1023u;
  uint8_t* smem = smem_dyn + (base - dyn);
  const uint32_t a_base = base;                          // H128: K half h at + 16 KB * h
  const uint32_t b_base = base + kABytes;                // batches: stage s at + 64 KB * s, K half h at + 32 KB * h
  const uint32_t bar_base = base + kBarOffset;
  auto full = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
  auto acc_empty = [&](int s) { return bar_base + 8u * (2 * kStages + 2 + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kMiscOffset);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile float* red = reinterpret_cast<volatile float*>(smem + kMiscOffset + 16);   // [slot][parity][quarter]

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  const int64_t batches = (M + kTokens - 1) / kTokens;

  // The producer's thread starts the copy of the CTA's first batch before anything else: it depends
  // on one barrier only, and its latency (tensor-map fetch + DRAM) is the longest item of the set-up.
  // The later stages are requested after the set-up barrier, so that every CTA's first batch is
  // ahead of them in the memory system.
  uint32_t produced = 0;
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&xmap) : "memory");
    mbar_init(full(0), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (int64_t(blockIdx.x) < batches) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full(0)), "r"(uint32_t(kStageBytes))
                   : "memory");
      load_half(b_base, &xmap, full(0), 0, int(int64_t(blockIdx.x) * kTokens));
      load_half(b_base + kStageBytes / 2, &xmap, full(0), 1, int(int64_t(blockIdx.x) * kTokens));
      produced = 1;
    }
    for (int s = 0; s < kStages; ++s) {
      if (s > 0) mbar_init(full(s), 1);
      mbar_init(empty(s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(acc_full(s), 1);
      mbar_init(acc_empty(s), kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // H128 in the operand's shared-memory form: row i = 128 bytes per K half, 16-byte unit u at u ^ (i & 7)
  for (int idx = threadIdx.x; idx < 128 * 16; idx += kThreads) {
    const int i = idx >> 4, unit = idx & 15;          // unit: K half (bit 3) and 16-byte unit inside it
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
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // H128 was written by ordinary stores
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
      // the first batch is already on its way (see above)
      uint32_t it = produced;
      for (int64_t b = int64_t(blockIdx.x) + int64_t(produced) * gridDim.x; b < batches; b += gridDim.x, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (it / kStages) & 1u;
        if (!mbar_wait(empty(s), ph ^ 1u, abort_flag, kSiteProducer)) break;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full(s)), "r"(uint32_t(kStageBytes))
                     : "memory");
        const uint32_t dst = b_base + uint32_t(s) * kStageBytes;
        load_half(dst, &xmap, full(s), 0, int(b * kTokens));
        load_half(dst + kStageBytes / 2, &xmap, full(s), 1, int(b * kTokens));
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
        if (!mbar_wait(acc_empty(ab), aph ^ 1u, abort_flag, kSiteMmaAcc)) break;
        if (!mbar_wait(full(s), ph, abort_flag, kSiteMmaFull)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + uint32_t(ab * 256);
        const uint32_t b_addr = b_base + uint32_t(s) * kStageBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          // K half ks >> 2; 16 fp16 = 32 bytes further along K inside the swizzle atom: + 2 units
          const uint64_t da = desc_sw128(a_base + uint32_t((ks >> 2) * 16384)) + uint64_t(2 * (ks & 3));
          const uint64_t db = desc_sw128(b_addr + uint32_t((ks >> 2) * (kStageBytes / 2))) + uint64_t(2 * (ks & 3));
          mma_f16(tmem_d, da, db, C::kIdesc, ks > 0 ? 1u : 0u);
        }
        commit(empty(s));
        commit(acc_full(ab));
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;            // the tensor-memory lanes this warp may read: 32 quarter .. + 31
    const int slot = (warp - 4) >> 2;        // takes the tokens slot, slot + kEpiSlots, .. of a batch
    const int i = quarter * 32 + lane;       // output index inside a group (position = 128 g + i)
    uint32_t it = 0, tok_count = 0;
    bool ok = true;
    for (int64_t b = blockIdx.x; b < batches && ok; b += gridDim.x, ++it) {
      const int ab = it & 1;
      const uint32_t aph = (it >> 1) & 1u;
      if (!mbar_wait(acc_full(ab), aph, abort_flag, kSiteEpilogue)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int tk = slot; tk < kTokens; tk += kTokens) {
        const int64_t m = b * kTokens + tk;
        if (m >= M) break;                   // the same for the four warps that share the token
        float r[32];
        tmem_load32(tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(ab * 256 + tk * 32), r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        finish_token<kQuant, kLowClamp>(r, 0.015625f, i, lane, quarter, red + (slot * 2 + (tok_count & 1)) * 4, 1 + slot,
                                         clip, m, q_out, step_out, y_out);
        ++tok_count;
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(ab));
    }
  }

  if (*abort_flag != 0) {
    // after a timeout: give copies and tensor-core operations already started the time to land
    // before the CTA returns its shared and tensor memory
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

}  // namespace wtc
}  // namespace smoothrot
