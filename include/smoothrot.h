/*
 * libsmoothrot: the W4A4 SmoothRot linear layer on one NVIDIA B200 (sm_100a).
 *
 * The library implements the quantized linear layer that the SmoothRot method
 * produces.  Notation (the paper's, with PyTorch's weight layout):
 *
 *   X  [M x K] fp16   activations, one row per token (K = input channels)
 *   W  [N x K] fp16   weights, one row per output channel;  Y = X W^T
 *   s  [K]     fp32   smoothing scales, Lambda = diag(s)
 *   d  [K]     fp32   +1/-1 sign diagonal that randomises the Hadamard matrix
 *   H          +1/-1  Hadamard matrix of order K (H H^T = K I):
 *                     K = 2^p : Sylvester / Walsh, H[i][j] = (-1)^popcount(i & j)
 *                     K = 28 * 2^p : kron(H28, H_{2^p}), index j = a * 2^p + b,
 *                     H28 = Paley construction I over GF(27) (smoothrot_paley28)
 *                     K = 12 * 2^p, 20 * 2^p : the same with Paley I over GF(11), GF(19)
 *                     (smoothrot_base_matrix; an addition for other layer widths, the
 *                     paper's models need only the two forms above)
 *
 * The equivalent transformation (Eq. 2 of the paper) is
 *   Y = (X diag(pre_x) H / sqrt(K)) (W diag(pre_w) H / sqrt(K))^T,
 *   pre_x = d / s,  pre_w = s * d,
 * i.e. A = (H Lambda)^-1 of the Methodology section with the random signs
 * merged into the diagonal.  Both factors are quantized to signed 4-bit codes
 * (Eq. 1, symmetric form, codes in [-8, 7]) with one fp32 step size per row.
 *
 * Packed INT4 layout (used for Xq and Wq): row-major, K/2 bytes per row; byte
 * i of a row holds code 2i in bits 0-3 and code 2i+1 in bits 4-7, each as
 * 4-bit two's complement.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers unless marked "host".  The
 *     caller owns every buffer; the library allocates nothing and keeps no
 *     reference after the work it enqueued has run.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls only enqueue work; they do not synchronise.
 *   - Leading dimensions (ldx, ldw, ldy) count elements, not bytes.
 *   - fp16 inputs must be 16-byte aligned with leading dimensions that are
 *     multiples of 8; packed tensors must be 16-byte aligned.
 *   - K must be 2^p with 7 <= p <= 13, or 12 * 2^p, 20 * 2^p or 28 * 2^p with 3 <= p <= 10.
 *   - Return value: SMOOTHROT_OK (0) or a negative smoothrot_status.  On an
 *     error nothing has been enqueued.  A size of zero rows is valid and
 *     enqueues nothing.
 */
#ifndef SMOOTHROT_H_
#define SMOOTHROT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SMOOTHROT_OK = 0,
  SMOOTHROT_INVALID_ARG = -1,         /* null pointer, negative size, bad ratio */
  SMOOTHROT_UNSUPPORTED_K = -2,       /* K is not one of the supported orders */
  SMOOTHROT_BAD_ALIGNMENT = -3,       /* pointer or leading dimension misaligned */
  SMOOTHROT_WORKSPACE_TOO_SMALL = -4, /* see smoothrot_workspace_bytes */
  SMOOTHROT_CUDA_ERROR = -5,          /* a CUDA runtime / driver call failed */
  SMOOTHROT_DEVICE_TIMEOUT = -6,      /* a bounded wait inside a kernel ran out */
  SMOOTHROT_STATIC_SCRATCH_EXCEEDED = -7 /* shape needs more than SMOOTHROT_STATIC_SCRATCH_BYTES */
} smoothrot_status;

/* Host. Text for a status code; never NULL. */
const char* smoothrot_status_string(int status);

/*
 * Scale calibration.  Methodology section:
 *     s_j = max|X_j|^alpha / max|W_j|^(1 - alpha)
 * with max|X_j| taken over all calibration tokens of the layer's raw input
 * and max|W_j| over the output channels of the original weights.
 *
 * Call once per calibration batch.  Every call folds the batch into the
 * running per-channel maximum  amax[j] = max(amax[j], max_t |X[t][j]|);
 * the caller zero-fills amax before the first batch.  X may be NULL with
 * T = 0.  When `finalize` is non-zero the call also reads W [N x K] and writes
 *     s[j]     = max(amax[j], eps)^alpha / max(wmax[j], eps)^(1 - alpha),
 *                floored at eps = 1e-5  (fp64 arithmetic, rounded to fp32)
 * and, if `d` is non-NULL, the two diagonals the other calls take:
 *     pre_w[j] = s[j] * d[j]          (for smoothrot_fuse_weights)
 *     pre_x[j] = d[j] / s[j]          (for smoothrot_quant_act)
 * pre_w_out / pre_x_out may each be NULL.  s_out doubles as the scratch for
 * max|W_j| while the call runs.  W, s_out are ignored when finalize == 0.
 */
int smoothrot_calibrate(const void* X_f16, int64_t T, int64_t K, int64_t ldx,
                        const void* W_f16, int64_t N, int64_t ldw,
                        float alpha, int finalize,
                        float* amax_inout, float* s_out,
                        const float* d, float* pre_w_out, float* pre_x_out,
                        void* stream);

/*
 * Offline weight path (Methodology section; Fig. 2's down-projection block
 * "H Lambda W"; Experimental settings, "Quantization": per-channel symmetric
 * round-to-nearest 4-bit weights).  For every row n of W:
 *     w^   = (W[n][:] * pre) H / sqrt(K)            pre = s * d, or NULL = ones
 *     dw[n]= clip_w * max|w^| / 7                   (1.0 if the row is all zero)
 *     code = clamp(round_half_even(w^ / dw[n]), -8, 7),  packed 2 per byte
 * Wq_out is [N x K/2] bytes, dw_out [N] fp32.  0 < clip_w <= 1.
 */
int smoothrot_fuse_weights(const void* W_f16, int64_t N, int64_t K, int64_t ldw,
                           const float* pre, float clip_w,
                           uint8_t* Wq_out, float* dw_out, void* stream);

/*
 * Offline weight path with the clip-ratio search of the paper's weight quantizer (Experimental
 * settings, "Quantization": per-channel symmetric weights; each clip ratio is the candidate with the
 * least squared quantization error, the candidates being tried one after another).  As smoothrot_fuse_weights, but for every row
 * the ratio is chosen from the grid
 *     ratio_i = fp32(1 - i * (1 - lowest_ratio) / (ratio_count - 1)),   i = 0 .. ratio_count - 1
 * (the paper gives no grid; 1.00 .. 0.50 in 51 steps is what the tests and the oracle use) as the
 * first i that minimises  sum_k (w^_k - code_k * step_i)^2,  step_i = fp32(ratio_i * max|w^|) / 7,
 * with the codes of Eq. 1's symmetric quantizer at that step; the error is summed in fp64.
 * best_out [N] int32 (may be NULL) receives the chosen i.  `workspace` holds the rotated fp32
 * rows: smoothrot_fuse_weights_search_workspace_bytes(N, K) bytes for one pass, or any multiple
 * of 4 K bytes (at least one row) to work in slices.  0 < lowest_ratio <= 1, 1 <= ratio_count <= 1024.
 */
size_t smoothrot_fuse_weights_search_workspace_bytes(int64_t N, int64_t K);
int smoothrot_fuse_weights_search(const void* W_f16, int64_t N, int64_t K, int64_t ldw,
                                  const float* pre, float lowest_ratio, int ratio_count,
                                  uint8_t* Wq_out, float* dw_out, int32_t* best_out,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Online activation path (Fig. 2, "hadamard" then "quantize" before the
 * down-projection; Experimental settings, "Quantization": per-token symmetric
 * 4-bit activations with a constant clip ratio, 0.9 in the paper).  For every
 * token m:
 *     x^   = (X[m][:] * pre) H / sqrt(K)            pre = d / s, or NULL when
 *                                                   Lambda^-1 already sits in
 *                                                   the producing layer
 *     dx[m]= clip_a * max|x^| / 7                   (1.0 if the row is all zero)
 *     code = clamp(round_half_even(x^ / dx[m]), -8, 7),  packed 2 per byte
 * Xq_out is [M x K/2] bytes, dx_out [M] fp32.  0 < clip_a <= 1.
 */
int smoothrot_quant_act(const void* X_f16, int64_t M, int64_t K, int64_t ldx,
                        const float* pre, float clip_a,
                        uint8_t* Xq_out, float* dx_out, void* stream);

/*
 * Online activation quantizer of the layers that have no online Hadamard transform.  Methodology
 * section, last paragraph: every quantized layer quantizes its activations online, in the forward
 * pass, while only two layers also rotate them there (smoothrot_quant_act and
 * smoothrot_quant_act_heads); every other quantized layer receives activations that are already
 * in the rotated basis.  For every token m:
 *     x^   = X[m][:] * pre                       (pre [K] fp32, or NULL for none)
 *     dx[m], codes: from x^ exactly as in smoothrot_quant_act.
 * X [M x ldx] fp16, Xq_out [M x K/2] bytes, dx_out [M] fp32.  K a multiple of 8, K <= 16384.
 */
int smoothrot_quant_act_plain(const void* X_f16, int64_t M, int64_t K, int64_t ldx,
                              const float* pre, float clip_a,
                              uint8_t* Xq_out, float* dx_out, void* stream);

/*
 * Online activation path in front of the attention output projection.  Methodology section: the
 * forward pass contains two online Hadamard transforms, for which the paper defers to QuaRot; it
 * spells out only the one before the down-projection (smoothrot_quant_act).  The other
 * one, as QuaRot describes it, mixes the heads of the attention output: a row of X is the
 * concatenation of n_heads head outputs of head_dim values, and
 *     x^[m][g * head_dim + e] = sum_h X[m][h * head_dim + e] * pre[h * head_dim + e] * H[h][g] / sqrt(n_heads)
 * with H the Sylvester matrix of order n_heads, i.e. the row times (H_heads (x) I_head_dim) /
 * sqrt(n_heads); the per-head factor (I (x) H_head_dim) of the full rotation is folded into the
 * value projection offline.  The transform is exact in the paper's setting, so `pre` is normally
 * NULL.  dx and the codes follow from x^ exactly as in smoothrot_quant_act.
 * X is [M x ldx] fp16 with ldx >= K = n_heads * head_dim, Xq_out [M x K/2] bytes, dx_out [M] fp32.
 * Supported: n_heads in {8, 16, 32, 64}, head_dim in {64, 128, 256} (else SMOOTHROT_UNSUPPORTED_K).
 */
int smoothrot_quant_act_heads(const void* X_f16, int64_t M, int64_t n_heads, int64_t head_dim, int64_t ldx,
                              const float* pre, float clip_a,
                              uint8_t* Xq_out, float* dx_out, void* stream);

/*
 * The online activation path fed directly by the gated linear unit (Fig. 2: the edge
 * "sigma(gate) (.) up -> hadamard -> quantize" in front of the down-projection; Methodology
 * section: Lambda^-1 is absorbed into the up-projection because the gated product is
 * channel-wise, so `pre` is normally NULL or the sign diagonal alone).  Same as
 * smoothrot_quant_act on X[m][j] = SiLU(gate[m][j]) * up[m][j], SiLU(g) = g / (1 + exp(-g)),
 * except that X is formed in fp32 inside the kernel and never rounded to fp16 or written to
 * memory.  gate, up: [M x K] fp16 with leading dimensions ld_gate, ld_up (multiples of 8,
 * 16-byte aligned rows).  K = 14336 runs the dedicated kernel; other supported K run the generic
 * one-row-per-block kernel.
 */
int smoothrot_quant_act_glu(const void* gate_f16, const void* up_f16, int64_t M, int64_t K,
                            int64_t ld_gate, int64_t ld_up, const float* pre, float clip_a,
                            uint8_t* Xq_out, float* dx_out, void* stream);

/*
 * The quantized layer (Eq. 2's product on the integer codes of Eq. 1, then
 * Eq. 1's dequantizer Q(x) = x_int * step applied to both factors):
 *     acc[m][n] = sum_k Xq[m][k] * Wq[n][k]                    (int32, exact)
 *     Y[m][n]   = fp16( float(acc[m][n]) * dx[m] * dw[n] )
 * Xq [M x K/2], Wq [N x K/2] packed; dx [M], dw [N] fp32; Y [M x ldy] fp16
 * with ldy >= N, ldy a multiple of 8, Y 16-byte aligned.  K must be a multiple
 * of 128 and at most 65536; any M >= 0 and any N >= 0 that is a multiple of 8.
 * `workspace` must hold smoothrot_workspace_bytes(M, N, K) bytes (it may be
 * NULL when that is 0); its contents on entry do not matter.
 */
int smoothrot_linear(const uint8_t* Xq, const float* dx, int64_t M,
                     const uint8_t* Wq, const float* dw, int64_t N, int64_t K,
                     void* Y_f16, int64_t ldy,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * smoothrot_linear without a caller-provided workspace.  (An addition of this
 * library; the paper has no counterpart.)
 *
 * Who needs it: code that must run the layer but is not in a position to
 * obtain device memory for the split-K scratch.  Typical cases are a plug-in
 * inside a serving process whose host application handed out all device
 * memory at start-up and forbids cudaMalloc afterwards, a component that is
 * only ever given the input and output buffers of the layer, or a process in
 * which cudaMalloc would fail because another allocator has already reserved
 * the whole device.  For such callers the scratch lives inside the library: a
 * fixed array of SMOOTHROT_STATIC_SCRATCH_BYTES in device memory that belongs
 * to the loaded module.  Every GPU on which the library is used keeps that
 * many bytes occupied until the process exits, whether or not this entry
 * point is ever called there.
 *
 * Same arguments, results and error behaviour as smoothrot_linear (the same
 * checks in the same order, before anything else), minus the workspace pair.  The call itself allocates and frees nothing.  Shapes whose
 * smoothrot_workspace_bytes(M, N, K) exceeds SMOOTHROT_STATIC_SCRATCH_BYTES
 * are refused with SMOOTHROT_STATIC_SCRATCH_EXCEEDED and nothing is enqueued
 * (use smoothrot_linear with your own workspace for those).
 *
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current) and remembers it; make that
 * first call before starting any stream capture on the device.
 *
 * There is ONE array per device, shared by every call: two calls whose work
 * may overlap on the GPU (different streams, or several host threads) race on
 * it and produce garbage.  Calls on one stream are safe.  The array keeps
 * whatever the previous call left; this entry point never depends on those
 * contents, because each call overwrites every partial sum it later reads.
 */
#define SMOOTHROT_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
int smoothrot_linear_static_scratch(const uint8_t* Xq, const float* dx, int64_t M,
                                    const uint8_t* Wq, const float* dw, int64_t N, int64_t K,
                                    void* Y_f16, int64_t ldy, void* stream);

/*
 * KV-cache quantizer (Eq. 1, asymmetric form; Experimental settings, "Quantization": KV caches
 * are quantized asymmetrically with a group size of 128 and a clip ratio of 0.95).  For every
 * group of 128 consecutive values of a row of X [rows x C] fp16 (C a multiple of 128):
 *     hi = fp32(clip * max), lo = fp32(clip * min)        (the ratio shrinks both ends)
 *     step = (hi - lo) / 15                               (1.0 for a constant group)
 *     zero = -round_half_even(lo / step)
 *     code = clamp(round_half_even(x / step) + zero, 0, 15)
 * all in fp32.  q_out [rows x C/2] bytes holds the unsigned codes, value 2i in bits 0-3 and value
 * 2i+1 in bits 4-7; step_out, zero_out [rows x C/128] fp32 (zero is integer valued and may lie
 * outside 0..15 when a group does not straddle zero).  0 < clip <= 1.
 * smoothrot_kv_dequant is Eq. 1's dequantizer  Y = fp16((code - zero) * step),  Y [rows x ldy].
 */
int smoothrot_kv_quant(const void* X_f16, int64_t rows, int64_t C, int64_t ldx, float clip,
                       uint8_t* q_out, float* step_out, float* zero_out, void* stream);
int smoothrot_kv_dequant(const uint8_t* q, const float* step, const float* zero, int64_t rows,
                         int64_t C, void* Y_f16, int64_t ldy, void* stream);

/*
 * The whole online layer for a handful of tokens in one kernel: the online activation path
 * followed by smoothrot_linear (Fig. 2: ["hadamard" ->] "quantize" -> the quantized projection; Eq. 2
 * on Eq. 1's integer codes), for decode steps, where two launches cost more than the work.  Every
 * CTA prepares the tokens for itself while its share of the weights is in flight.
 *   rotation = 1: the tokens go through smoothrot_quant_act's path (x * pre) H / sqrt(K), same
 *                 formulas, fp32 butterflies in a different order of additions.  K = 4096, M <= 4.
 *   rotation = 0: through smoothrot_quant_act_plain's path (x * pre, no rotation), same codes.
 *                 K in {1024, 2048, 4096}, M <= 8.
 * The codes and steps are written to Xq_out [M x K/2] / dx_out [M] when those are non-NULL (device,
 * optional).  X [M x ldx] fp16, pre [K] or NULL, Wq [N x K/2] and dw [N] from
 * smoothrot_fuse_weights, Y [M x ldy] fp16, N a multiple of 8.  Other shapes:
 * SMOOTHROT_INVALID_ARG (M) / SMOOTHROT_UNSUPPORTED_K.  No workspace.
 */
int smoothrot_linear_decode(const void* X_f16, int64_t M, int64_t K, int64_t ldx, int rotation,
                            const float* pre, float clip_a, const uint8_t* Wq, const float* dw,
                            int64_t N, void* Y_f16, int64_t ldy, uint8_t* Xq_out, float* dx_out,
                            void* stream);

/* As smoothrot_linear_decode, for the attention output projection: the tokens go through
 * smoothrot_quant_act_heads' path, (x * pre)(H_heads (x) I_head_dim) / sqrt(heads).  Supported:
 * 32 heads of 128 (K = 4096), M <= 4. */
int smoothrot_linear_decode_heads(const void* X_f16, int64_t M, int64_t n_heads, int64_t head_dim,
                                  int64_t ldx, const float* pre, float clip_a, const uint8_t* Wq,
                                  const float* dw, int64_t N, void* Y_f16, int64_t ldy,
                                  uint8_t* Xq_out, float* dx_out, void* stream);

/* Host. Scratch bytes smoothrot_linear / smoothrot_debug_gemm_i32 want for
 * this shape (0 for shapes that need none).  With M <= 128 a shape that reports
 * a size cannot run without it (SMOOTHROT_WORKSPACE_TOO_SMALL).  With M >= 256 the
 * scratch only serves to split K over otherwise idle SMs (few output tiles, long
 * K): with a smaller or absent workspace the call runs unsplit, slower but with
 * the same result. */
size_t smoothrot_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Host. Name of the kernel (or kernel pair) smoothrot_linear launches for this shape when it is
 * given the workspace smoothrot_workspace_bytes reports: a static string, "none" for shapes the
 * call rejects.  For reports and benchmarks; nothing is launched. */
const char* smoothrot_linear_plan_name(int64_t M, int64_t N, int64_t K);

/*
 * Test exports: values the fused kernels never write to memory.
 *   smoothrot_debug_hadamard: Y[m][:] = (X[m][:] * pre) H / sqrt(K) as fp32
 *     [M x K], the rotation alone (Methodology section).
 *   smoothrot_debug_hadamard_heads: the same for the head-mixing transform of
 *     smoothrot_quant_act_heads, Y [M x n_heads * head_dim] fp32.
 *   smoothrot_debug_gemm_i32: the int32 accumulators acc [M x N] of
 *     smoothrot_linear, computed by the same kernels.
 */
int smoothrot_debug_hadamard(const void* X_f16, int64_t M, int64_t K, int64_t ldx,
                             const float* pre, float* Y_f32, void* stream);
int smoothrot_debug_hadamard_heads(const void* X_f16, int64_t M, int64_t n_heads, int64_t head_dim,
                                   int64_t ldx, const float* pre, float* Y_f32, void* stream);
int smoothrot_debug_gemm_i32(const uint8_t* Xq, int64_t M, const uint8_t* Wq, int64_t N,
                             int64_t K, int32_t* acc,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Test exports for the bounded device-side waits (no passage of the paper: the kernels never
 * spin without bound, and these two calls let a test see a wait run out without hanging
 * anything).
 *   smoothrot_debug_set_wait_limit_ns: host, synchronous.  Sets the limit of every bounded wait
 *     of the library's kernels on the current device, in nanoseconds; 0 restores the default
 *     (two seconds).
 *   smoothrot_debug_wait_expiry: enqueues one warp that waits, through the same bounded wait as
 *     the GEMM kernels, on a barrier nobody arrives on.  When the limit has passed the warp
 *     records code 7 in the status word smoothrot_device_status reads, and the kernel returns.
 */
int smoothrot_debug_set_wait_limit_ns(uint64_t ns);
int smoothrot_debug_wait_expiry(void* stream);

/* Host. Writes the library's own order-28 Paley matrix, row-major, entries
 * +1 / -1, into out[784] (a host buffer). */
int smoothrot_paley28(int8_t* out_host);

/* Host. The same for the small factor of order 12, 20 or 28 (Paley construction I over GF(11),
 * GF(19), GF(27); first row all +1, first column +1 then -1): order * order entries, row-major,
 * into a host buffer.  SMOOTHROT_INVALID_ARG for another order or a null pointer. */
int smoothrot_base_matrix(int order, int8_t* out_host);

/*
 * Host, synchronous.  Kernels never spin without bound: a wait that runs out
 * records a non-zero code in a device-side status word and the kernel
 * returns.  This call copies that word for the current device into
 * *status_host (0 = no timeout so far) and clears it when `clear` is non-zero.
 */
int smoothrot_device_status(int* status_host, int clear);

/* Host. Number of kernels this library has launched since it was loaded
 * (all devices, all streams); used by the benchmark's launch count. */
int64_t smoothrot_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SMOOTHROT_H_ */
