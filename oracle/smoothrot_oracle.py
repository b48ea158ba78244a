"""CPU oracle for the SmoothRot W4A4 linear layer.  TEST INFRASTRUCTURE ONLY.

A plain, slow restatement of what the paper's quantized linear layer computes,
written from the paper's formulas.  It is what the CUDA library is checked
against; the library itself never imports, links or calls anything here, and
this file imports nothing from the library.  Only the tests, the smoke check
and the benchmark's CPU-baseline leg use it.

What follows the paper, by passage:

* Eq. 1 and the text under it: the uniform integer quantizer, symmetric form
  (zero point 0, step = max|x| / (2^(b-1) - 1)), and the dequantizer
  Q(x) = x_int * step.
* Eq. 2: the equivalent transformation  Y = X W = (X A)(A^-1 W).
* Section "Methodology": the smoothing scale
  s_j = max|X_j|^alpha / max|W_j|^(1-alpha), the diagonal Lambda = diag(s)
  folded into the weights, and the Hadamard rotation applied online to the
  activations and offline to the weights, A = (H Lambda)^-1.
* Section "Experimental settings", paragraph "Quantization": 4 bits,
  per-token symmetric activations with clip ratio 0.9, per-output-channel
  symmetric round-to-nearest weights.
* Eq. 1, asymmetric form, and "Quantization": KV caches with asymmetric
  quantization, group size 128 and clip ratio 0.95 (kv_quantize).
* Fig. 2 (the feed-forward block): the down-projection input is the gated
  product sigma(gate) (.) up; quant_act_glu takes that edge in one step.
* Fig. 2 and section "Methodology": the whole feed-forward block, with
  Lambda^-1 absorbed into the up-projection and Lambda into the
  down-projection (absorb_into_up, ffn_block and their float64 companions).
* Section "Methodology", last paragraph: activations are quantized online, in
  the forward pass, for every quantized layer; the layers without an online
  Hadamard transform quantize their input as it is (quant_act_plain).
* Section "Methodology": the forward pass contains two online Hadamard
  transforms, for which the paper defers to QuaRot; it details the one in
  front of the down-projection only.  The other sits in front of the
  attention output projection and, as QuaRot describes it, mixes the heads:
  (H_heads (x) I_head_dim) / sqrt(heads), the per-head factor
  (I (x) H_head_dim) being folded into the value projection offline
  (rotate_heads, rotate_per_head, quant_act_heads).

Floating point: transforms and scales are computed in float64 and rounded once
to float32; the quantizer decisions (step, division, rounding) are taken in
float32, the precision the step sizes are stored in.

Parity status: every function below is pinned by a test in tests/test_oracle_*.py
against a closed form, an invariant, brute force or an independent library
routine.  Nothing here reproduces the paper's perplexity or accuracy tables
(they need its datasets and trained weights): for those, parity unpinned.

Readings taken where the paper is silent or garbled are listed in the design
notes of the repository; the ones that matter to this file are repeated at
the function that takes them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

EPS = 1e-5          # floor on absmax values and on s (not from the paper: a guard)
QMIN, QMAX = -8, 7  # signed 4-bit range


# ---------------------------------------------------------------------------
# Hadamard matrices
# ---------------------------------------------------------------------------

def sylvester(n: int) -> np.ndarray:
    """Walsh-Hadamard matrix of order n = 2^p in natural (Sylvester) order:
    H[i, j] = (-1)^popcount(i & j).  Entries +1/-1 as int8."""
    assert n >= 1 and (n & (n - 1)) == 0, "order must be a power of two"
    idx = np.arange(n, dtype=np.int64)
    a = idx[:, None] & idx[None, :]
    pop = np.zeros_like(a)
    while a.any():
        pop += a & 1
        a >>= 1
    return (1 - 2 * (pop & 1)).astype(np.int8)


# GF(27) = GF(3)[x] / (x^3 + 2x + 1).  An element a0 + a1 x + a2 x^2 has
# index a0 + 3 a1 + 9 a2.
def _gf27_digits(e: int):
    return (e % 3, (e // 3) % 3, e // 9)


def _gf27_index(c) -> int:
    return (c[0] % 3) + 3 * (c[1] % 3) + 9 * (c[2] % 3)


def gf27_sub(a: int, b: int) -> int:
    x, y = _gf27_digits(a), _gf27_digits(b)
    return _gf27_index([x[i] - y[i] for i in range(3)])


def gf27_mul(a: int, b: int) -> int:
    x, y = _gf27_digits(a), _gf27_digits(b)
    p = [0] * 5
    for i in range(3):
        for j in range(3):
            p[i + j] += x[i] * y[j]
    # reduce with x^3 = -2x - 1 = x + 2 (mod 3), highest power first
    for k in (4, 3):
        c = p[k]
        p[k] = 0
        p[k - 2] += c      # x^k = x^(k-3) * (x + 2)
        p[k - 3] += 2 * c
    return _gf27_index(p)


def gf27_chi(e: int) -> int:
    """Quadratic character of GF(27): 0 at zero, +1 on non-zero squares, -1 otherwise."""
    if e == 0:
        return 0
    return 1 if any(gf27_mul(y, y) == e for y in range(1, 27)) else -1


def paley28() -> np.ndarray:
    """Paley construction I for q = 27 (q = 3 mod 4): with the Jacobsthal matrix
    Q[a, b] = chi(a - b) over GF(27) and the skew matrix S = [[0, 1^T], [-1, Q]],
    H28 = I + S.  First row all +1; first column +1 then all -1."""
    q = 27
    S = np.zeros((q + 1, q + 1), dtype=np.int64)
    S[0, 1:] = 1
    S[1:, 0] = -1
    for a in range(q):
        for b in range(q):
            S[1 + a, 1 + b] = gf27_chi(gf27_sub(a, b))
    return (np.eye(q + 1, dtype=np.int64) + S).astype(np.int8)


def legendre(e: int, q: int) -> int:
    """Quadratic character of the prime field GF(q): 0 at zero, +1 on the non-zero squares
    y*y mod q, -1 otherwise (the squares are found by listing them)."""
    e %= q
    if e == 0:
        return 0
    return 1 if any((y * y) % q == e for y in range(1, q)) else -1


def paley_prime(q: int) -> np.ndarray:
    """Paley construction I for a prime q = 3 mod 4, same conventions as paley28 with the
    field elements 0..q-1 in their natural order: Q[a, b] = chi(a - b), S = [[0, 1^T], [-1, Q]],
    H = I + S of order q + 1.  An addition for layer widths 12 * 2^p and 20 * 2^p (q = 11, 19);
    the paper's models need the orders 2^p and 28 * 2^p only."""
    assert q in (11, 19), "only the orders 12 and 20 are built this way"
    S = np.zeros((q + 1, q + 1), dtype=np.int64)
    S[0, 1:] = 1
    S[1:, 0] = -1
    for a in range(q):
        for b in range(q):
            S[1 + a, 1 + b] = legendre(a - b, q)
    return (np.eye(q + 1, dtype=np.int64) + S).astype(np.int8)


def base_matrix(base: int) -> np.ndarray:
    """The small factor of the Kronecker product: Paley I of order 12, 20 or 28."""
    if base == 28:
        return paley28()
    if base in (12, 20):
        return paley_prime(base - 1)
    raise ValueError(f"no base matrix of order {base}")


def split_order(K: int):
    """K = base * 2^p with base 1 (Walsh) or 4 * odd for odd in {3, 5, 7}: 12, 20, 28 (Paley x Walsh).
    The odd part of K decides the base, so the split is unique.  Returns (base, 2^p)."""
    if K >= 1 and (K & (K - 1)) == 0:
        return 1, K
    for base in (28, 20, 12):
        if K >= base and K % base == 0:
            n = K // base
            if (n & (n - 1)) == 0:
                return base, n
    raise ValueError(f"no Hadamard construction for order {K}")


def hadamard_matrix(K: int) -> np.ndarray:
    """The +1/-1 matrix H of order K used for the rotation: Sylvester for 2^p,
    and for base * 2^p the Kronecker product with the Paley matrix on the slow
    index:  H[a*n + b, a'*n + b'] = Hbase[a, a'] * Hn[b, b']."""
    base, n = split_order(K)
    if base == 1:
        return sylvester(n)
    return np.kron(base_matrix(base).astype(np.int8), sylvester(n)).astype(np.int8)


# ---------------------------------------------------------------------------
# Rotation  y = (x * pre) H / sqrt(K)
# ---------------------------------------------------------------------------

def rotate_dense(x: np.ndarray, pre, K: int) -> np.ndarray:
    """The definition: rows of x, multiplied elementwise by `pre` (or by one),
    times the dense matrix H, divided by sqrt(K).  float64 throughout."""
    v = np.asarray(x, dtype=np.float64)
    if pre is not None:
        v = v * np.asarray(pre, dtype=np.float64)[None, :]
    H = hadamard_matrix(K).astype(np.float64)
    return (v @ H) / np.sqrt(np.float64(K))


def _walsh_last_axis(v: np.ndarray) -> np.ndarray:
    """In-place style float64 Walsh-Hadamard butterflies along the last axis
    (natural order, unnormalised): the Sylvester recursion H_2n = [[H, H], [H, -H]]."""
    n = v.shape[-1]
    h = 1
    lead = v.shape[:-1]
    while h < n:
        w = v.reshape(*lead, n // (2 * h), 2, h)
        a = w[..., 0, :] + w[..., 1, :]
        b = w[..., 0, :] - w[..., 1, :]
        v = np.stack((a, b), axis=-2).reshape(*lead, n)
        h *= 2
    return v


def rotate(x: np.ndarray, pre, K: int) -> np.ndarray:
    """Same map as rotate_dense, by float64 butterflies: for K = base * n the row
    is viewed as [base, n], the Walsh transform runs along n and the Paley
    matrix along the base axis (the Kronecker product, factor by factor)."""
    v = np.asarray(x, dtype=np.float64)
    assert v.ndim == 2 and v.shape[1] == K
    if pre is not None:
        v = v * np.asarray(pre, dtype=np.float64)[None, :]
    base, n = split_order(K)
    if base == 1:
        y = _walsh_last_axis(v)
    else:
        w = _walsh_last_axis(v.reshape(v.shape[0], base, n))
        P = base_matrix(base).astype(np.float64)
        # y[m, a', b] = sum_a w[m, a, b] * Hbase[a, a']
        y = np.einsum("mab,ac->mcb", w, P).reshape(v.shape[0], K)
    return y / np.sqrt(np.float64(K))


# ---------------------------------------------------------------------------
# Calibration: s_j = max|X_j|^alpha / max|W_j|^(1 - alpha)
# ---------------------------------------------------------------------------

def channel_absmax(X: np.ndarray) -> np.ndarray:
    """max over rows of |X[:, j]| as float32 (exact for fp16 inputs)."""
    X = np.asarray(X)
    if X.shape[0] == 0:
        return np.zeros(X.shape[1], dtype=np.float32)
    return np.abs(X.astype(np.float32)).max(axis=0)


def smoothing_scales(amax: np.ndarray, wmax: np.ndarray, alpha: float) -> np.ndarray:
    """s_j from the two per-channel maxima, float64 inside, float32 out.
    amax, wmax and s are floored at EPS (a guard the paper does not spell out)."""
    a = np.maximum(np.asarray(amax, dtype=np.float64), EPS)
    w = np.maximum(np.asarray(wmax, dtype=np.float64), EPS)
    s = np.power(a, np.float64(alpha)) / np.power(w, np.float64(1.0 - alpha))
    return np.maximum(s, EPS).astype(np.float32)


def calibrate(X_calib: np.ndarray, W: np.ndarray, alpha: float):
    """Returns (amax[K], s[K]).  max|X_j| ranges over all calibration tokens of
    the layer's raw input; max|W_j| over the output channels of the original W
    ([N, K] layout) for input channel j."""
    amax = channel_absmax(X_calib)
    wmax = channel_absmax(W)
    return amax, smoothing_scales(amax, wmax, alpha)


# ---------------------------------------------------------------------------
# Quantizer (Eq. 1, symmetric, b = 4) and the 2-codes-per-byte packing
# ---------------------------------------------------------------------------

def quantize_rows(v: np.ndarray, clip: float):
    """Per-row symmetric 4-bit quantization of a float32 matrix.

    step[r] = float32(clip * max|v[r]|) / 7   (1.0 for an all-zero row)
    code    = clamp(round_half_even(v / step), -8, 7)

    The clamp is the signed range: the printed Eq. 1 clamps to [0, 2^b - 1],
    which with zero point 0 would erase every negative value, so the signed
    reading is taken.  All arithmetic here is float32.
    Returns (codes int8 [R, C], step float32 [R])."""
    v = np.asarray(v, dtype=np.float32)
    amax = np.abs(v).max(axis=1) if v.shape[1] else np.zeros(v.shape[0], np.float32)
    step = (np.float32(clip) * amax).astype(np.float32) / np.float32(7.0)
    step = np.where(amax == 0, np.float32(1.0), step).astype(np.float32)
    q = np.rint(v / step[:, None])          # float32 division, round half to even
    codes = np.clip(q, QMIN, QMAX).astype(np.int8)
    return codes, step


def pack_codes(codes: np.ndarray) -> np.ndarray:
    """[R, C] int8 codes in [-8, 7] -> [R, C/2] uint8: byte i holds code 2i in
    bits 0-3 and code 2i+1 in bits 4-7, each as 4-bit two's complement."""
    c = np.asarray(codes).astype(np.int16)
    assert c.shape[-1] % 2 == 0
    lo = c[..., 0::2] & 0xF
    hi = c[..., 1::2] & 0xF
    return (lo | (hi << 4)).astype(np.uint8)


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_codes: [R, C/2] uint8 -> [R, C] int8."""
    p = np.asarray(packed, dtype=np.uint8).astype(np.int16)
    lo = p & 0xF
    hi = (p >> 4) & 0xF
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


def dequantize_rows(codes: np.ndarray, step: np.ndarray) -> np.ndarray:
    """Q(x) = x_int * step  (Eq. 1's dequantizer, zero point 0), float64."""
    return codes.astype(np.float64) * np.asarray(step, dtype=np.float64)[:, None]


# ---------------------------------------------------------------------------
# KV-cache quantizer (Eq. 1, asymmetric form; Experimental settings: asymmetric,
# group size 128, clip ratio 0.95)
# ---------------------------------------------------------------------------
KV_GROUP = 128


def kv_quantize(X: np.ndarray, clip: float = 0.95, group: int = KV_GROUP):
    """Asymmetric 4-bit quantization of each group of `group` consecutive values of a row.
    Eq. 1's asymmetric form with the clip ratio shrinking both ends of the range:
        hi = float32(clip * max),  lo = float32(clip * min)
        step = (hi - lo) / 15            (1.0 if hi == lo: a constant group; a reading, the
                                          paper does not treat the degenerate case)
        zero = -round_half_even(lo / step)
        code = clamp(round_half_even(x / step) + zero, 0, 15)
    All decisions in float32.  Returns (codes uint8 [R, C] in 0..15, step f32 [R, C/group],
    zero f32 [R, C/group], integer valued)."""
    X = np.asarray(X)
    R, C = X.shape
    assert C % group == 0
    x = X.astype(np.float32).reshape(R, C // group, group)
    hi = (np.float32(clip) * x.max(axis=2)).astype(np.float32)
    lo = (np.float32(clip) * x.min(axis=2)).astype(np.float32)
    step = ((hi - lo).astype(np.float32) / np.float32(15.0)).astype(np.float32)
    step = np.where(hi == lo, np.float32(1.0), step).astype(np.float32)
    zero = (-np.rint((lo / step).astype(np.float32))).astype(np.float32)
    q = np.rint((x / step[:, :, None]).astype(np.float32)) + zero[:, :, None]
    codes = np.clip(q, 0, 15).astype(np.uint8).reshape(R, C)
    return codes, step, zero


def kv_dequantize(codes: np.ndarray, step: np.ndarray, zero: np.ndarray, group: int = KV_GROUP) -> np.ndarray:
    """Q(x) = (x_int - zero) * step  (Eq. 1's dequantizer), float64, [R, C]."""
    R, C = codes.shape
    c = codes.astype(np.float64).reshape(R, C // group, group)
    y = (c - zero.astype(np.float64)[:, :, None]) * step.astype(np.float64)[:, :, None]
    return y.reshape(R, C)


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """[R, C] uint8 codes in 0..15 -> [R, C/2] uint8, value 2i in bits 0-3, value 2i+1 in bits 4-7."""
    c = np.asarray(codes, dtype=np.uint8)
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    p = np.asarray(packed, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = p & 0xF
    out[..., 1::2] = p >> 4
    return out


# ---------------------------------------------------------------------------
# The two halves of the layer preparation / forward
# ---------------------------------------------------------------------------

def fuse_weights(W: np.ndarray, pre_w, K: int, clip_w: float = 1.0):
    """Offline weight path: each row of W ([N, K]) is multiplied by pre_w
    (= s * d: Lambda and the random signs), rotated by H / sqrt(K), and
    quantized per output channel.  Returns (packed [N, K/2] u8, step [N] f32,
    rotated float32 [N, K])."""
    wr = rotate(W, pre_w, K).astype(np.float32)
    codes, step = quantize_rows(wr, clip_w)
    return pack_codes(codes), step, wr


def clip_ratios(count: int = 51, lowest: float = 0.5) -> np.ndarray:
    """The grid of the weight clip search: `count` ratios from 1.0 down to `lowest`, equally
    spaced, as float32.  The paper only says that each ratio is the one with the least squared
    quantization error among candidates tried one after another; the grid is this repository's reading."""
    i = np.arange(count, dtype=np.float64)
    return (1.0 - i * (1.0 - lowest) / (count - 1)).astype(np.float32)


def clip_search_rows(v: np.ndarray, ratios: np.ndarray):
    """Per row of the float32 matrix v: quantize with every clip ratio of the grid (Eq. 1,
    symmetric, step = float32(ratio * max|v|) / 7, all decisions in float32 as in quantize_rows),
    measure the squared error  sum_k (v_k - code_k * step)^2  in float64, and keep the first ratio
    that attains the minimum (the largest such ratio).
    Returns (codes int8 [R, C], step float32 [R], best index [R], errors float64 [R, len(ratios)])."""
    v = np.asarray(v, dtype=np.float32)
    R = v.shape[0]
    errs = np.empty((R, len(ratios)), dtype=np.float64)
    all_codes, all_steps = [], []
    for i, ratio in enumerate(ratios):
        codes, step = quantize_rows(v, np.float32(ratio))
        deq = codes.astype(np.float64) * step.astype(np.float64)[:, None]
        errs[:, i] = ((v.astype(np.float64) - deq) ** 2).sum(axis=1)
        all_codes.append(codes)
        all_steps.append(step)
    best = np.argmin(errs, axis=1)          # first minimum
    rows = np.arange(R)
    codes = np.stack(all_codes)[best, rows]
    step = np.stack(all_steps)[best, rows]
    return codes, step, best, errs


def fuse_weights_search(W: np.ndarray, pre_w, K: int, ratios: np.ndarray):
    """Offline weight path with the clip-ratio search of the paper's weight quantizer
    (Experimental settings, "Quantization": the weight clip ratios are picked by least squared
    error over a scan of candidates): rotate as in fuse_weights, then clip_search_rows per output channel.
    Returns (packed [N, K/2] u8, step [N] f32, best index [N], errors [N, len(ratios)], rotated f32)."""
    wr = rotate(W, pre_w, K).astype(np.float32)
    codes, step, best, errs = clip_search_rows(wr, ratios)
    return pack_codes(codes), step, best, errs, wr


def quant_act(X: np.ndarray, pre_x, K: int, clip_a: float = 0.9):
    """Online activation path: rows times pre_x (= d / s, or None when
    Lambda^-1 already sits in the producing layer), rotated, quantized per
    token.  Returns (packed [M, K/2] u8, step [M] f32, rotated float32 [M, K])."""
    xr = rotate(X, pre_x, K).astype(np.float32)
    codes, step = quantize_rows(xr, clip_a)
    return pack_codes(codes), step, xr


def quant_act_plain(X: np.ndarray, pre_x, clip_a: float = 0.9):
    """The online activation quantizer of the layers that need no online Hadamard transform (the
    paper integrates only two of those into the forward pass, in front of the down-projection and
    of the attention output projection; every other linear layer sees activations that are already
    in the rotated basis and only quantizes them): rows times pre_x (or one), rounded once to
    float32, then Eq. 1's per-token symmetric quantizer with the clip ratio.
    Returns (packed [M, K/2] u8, step [M] f32, the scaled float32 rows [M, K])."""
    v = np.asarray(X, dtype=np.float64)
    if pre_x is not None:
        v = v * np.asarray(pre_x, dtype=np.float64)[None, :]
    v = v.astype(np.float32)
    codes, step = quantize_rows(v, clip_a)
    return pack_codes(codes), step, v


def rotate_heads(x: np.ndarray, pre, n_heads: int) -> np.ndarray:
    """The online transform in front of the attention output projection: a row is the
    concatenation of n_heads head outputs of head_dim values each, and the heads are mixed
    by the Walsh-Hadamard matrix,
        y[m, g * head_dim + e] = sum_h x[m, h * head_dim + e] * pre[h * head_dim + e] * H[h, g] / sqrt(n_heads),
    i.e. the row times (H_heads (x) I_head_dim) / sqrt(n_heads).  Reading: the paper names
    this transform only by reference to QuaRot; there it is exact (no diagonal), so `pre` is
    normally None.  float64."""
    v = np.asarray(x, dtype=np.float64)
    assert v.ndim == 2 and v.shape[1] % n_heads == 0
    if pre is not None:
        v = v * np.asarray(pre, dtype=np.float64)[None, :]
    M, K = v.shape
    H = sylvester(n_heads).astype(np.float64)
    y = np.einsum("mhe,hg->mge", v.reshape(M, n_heads, K // n_heads), H)
    return y.reshape(M, K) / np.sqrt(np.float64(n_heads))


def rotate_per_head(x: np.ndarray, head_dim: int) -> np.ndarray:
    """The other factor of the same rotation, (I_heads (x) H_head_dim) / sqrt(head_dim): every
    head's head_dim values are transformed on their own.  In the model it is folded into the
    value projection offline (and applied online to queries and keys); here it exists so that
    the product of the two factors can be checked against the full rotation.  float64."""
    v = np.asarray(x, dtype=np.float64)
    assert v.ndim == 2 and v.shape[1] % head_dim == 0
    M, K = v.shape
    y = _walsh_last_axis(v.reshape(M, K // head_dim, head_dim))
    return y.reshape(M, K) / np.sqrt(np.float64(head_dim))


def quant_act_heads(X: np.ndarray, pre_x, n_heads: int, clip_a: float = 0.9):
    """Online activation path in front of the attention output projection: rotate_heads, then
    the per-token symmetric quantizer of quant_act.  Returns (packed [M, K/2] u8, step [M] f32,
    rotated float32 [M, K])."""
    xr = rotate_heads(X, pre_x, n_heads).astype(np.float32)
    codes, step = quantize_rows(xr, clip_a)
    return pack_codes(codes), step, xr


def silu(g: np.ndarray) -> np.ndarray:
    """sigma(g) * g with the logistic function sigma, float64 (the GLU activation of Fig. 2:
    the down-projection input is sigma(gate) (.) up, the two outputs of the fused gate/up layer)."""
    g = np.asarray(g, dtype=np.float64)
    with np.errstate(over="ignore"):
        return g / (1.0 + np.exp(-g))


def glu_product(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    """The down-projection input of Fig. 2: SiLU(gate) * up, element by element, float64,
    not rounded to fp16 (the fused kernel never stores it)."""
    return silu(gate) * np.asarray(up, dtype=np.float64)


def quant_act_glu(gate: np.ndarray, up: np.ndarray, pre_x, K: int, clip_a: float = 0.9):
    """Online activation path fed by the gated linear unit: the edge
    "x -> hadamard -> quantize" of Fig. 2 in one step.  Rows SiLU(gate) * up (float64), times
    pre_x (or None: Lambda^-1 already sits in the up-projection), rotated, quantized per token.
    Returns (packed [M, K/2] u8, step [M] f32, rotated float32 [M, K])."""
    xr = rotate(glu_product(gate, up), pre_x, K).astype(np.float32)
    codes, step = quantize_rows(xr, clip_a)
    return pack_codes(codes), step, xr


# ---------------------------------------------------------------------------
# The feed-forward block of Fig. 2: up/gate projection -> sigma(gate) (.) up ->
# hadamard -> quantize -> down projection, with Lambda^-1 in the up-projection
# and Lambda in the down-projection (section "Methodology").
# ---------------------------------------------------------------------------

def absorb_into_up(W_up: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Lambda^-1 absorbed into the up-projection (section "Methodology": the smoothing diagonal
    of the down-projection input goes into the up-projection, which is legal because the gated
    product is taken channel by channel): output channel j of W_up ([I, K1], rows = the
    down-projection's input channels) is divided by s_j.  float64, not rounded."""
    return np.asarray(W_up, dtype=np.float64) / np.asarray(s, dtype=np.float64)[:, None]


def ffn_plain_fp64(X, W_gate, W_up, W_down) -> np.ndarray:
    """(SiLU(X W_gate^T) (.) X W_up^T) W_down^T: the block of Fig. 2 without any transformation
    or quantization, float64."""
    X = np.asarray(X, np.float64)
    h = glu_product(X @ np.asarray(W_gate, np.float64).T, X @ np.asarray(W_up, np.float64).T)
    return h @ np.asarray(W_down, np.float64).T


def ffn_transformed_fp64(X, W_gate, W_up, W_down, s, d) -> np.ndarray:
    """The same block after the method's transformation and before any quantization, float64:
    the up-projection carries Lambda^-1 (absorb_into_up), the gated product is multiplied by the
    sign diagonal d and rotated online by H / sqrt(I), and the down-projection's rows carry
    Lambda, d and the same rotation (fuse_weights' map).  By Eq. 2, applied through the
    channel-wise product, this equals ffn_plain_fp64 in exact arithmetic."""
    X = np.asarray(X, np.float64)
    I = np.asarray(W_down).shape[1]
    d64 = np.ones(I) if d is None else np.asarray(d, np.float64)
    h = glu_product(X @ np.asarray(W_gate, np.float64).T, X @ absorb_into_up(W_up, s).T)
    hr = rotate(h, d64, I)
    wr = rotate(np.asarray(W_down, np.float64), np.asarray(s, np.float64) * d64, I)
    return hr @ wr.T


def ffn_calibrate(X_calib, W_gate, W_up, W_down, alpha: float):
    """Smoothing scales of the down-projection: the calibration set is sent through the
    unquantized gate/up projections in float64, the gated products are rounded once to fp16 (the
    dtype calibration inputs are handed over in) and enter `calibrate` with the original W_down.
    Returns (h_calib fp16 [T, I], amax [I], s [I])."""
    Xc = np.asarray(X_calib, np.float64)
    h = glu_product(Xc @ np.asarray(W_gate, np.float64).T, Xc @ np.asarray(W_up, np.float64).T)
    with np.errstate(over="ignore"):
        h16 = np.clip(h, -65504.0, 65504.0).astype(np.float16)
    amax, s = calibrate(h16, W_down, alpha)
    return h16, amax, s


def ffn_block(X, W_gate, W_up, W_down, s, d, clip_a: float = 0.9, clip_w: float = 1.0):
    """The quantized feed-forward block of Fig. 2, every arrow one step of this file:

        W_up'  = fp16(absorb_into_up(W_up, s))                 (weights are stored in fp16)
        gate/up layer:  quant_act(X, None, K1) -> linear with fuse_weights([W_gate; W_up'], None, K1)
                        -> G, U  fp16 [M, I]   (one fused layer of 2 I output channels)
        x -> hadamard -> quantize:  quant_act_glu(G, U, d, I)  (Lambda^-1 already sits in W_up')
        down layer:  linear with fuse_weights(W_down, s * d, I)

    The block input is rotated online by the order-K1 Hadamard matrix and the gate/up weights
    carry the same rotation, which stands in for the residual-stream rotation the paper folds
    into the neighbouring layers offline.  Returns a dict of every intermediate."""
    X = np.asarray(X)
    K1 = X.shape[1]
    I = np.asarray(W_down).shape[1]
    with np.errstate(over="ignore"):
        W_up_abs = absorb_into_up(W_up, s).astype(np.float16)
    W_gu = np.concatenate([np.asarray(W_gate, np.float16), W_up_abs], axis=0)
    wq_gu, dw_gu, _ = fuse_weights(W_gu, None, K1, clip_w)
    xq, dx, _ = quant_act(X, None, K1, clip_a)
    Y_gu = linear(xq, dx, wq_gu, dw_gu)
    G, U = Y_gu[:, :I], Y_gu[:, I:]
    d32 = None if d is None else np.asarray(d, np.float32)
    hq, dh, hr = quant_act_glu(G, U, d32, I, clip_a)
    pre_w = np.asarray(s, np.float64) * (1.0 if d is None else np.asarray(d, np.float64))
    wq_d, dw_d, _ = fuse_weights(W_down, pre_w.astype(np.float32), I, clip_w)
    Y = linear(hq, dh, wq_d, dw_d)
    return dict(W_up_abs=W_up_abs, wq_gu=wq_gu, dw_gu=dw_gu, xq=xq, dx=dx, Y_gu=Y_gu,
                hq=hq, dh=dh, hr=hr, pre_w=pre_w.astype(np.float32), wq_d=wq_d, dw_d=dw_d, Y=Y)


def gemm_i32_numpy(xq: np.ndarray, wq: np.ndarray) -> np.ndarray:
    """acc[m, n] = sum_k xq[m, k] * wq[n, k]  on unpacked int8 codes, summed
    in int64 and checked to fit int32."""
    acc = xq.astype(np.int64) @ wq.astype(np.int64).T
    assert acc.size == 0 or (np.abs(acc).max() < 2 ** 31)
    return acc.astype(np.int32)


_GEMM_LIB = None


def _so_path() -> str:
    """The shared object is compiled for the host it runs on (-march=native),
    so its name carries a digest of the host's CPU feature flags: a copy built
    on another machine is never loaded."""
    import hashlib
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    tag = hashlib.sha1(flags.encode()).hexdigest()[:10]
    here = os.path.dirname(os.path.abspath(__file__))
    return os.path.join(here, f"liboracle_gemm_{tag}.so")


def _gemm_lib():
    """Builds (once per host type) and loads the plain C triple loop in gemm_i32.c."""
    global _GEMM_LIB
    if _GEMM_LIB is None:
        here = os.path.dirname(os.path.abspath(__file__))
        src = os.path.join(here, "gemm_i32.c")
        so = _so_path()
        if (not os.path.exists(so)) or os.path.getmtime(so) < os.path.getmtime(src):
            build_c()
        lib = ctypes.CDLL(so)
        lib.oracle_gemm_i32.restype = ctypes.c_int
        lib.oracle_gemm_i32.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                        ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
        lib.oracle_gemm_threads.restype = ctypes.c_int
        _GEMM_LIB = lib
    return _GEMM_LIB


def build_c() -> str:
    """Compile gemm_i32.c into a shared object next to it; returns the path."""
    here = os.path.dirname(os.path.abspath(__file__))
    src = os.path.join(here, "gemm_i32.c")
    so = _so_path()
    tmp = so + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC", "-o", tmp, src])
    os.replace(tmp, so)
    return so


def gemm_threads() -> int:
    """Number of host threads the C loop uses."""
    return int(_gemm_lib().oracle_gemm_threads())


def gemm_i32(xq: np.ndarray, wq: np.ndarray) -> np.ndarray:
    """Same sum as gemm_i32_numpy, by the C triple loop (rows of the output
    shared among host threads), for sizes where numpy's integer matmul is too slow."""
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = xq.shape
    N, K2 = wq.shape
    assert K == K2
    acc = np.empty((M, N), dtype=np.int32)
    rc = _gemm_lib().oracle_gemm_i32(xq.ctypes.data, M, wq.ctypes.data, N, K, acc.ctypes.data)
    if rc != 0:
        raise OverflowError("an accumulator left the int32 range")
    return acc


def dequant_output(acc: np.ndarray, dx: np.ndarray, dw: np.ndarray) -> np.ndarray:
    """Y[m, n] = fp16( acc[m, n] * dx[m] * dw[n] ): the exact product in
    float64, rounded once to fp16."""
    y = acc.astype(np.float64) * np.asarray(dx, np.float64)[:, None] * np.asarray(dw, np.float64)[None, :]
    with np.errstate(over="ignore"):
        return y.astype(np.float16)


def linear(xq_packed: np.ndarray, dx: np.ndarray, wq_packed: np.ndarray, dw: np.ndarray) -> np.ndarray:
    """The quantized layer proper: integer GEMM on the unpacked codes, then
    the per-token x per-output-channel dequantization to fp16."""
    acc = gemm_i32(unpack_codes(xq_packed), unpack_codes(wq_packed))
    return dequant_output(acc, dx, dw)


def smoothrot_layer(X, X_calib, W, d, alpha, clip_a=0.9, clip_w=1.0):
    """Whole path on one layer: calibrate -> fuse weights -> quantize
    activations -> integer GEMM -> dequantize.  Returns a dict of every
    intermediate."""
    K = X.shape[1]
    amax, s = calibrate(X_calib, W, alpha)
    d = np.asarray(d, dtype=np.float32)
    pre_w = (s.astype(np.float64) * d).astype(np.float32)
    pre_x = (d.astype(np.float64) / s.astype(np.float64)).astype(np.float32)
    wq, dw, wr = fuse_weights(W, pre_w, K, clip_w)
    xq, dx, xr = quant_act(X, pre_x, K, clip_a)
    acc = gemm_i32(unpack_codes(xq), unpack_codes(wq))
    Y = dequant_output(acc, dx, dw)
    return dict(amax=amax, s=s, pre_w=pre_w, pre_x=pre_x, wq=wq, dw=dw, wr=wr,
                xq=xq, dx=dx, xr=xr, acc=acc, Y=Y)
