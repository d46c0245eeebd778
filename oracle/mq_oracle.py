"""CPU oracle for the W4A8 modality-specific static-quantized (MSQ) linear path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
kernels are compared against.  It is imported by the tests, by the smoke check
and by the benchmark's CPU-baseline leg, and by nothing else; the product path
never calls it and shares no code, table or constant with it.

Every function restates, in NumPy, one step of the method as the paper (MQuant,
arXiv 2502.00425) defines it, and names the passage it follows.  Quantization
is not an approximation of something else: the codes ARE the definition, so
the oracle is the algorithm written out step by step.  Where the paper leaves a
choice open the reading taken is stated next to the code.

Precision.  The paper fixes no arithmetic type.  Real-valued reference results
(dense rotation, attention, dequantized outputs) are computed in float64.  The
decisions that produce an integer (activation and weight codes, the static
scales the codes depend on) are taken in float32, the precision the kernels use,
so that both sides round the same number; the float32 fast transform keeps one
canonical butterfly order for the same reason.

Parity pins (tests/test_oracle_*.py) tie every function to something other than
itself: integer identities of the Hadamard matrix, the closed form of the first
transform coefficient (Sec. 3.2, the equation between Eq. 7 and Eq. 9), the
scale formula of Eq. 2 on hand-made arrays, hand-worked rounding and clamping
cases, brute-force integer products, the printed index map of App. A.2 and the
three cases of Eq. 5, and the attention-invariance claim of Sec. 3.1.
No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

TEXT, VISUAL = 0, 1
INT8_MIN, INT8_MAX = -128, 127
INT4_MIN, INT4_MAX = -8, 7


# ----------------------------------------------------------------------------- bf16
def bf16_rne(x):
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32.

    bfloat16 is the upper 16 bits of an IEEE float32, so rounding adds half an
    ulp of the kept part (plus the parity bit) and truncates."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    out = r.astype(np.uint32).view(np.float32).copy()
    out[np.isnan(x)] = np.float32(np.nan)
    return out


# ----------------------------------------------------------------------------- Hadamard
def hadamard_matrix(n: int) -> np.ndarray:
    """Unnormalised Walsh-Hadamard matrix of order n = 2^k with entries +-1.

    App. A.3: H_2 = [[1,1],[1,-1]]/sqrt(2) and H_{2^k} = H_2 (x) H_{2^(k-1)};
    the 1/sqrt(2) factors are left out here (they collect into 1/sqrt(n))."""
    if n < 1 or (n & (n - 1)) != 0:
        raise ValueError("Hadamard order must be a power of two")
    H = np.ones((1, 1), dtype=np.int64)
    H2 = np.array([[1, 1], [1, -1]], dtype=np.int64)
    while H.shape[0] < n:
        H = np.kron(H2, H)
    return H


def rotate_dense(x, n: int) -> np.ndarray:
    """Block-diagonal rotation x . (I_{K/n} (x) H_n / sqrt(n)) as a dense float64 product.

    Sec. 3.2 takes H orthonormal (entries 1/sqrt(n)).  The paper defines H only
    for powers of two; for an input width K that is not one (18944 = 148 x 128)
    the rotation is read as block-diagonal over consecutive blocks of n columns,
    which is still orthogonal, so the computational-invariance argument of
    App. A.14 carries over."""
    x = np.asarray(x, dtype=np.float64)
    K = x.shape[-1]
    if n == 0:
        return x.copy()
    if K % n:
        raise ValueError("K must be a multiple of the rotation block")
    H = hadamard_matrix(n).astype(np.float64) / np.sqrt(np.float64(n))
    blocks = x.reshape(x.shape[:-1] + (K // n, n))
    return (blocks @ H).reshape(x.shape)


def fwht_blocks(x, n: int, dtype=np.float32, normalise: bool = True) -> np.ndarray:
    """Fast Walsh-Hadamard transform of every length-n block of the last axis.

    The fast form of App. A.3's Kronecker recursion: log2(n) butterfly stages
    with strides h = 1, 2, 4, ..., n/2, each replacing the pair (v[i], v[i+h])
    (for i with bit h clear) by (v[i] + v[i+h], v[i] - v[i+h]); afterwards one
    multiplication by 1/sqrt(n) (Sec. 3.2: orthonormal H).  In float32 this is
    the canonical rounding order: every add/sub and the final multiply rounds
    once, the normalisation constant is float32(1/sqrt(n)).  normalise=False
    stops after the butterflies (the full-width Kronecker rotation normalises
    once at its very end)."""
    x = np.asarray(x)
    K = x.shape[-1]
    if n == 0:
        return x.astype(dtype)
    if n < 1 or (n & (n - 1)) != 0 or K % n:
        raise ValueError("rotation block must be a power of two dividing K")
    v = x.astype(dtype).reshape(-1, K // n, n).copy()
    h = 1
    while h < n:
        w = v.reshape(v.shape[0], v.shape[1], n // (2 * h), 2, h)
        a = w[:, :, :, 0, :].copy()
        b = w[:, :, :, 1, :].copy()
        w[:, :, :, 0, :] = a + b
        w[:, :, :, 1, :] = a - b
        h *= 2
    if normalise:
        c = dtype(1.0) / np.sqrt(dtype(n)) if dtype == np.float64 else np.float32(1.0 / np.sqrt(np.float64(n)))
        v = v * c
    return v.reshape(x.shape).astype(dtype)


# ----------------------------------------------------------------------------- modality table
def row_modality(T: int, seg_end, seg_mod) -> np.ndarray:
    """Modality of each row from the segment table (Eq. 3: each contiguous span of
    the sequence carries the scale of its modality).  A row belongs to the first
    segment whose exclusive end exceeds it; rows past the last end are text."""
    out = np.zeros(T, dtype=np.uint8)
    seg_end = np.asarray(seg_end, dtype=np.int64)
    for t in range(T):
        for e, m in zip(seg_end.tolist(), np.asarray(seg_mod).tolist()):
            if t < e:
                out[t] = m
                break
    return out


# ----------------------------------------------------------------------------- scales and quantizers
def static_scale(values, qmax: int = 127) -> np.float32:
    """Eq. 2: s = max|x| / (2^(b-1) - 1), in float32.  An empty or all-zero
    tensor gets s = 1 so that the quantizer stays defined."""
    values = np.asarray(values, dtype=np.float32)
    if values.size == 0:
        return np.float32(1.0)
    m = np.float32(np.max(np.abs(values)))
    if not (m > 0):
        return np.float32(1.0)
    return np.float32(m / np.float32(qmax))


def calibrate_static_scales(x_calib, seg_end, seg_mod, rot_block: int):
    """MSQ calibration (Sec. 3.1, Eq. 3; Algorithm 1 step 6(b)): one static
    per-tensor scale for the visual rows and one for the text rows, each the
    Eq. 2 scale over all calibration values of that modality.  The statistic is
    taken on the numbers the quantizer will see, i.e. after the online rotation
    when there is one (the quantizer sits behind the transform in Fig. 4(a))."""
    x_calib = np.asarray(x_calib, dtype=np.float32)
    r = fwht_blocks(x_calib, rot_block, np.float32)
    mod = row_modality(x_calib.shape[0], seg_end, seg_mod)
    return static_scale(r[mod == VISUAL]), static_scale(r[mod == TEXT])


def quantize_act_int8(r, s_rows) -> np.ndarray:
    """Eq. 2 with z = 0 and b = 8, scale chosen per row by modality (Eq. 3):
    q = clamp(round(r * (1/s)), -128, 127).

    Readings: symmetric (Eq. 2's own scale formula is the symmetric one);
    round-to-nearest with ties to even; the clamp covers the full two's-complement
    range "determined by the bit-width"; the division is done as a multiplication
    by the float32 reciprocal of s, computed once per scale, since that is what a
    static-scale kernel does (quantize_act_int8_divide below is the literal x/s).
    NaN maps to 0 and infinities saturate."""
    r = np.asarray(r, dtype=np.float32)
    s_rows = np.asarray(s_rows, dtype=np.float32).reshape(-1, 1)
    inv = (np.float32(1.0) / s_rows).astype(np.float32)
    y = (r * inv).astype(np.float32)
    with np.errstate(invalid="ignore"):
        q = np.rint(y)
    q = np.where(np.isnan(q), 0.0, q)
    return np.clip(q, INT8_MIN, INT8_MAX).astype(np.int8)


def quantize_act_int8_divide(r, s_rows) -> np.ndarray:
    """Eq. 2 literally, with a true float32 division x / s (informational twin)."""
    r = np.asarray(r, dtype=np.float32)
    s_rows = np.asarray(s_rows, dtype=np.float32).reshape(-1, 1)
    with np.errstate(invalid="ignore"):
        q = np.rint((r / s_rows).astype(np.float32))
    q = np.where(np.isnan(q), 0.0, q)
    return np.clip(q, INT8_MIN, INT8_MAX).astype(np.int8)


def row_scales(T: int, seg_end, seg_mod, s_vis, s_txt) -> np.ndarray:
    mod = row_modality(T, seg_end, seg_mod)
    return np.where(mod == VISUAL, np.float32(s_vis), np.float32(s_txt)).astype(np.float32)


def quantize_weight_int4(w):
    """Per-output-channel symmetric 4-bit round-to-nearest weight quantizer
    (Eq. 2 with b = 4, z = 0; Algorithm 1 outputs per-channel weight scales).
    s_w[n] = max_k |W[n,k]| / 7 (1 for an all-zero row); codes clamp to [-8, 7];
    offline, so the division is the literal one of Eq. 2.  Plain rounding stands
    in for GPTQ, which needs the paper's calibration data."""
    w = np.asarray(w, dtype=np.float32)
    m = np.max(np.abs(w), axis=1).astype(np.float32)
    s = np.where(m > 0, m / np.float32(7.0), np.float32(1.0)).astype(np.float32)
    q = np.rint((w / s[:, None]).astype(np.float32))
    return np.clip(q, INT4_MIN, INT4_MAX).astype(np.int8), s


def pack_w4(q) -> np.ndarray:
    """Two 4-bit two's-complement codes per byte: byte j of row n holds code
    (n, 2j) in its low nibble and code (n, 2j+1) in its high nibble."""
    q = np.asarray(q, dtype=np.int8)
    u = (q.astype(np.int16) & 0xF).astype(np.uint8)
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


def unpack_w4(p) -> np.ndarray:
    p = np.asarray(p, dtype=np.uint8)
    lo = (p & 0xF).astype(np.int16)
    hi = (p >> 4).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty((p.shape[0], p.shape[1] * 2), dtype=np.int8)
    out[:, 0::2] = lo
    out[:, 1::2] = hi
    return out


# ----------------------------------------------------------------------------- GEMM and dequant
def int_gemm(qx, qw) -> np.ndarray:
    """acc[t,n] = sum_k qx[t,k] * qw[n,k] as exact integers.

    The products are formed by a float64 matrix multiplication (a library
    primitive used as one step): every partial sum is an integer far below 2^53
    (|acc| <= 128 * 8 * K), so float64 represents it exactly."""
    qx = np.asarray(qx)
    qw = np.asarray(qw)
    K = qx.shape[1]
    if 128.0 * 128.0 * K >= 2.0 ** 53:
        raise ValueError("K too large for exact float64 accumulation")
    acc = qx.astype(np.float64) @ qw.astype(np.float64).T
    out = acc.astype(np.int64)
    if np.any(np.abs(out) > 2 ** 31 - 1):
        raise OverflowError("int32 accumulator overflow")
    return out.astype(np.int32)


def int_gemm_loops(qx, qw) -> np.ndarray:
    """The same sum as three nested loops over Python integers (tiny shapes only)."""
    T, K = np.shape(qx)
    N = np.shape(qw)[0]
    qx = np.asarray(qx).tolist()
    qw = np.asarray(qw).tolist()
    out = np.zeros((T, N), dtype=np.int64)
    for t in range(T):
        for n in range(N):
            a = 0
            for k in range(K):
                a += qx[t][k] * qw[n][k]
            out[t, n] = a
    return out


def dequant(acc, s_rows, s_w, bias=None, dtype=np.float64) -> np.ndarray:
    """y[t,n] = acc[t,n] * (s_a(t) * s_w[n]) (+ bias[n]): Eq. 2's "multiply the
    integers back by the scale" for both operands of the product at once.
    dtype=float32 reproduces the kernel's rounding order (scale product first)."""
    acc = np.asarray(acc)
    s_rows = np.asarray(s_rows, dtype=np.float32).astype(dtype).reshape(-1, 1)
    s_w = np.asarray(s_w, dtype=np.float32).astype(dtype).reshape(1, -1)
    y = acc.astype(dtype) * (s_rows * s_w).astype(dtype)
    y = y.astype(dtype)
    if bias is not None:
        y = (y + np.asarray(bias, dtype=np.float32).astype(dtype).reshape(1, -1)).astype(dtype)
    return y


def linear_w4a8_msq(x, seg_end, seg_mod, s_vis, s_txt, rot_block, qw, s_w, bias=None):
    """The whole hot path on one activation tile (Sec. 3.1 + Fig. 4(a)):
    rotate -> per-modality static int8 quantize -> integer GEMM against the 4-bit
    weight codes -> dequantize -> bfloat16.  Returns every intermediate."""
    x = np.asarray(x, dtype=np.float32)
    T = x.shape[0]
    r = fwht_blocks(x, rot_block, np.float32)
    s_rows = row_scales(T, seg_end, seg_mod, s_vis, s_txt)
    qx = quantize_act_int8(r, s_rows)
    acc = int_gemm(qx, qw)
    y64 = dequant(acc, s_rows, s_w, bias, np.float64)
    y32 = dequant(acc, s_rows, s_w, bias, np.float32)
    return {"rotated": r, "s_rows": s_rows, "qx": qx, "acc": acc, "y64": y64, "y32": y32,
            "y_bf16": bf16_rne(y32)}


# ----------------------------------------------------------------------------- other bit widths and weight groups
def quantize_weight_sym(w, bits: int = 4, group: int = 0):
    """Eq. 2 with z = 0 for a general weight bit-width b and scale granularity: qmax = 2^(b-1) - 1,
    s = max|w| / qmax over one output channel (group = 0) or over each run of `group` consecutive
    input channels of it (the group-wise W4 of the weight-only comparison, App. A.12: g = 128),
    codes clamp to [-2^(b-1), qmax]; literal division (offline).  W8 is the weight side of the W8A8
    rows of the main results table (Sec. 4.1).
    Returns (codes int8 [N, K], scales float32 [N] or [N, K / group])."""
    w = np.asarray(w, dtype=np.float32)
    N, K = w.shape
    qmax = np.float32(2 ** (bits - 1) - 1)
    if group:
        assert K % group == 0
        blocks = w.reshape(N, K // group, group)
        m = np.max(np.abs(blocks), axis=2).astype(np.float32)
        s = np.where(m > 0, m / qmax, np.float32(1.0)).astype(np.float32)
        q = np.rint((blocks / s[:, :, None]).astype(np.float32)).reshape(N, K)
    else:
        m = np.max(np.abs(w), axis=1).astype(np.float32)
        s = np.where(m > 0, m / qmax, np.float32(1.0)).astype(np.float32)
        q = np.rint((w / s[:, None]).astype(np.float32))
    return np.clip(q, -(2 ** (bits - 1)), 2 ** (bits - 1) - 1).astype(np.int8), s


def quantize_act_sym(r, s_rows, bits: int = 8) -> np.ndarray:
    """quantize_act_int8 for a general activation bit-width: same reciprocal-multiply and
    round-half-even, clamp to [-2^(b-1), 2^(b-1) - 1].  b = 4 is the activation side of the
    W4A4 rows of the main results table (Sec. 4.1); the codes still travel as int8."""
    r = np.asarray(r, dtype=np.float32)
    s_rows = np.asarray(s_rows, dtype=np.float32).reshape(-1, 1)
    inv = (np.float32(1.0) / s_rows).astype(np.float32)
    with np.errstate(invalid="ignore", over="ignore"):
        q = np.rint((r * inv).astype(np.float32))
    q = np.where(np.isnan(q), 0.0, q)
    return np.clip(q, -(2 ** (bits - 1)), 2 ** (bits - 1) - 1).astype(np.int8)


def calibrate_static_scales_bits(x_calib, seg_end, seg_mod, rot_block: int, bits: int = 8):
    """calibrate_static_scales with Eq. 2's denominator 2^(b-1) - 1 for b-bit activations."""
    x_calib = np.asarray(x_calib, dtype=np.float32)
    r = fwht_blocks(x_calib, rot_block, np.float32)
    mod = row_modality(x_calib.shape[0], seg_end, seg_mod)
    qmax = 2 ** (bits - 1) - 1
    return static_scale(r[mod == VISUAL], qmax), static_scale(r[mod == TEXT], qmax)


def int_gemm_grouped(qx, qw, group: int) -> np.ndarray:
    """Partial sums per weight group: acc[t, n, g] = sum over the group's input channels."""
    qx = np.asarray(qx)
    qw = np.asarray(qw)
    T, K = qx.shape
    N = qw.shape[0]
    G = K // group
    out = np.empty((T, N, G), dtype=np.int32)
    for g in range(G):
        out[:, :, g] = int_gemm(qx[:, g * group:(g + 1) * group], qw[:, g * group:(g + 1) * group])
    return out


def dequant_grouped(acc_g, s_rows, s_wg, bias=None, dtype=np.float64) -> np.ndarray:
    """y[t,n] = sum_g acc[t,n,g] * (s_a(t) * s_w[n,g]) (+ bias[n]).  dtype=float32 fixes the rounding
    order: for g = 0, 1, ...: y <- fl(y + fl(float(acc_g) * fl(s_a * s_w[n,g]))), so that one group
    reproduces dequant() bit for bit."""
    acc_g = np.asarray(acc_g)
    T, N, G = acc_g.shape
    s_rows = np.asarray(s_rows, dtype=np.float32).astype(dtype).reshape(-1, 1)
    s_wg = np.asarray(s_wg, dtype=np.float32).astype(dtype).reshape(N, G)
    y = np.zeros((T, N), dtype=dtype)
    for g in range(G):
        c = (s_rows * s_wg[None, :, g]).astype(dtype)
        y = (y + (acc_g[:, :, g].astype(dtype) * c).astype(dtype)).astype(dtype)
    if bias is not None:
        y = (y + np.asarray(bias, dtype=np.float32).astype(dtype).reshape(1, -1)).astype(dtype)
    return y


def linear_wa_sym(x, seg_end, seg_mod, s_vis, s_txt, rot_block, qw, s_w, act_bits: int = 8, group: int = 0,
                  bias=None):
    """linear_w4a8_msq generalised to the neighbouring settings: b-bit static MSQ activations
    (codes from quantize_act_sym), weight codes of any width (the integer product does not care),
    and per-channel (group = 0) or group-wise weight scales."""
    x = np.asarray(x, dtype=np.float32)
    T = x.shape[0]
    r = fwht_blocks(x, rot_block, np.float32)
    s_rows = row_scales(T, seg_end, seg_mod, s_vis, s_txt)
    qx = quantize_act_sym(r, s_rows, act_bits)
    if group:
        acc_g = int_gemm_grouped(qx, qw, group)
        y64 = dequant_grouped(acc_g, s_rows, s_w, bias, np.float64)
        y32 = dequant_grouped(acc_g, s_rows, s_w, bias, np.float32)
        return {"rotated": r, "s_rows": s_rows, "qx": qx, "acc_g": acc_g, "y64": y64, "y32": y32,
                "y_bf16": bf16_rne(y32)}
    acc = int_gemm(qx, qw)
    y64 = dequant(acc, s_rows, s_w, bias, np.float64)
    y32 = dequant(acc, s_rows, s_w, bias, np.float32)
    return {"rotated": r, "s_rows": s_rows, "qx": qx, "acc": acc, "y64": y64, "y32": y32,
            "y_bf16": bf16_rne(y32)}


# ----------------------------------------------------------------------------- full-width rotation for K = m * 2^k
def _gf27_tables():
    """GF(27) = GF(3)[x] / (x^3 + 2x + 1): elements are base-3 digit triples c0 + 3 c1 + 9 c2."""
    def mul(a, b):
        pa = [a % 3, (a // 3) % 3, a // 9]
        pb = [b % 3, (b // 3) % 3, b // 9]
        prod = [0] * 5
        for i in range(3):
            for j in range(3):
                prod[i + j] = (prod[i + j] + pa[i] * pb[j]) % 3
        for d in (4, 3):                       # x^3 = -2x - 1 = x + 2 (mod 3)
            c = prod[d]
            prod[d] = 0
            prod[d - 2] = (prod[d - 2] + c) % 3
            prod[d - 3] = (prod[d - 3] + 2 * c) % 3
        return prod[0] + 3 * prod[1] + 9 * prod[2]

    def sub(a, b):
        return sum((((a // 3 ** d) % 3 - (b // 3 ** d) % 3) % 3) * 3 ** d for d in range(3))

    return mul, sub


def _quadratic_character(q: int):
    """chi(a) for the field of q elements (q an odd prime, or 27): +1 for non-zero squares, -1 for
    non-squares, 0 for 0, together with the field's subtraction."""
    if q == 27:
        mul, sub = _gf27_tables()
        squares = {mul(a, a) for a in range(1, 27)}
        assert len(squares) == 13
        chi = [0] + [1 if a in squares else -1 for a in range(1, 27)]
        return chi, sub
    assert q > 2 and all(q % d for d in range(2, int(q ** 0.5) + 1)), "q must be an odd prime (or 27)"
    chi = [0] + [1 if pow(a, (q - 1) // 2, q) == 1 else -1 for a in range(1, q)]
    return chi, lambda a, b: (a - b) % q


def paley_hadamard(m: int) -> np.ndarray:
    """A Hadamard matrix of order m (entries +-1, H H^T = m I) by Paley's constructions, for the
    orders a full-width online rotation of K = m * 2^k needs when K is not a power of two (the paper
    defines only H_{2^n}, App. A.3; the Kronecker form H_m (x) H_{2^k} is the usual completion):
      type I,  m = q + 1 with q = 3 (mod 4):  H = I + S,  S = [[0, 1^T], [-1, Q]],  Q[a,b] = chi(a - b);
      type II, m = 2 (q + 1) with q = 1 (mod 4):  H = [[C + I, C - I], [C - I, -C - I]],
               C = [[0, 1^T], [1, Q]].
    q is an odd prime or 27.  m = 28 (K = 14336 = 28 * 512) is type I over GF(27); m = 148
    (K = 18944 = 148 * 128) is type II with q = 73."""
    if m in (1, 2):
        return hadamard_matrix(m)
    for kind, q in ((1, m - 1), (2, m // 2 - 1)):
        if kind == 2 and m % 2:
            continue
        is_field = q == 27 or (q > 2 and all(q % d for d in range(2, int(q ** 0.5) + 1)))
        if not is_field or q % 4 != (3 if kind == 1 else 1):
            continue
        chi, sub = _quadratic_character(q)
        Q = np.array([[chi[sub(a, b)] for b in range(q)] for a in range(q)], dtype=np.int64)
        if kind == 1:
            S = np.zeros((q + 1, q + 1), dtype=np.int64)
            S[0, 1:] = 1
            S[1:, 0] = -1
            S[1:, 1:] = Q
            return (np.eye(q + 1, dtype=np.int64) + S).astype(np.int64)
        C = np.zeros((q + 1, q + 1), dtype=np.int64)
        C[0, 1:] = 1
        C[1:, 0] = 1
        C[1:, 1:] = Q
        I = np.eye(q + 1, dtype=np.int64)
        return np.block([[C + I, C - I], [C - I, -C - I]]).astype(np.int64)
    raise ValueError("no Paley construction for order %d" % m)


def kron_rotate_dense(x, h_m, n2: int) -> np.ndarray:
    """y = x (H_m (x) H_n2) / sqrt(K) in float64, K = m * n2, with the input channels of a row read as
    an m x n2 array X (channel = i * n2 + j): Y = H_m^T X H_n2 / sqrt(K)."""
    x = np.asarray(x, dtype=np.float64)
    h_m = np.asarray(h_m, dtype=np.float64)
    m = h_m.shape[0]
    T, K = x.shape
    assert K == m * n2
    X = x.reshape(T, m, n2)
    U = X @ hadamard_matrix(n2).astype(np.float64)
    Y = np.einsum("ia,tij->taj", h_m, U)
    return (Y / np.sqrt(np.float64(K))).reshape(T, K)


def kron_rotate_f32(x, h_m, n2: int) -> np.ndarray:
    """The same in float32 with a fixed order: the un-normalised butterflies of fwht_blocks on every
    run of n2 channels, then for every output (a, j) the sum over i = 0, 1, ... of +-U[i, j] added
    one at a time, then one multiply by float32(1 / sqrt(K))."""
    x = np.asarray(x, dtype=np.float32)
    h_m = np.asarray(h_m)
    m = h_m.shape[0]
    T, K = x.shape
    assert K == m * n2
    U = (fwht_blocks(x, n2, np.float32, normalise=False) if n2 > 1 else x).reshape(T, m, n2)
    Y = np.zeros((T, m, n2), dtype=np.float32)
    for i in range(m):
        Y = (Y + h_m[i].astype(np.float32)[None, :, None] * U[:, i, None, :]).astype(np.float32)
    c = np.float32(1.0 / np.sqrt(np.float64(K)))
    return (Y * c).astype(np.float32).reshape(T, K)


# ----------------------------------------------------------------------------- AIFS
def aifs_perm(is_visual, is_pad=None) -> np.ndarray:
    """AIFS order (Sec. 3.1; App. A.2: AIFS(1..L) = (m..n, 1..m-1, n+1..L)):
    all visual tokens first, in their original order, then all text tokens in
    their original order.  Generalised to any number of visual spans (the
    paper's own prompts interleave three images).  Left-pad tokens of a batched
    sequence travel with the visual block (App. A.4)."""
    is_visual = np.asarray(is_visual).astype(bool)
    first = is_visual.copy()
    if is_pad is not None:
        first |= np.asarray(is_pad).astype(bool)
    idx = np.arange(is_visual.shape[0], dtype=np.int32)
    return np.concatenate([idx[first], idx[~first]]).astype(np.int32)


def inverse_perm(perm) -> np.ndarray:
    perm = np.asarray(perm)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.shape[0], dtype=perm.dtype)
    return inv


def aifs_gather(x, perm) -> np.ndarray:
    """E^u[i] = E[perm[i]]."""
    return np.asarray(x)[np.asarray(perm)]


def aifs_scatter(x_u, perm) -> np.ndarray:
    """Inverse of aifs_gather: out[perm[i]] = x_u[i]."""
    x_u = np.asarray(x_u)
    out = np.empty_like(x_u)
    out[np.asarray(perm)] = x_u
    return out


def remap_positions(perm, pos_ids=None) -> np.ndarray:
    """App. A.2: the rotary embedding of a moved token uses its ORIGINAL index."""
    perm = np.asarray(perm)
    if pos_ids is None:
        pos_ids = np.arange(perm.shape[0], dtype=np.int32)
    return np.asarray(pos_ids)[perm].astype(np.int32)


def causal_mask(L: int) -> np.ndarray:
    """Eq. 4 as a boolean "may attend" matrix: allowed(i,j) <=> j <= i."""
    i = np.arange(L)[:, None]
    j = np.arange(L)[None, :]
    return j <= i


def unified_mask(perm, is_pad=None) -> np.ndarray:
    """The unified causal mask M^u of Eq. 5 for an arbitrary interleaving:
    row i (original token perm[i]) may attend column j (original token perm[j])
    iff perm[j] <= perm[i], i.e. iff it could in the original order (Eq. 4).
    Padded tokens are attended by nobody (App. A.4); a pad row keeps its own
    diagonal so its (discarded) softmax stays defined."""
    perm = np.asarray(perm, dtype=np.int64)
    allowed = perm[None, :] <= perm[:, None]
    if is_pad is not None:
        pad_u = np.asarray(is_pad).astype(bool)[perm]
        allowed = allowed & ~pad_u[None, :]
        allowed = allowed | (np.eye(perm.shape[0], dtype=bool) & pad_u[:, None])
    return allowed


def unified_mask_single_span(m: int, n: int, L: int) -> np.ndarray:
    """Eq. 5 case by case for ONE visual span at 1-based original positions m..n.

    With N_v = n - m + 1 visual tokens first, then the m-1 leading text tokens,
    then the trailing text (1-based unified indices i, j):
      visual row   (i <= N_v):        j <= i, or j among the leading text (N_v < j <= n);
      leading text (N_v < i <= n):    N_v < j <= i;
      trailing     (i > n):           j <= i.
    (The printed equation writes n - m for the visual count; with inclusive
    bounds m..n the count is n - m + 1, which is the value used here.)"""
    nv = n - m + 1
    allowed = np.zeros((L, L), dtype=bool)
    for i in range(1, L + 1):
        for j in range(1, L + 1):
            if i <= nv:
                ok = (j <= i) or (nv < j <= n)
            elif i <= n:
                ok = nv < j <= i
            else:
                ok = j <= i
            allowed[i - 1, j - 1] = ok
    return allowed


def segments_after_aifs(perm, is_visual, is_pad=None):
    """Segment table of the reordered rows: [visual (and pad) block][text block]."""
    first = np.asarray(is_visual).astype(bool)
    if is_pad is not None:
        first = first | np.asarray(is_pad).astype(bool)
    n_first = int(first.sum())
    L = int(np.asarray(perm).shape[0])
    return np.array([n_first, L], dtype=np.int32), np.array([VISUAL, TEXT], dtype=np.uint8)


# ----------------------------------------------------------------------------- attention checker
def rope(x, pos_ids, base: float = 10000.0) -> np.ndarray:
    """Rotary position embedding of App. A.2: consecutive channel pairs
    (2i, 2i+1) are rotated by angle pos * theta_i, theta_i = base^(-2i/D),
    i = 0..D/2-1.  float64; x is [L, D]."""
    x = np.asarray(x, dtype=np.float64)
    L, D = x.shape
    theta = base ** (-2.0 * np.arange(D // 2, dtype=np.float64) / D)
    ang = np.asarray(pos_ids, dtype=np.float64)[:, None] * theta[None, :]
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    out[:, 0::2] = x[:, 0::2] * c - x[:, 1::2] * s
    out[:, 1::2] = x[:, 0::2] * s + x[:, 1::2] * c
    return out


def attention(q, k, v, allowed) -> np.ndarray:
    """Softmax(Q K^T / sqrt(D) + M) V with M = 0 where allowed, -inf elsewhere
    (Eq. 4 / Eq. 5), single head, float64."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    s = q @ k.T / np.sqrt(np.float64(q.shape[1]))
    s = np.where(allowed, s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v


# ----------------------------------------------------------------------------- helpers for neighbouring steps
def rotate_weight_input_dim(w, n: int) -> np.ndarray:
    """Offline counterpart of the online rotation: W' = W . blockdiag(H_n/sqrt(n))
    along the input dimension, float64, so that (x H)(W H)^T = x W^T (App. A.14)."""
    return rotate_dense(np.asarray(w, dtype=np.float64), n)


# ----------------------------------------------------------------------------- RMS (Sec. 3.2)
def rms_detect(w, n: int) -> np.ndarray:
    """Eq. 9 per output channel and rotation block: the first row of the rotated weight,
    sqrt(n) * mean(w) over the block's n input channels (the equation between Eq. 7 and Eq. 9),
    exceeds the block's largest original weight -- a channel-mean outlier created by the
    online transform.  w is the UNROTATED weight [N, K]; returns bool [N, K / n].
    (The paper's W is [in, out]; its column j is our row.)"""
    w = np.asarray(w, dtype=np.float64)
    N, K = w.shape
    assert K % n == 0
    blocks = w.reshape(N, K // n, n)
    return np.sqrt(float(n)) * blocks.mean(axis=2) > blocks.max(axis=2)


def rms_split(w_rot, n: int):
    """Rotation Magnitude Suppression, steps 1 and 2 (Sec. 3.2): the first input channel of
    every rotation block of the ROTATED weight [N, K] is split off (it is handled by a
    separate GEMV) and zeroed in the main matrix so that it is not counted twice.
    Returns (w_main [N, K], w_side [N, K / n])."""
    w_rot = np.asarray(w_rot)
    w_main = w_rot.copy()
    w_side = w_rot[:, ::n].copy()
    w_main[:, ::n] = 0
    return w_main, w_side


def linear_w4a8_msq_rms(x, seg_end, seg_mod, s_vis, s_txt, rot_block, qw_main, s_w_main, qw_side, s_w_side,
                        bias=None):
    """The down-projection with RMS (Sec. 3.2, step 3: add the GEMV's partial output back):
      y = Q(x~) . Q(HW with the split rows zeroed)^T  +  Q(x~[:, first channel of each block]) . Q(split rows)^T.
    Both terms use the same int8 activation codes; each weight part has its own per-channel
    int4 scale.  float32 twin: each term is float(acc) * (s_a * s_w) with the scale product
    formed first, the terms are added, then the bias."""
    x = np.asarray(x, dtype=np.float32)
    T = x.shape[0]
    r = fwht_blocks(x, rot_block, np.float32)
    s_rows = row_scales(T, seg_end, seg_mod, s_vis, s_txt)
    qx = quantize_act_int8(r, s_rows)
    acc_main = int_gemm(qx, qw_main)
    acc_side = int_gemm(qx[:, ::rot_block], qw_side)
    y64 = dequant(acc_main, s_rows, s_w_main, None, np.float64) + dequant(acc_side, s_rows, s_w_side, None, np.float64)
    y32 = (dequant(acc_main, s_rows, s_w_main, None, np.float32)
           + dequant(acc_side, s_rows, s_w_side, None, np.float32)).astype(np.float32)
    if bias is not None:
        y64 = y64 + np.asarray(bias, dtype=np.float64).reshape(1, -1)
        y32 = (y32 + np.asarray(bias, dtype=np.float32).reshape(1, -1)).astype(np.float32)
    return {"qx": qx, "s_rows": s_rows, "acc_main": acc_main, "acc_side": acc_side, "y64": y64, "y32": y32,
            "y_bf16": bf16_rne(y32)}


def quantize_act_int8_dynamic(r):
    """Per-token dynamic A8 (the baseline MSQ replaces, Sec. 1): every row gets
    its own Eq. 2 scale from its own abs-max."""
    r = np.asarray(r, dtype=np.float32)
    s = np.array([static_scale(row) for row in r], dtype=np.float32)
    return quantize_act_int8(r, s), s


def linear_w4a8_dynamic(x, rot_block, qw, s_w, bias=None):
    """The comparison linear with per-token dynamic activation scales (Sec. 1, Sec. 4.3: the
    scheme whose per-token scale computation MSQ + AIFS remove): rotate, take each row's own
    Eq. 2 scale from the rotated row, quantize with it, integer GEMM, dequantize with that
    row's scale.  Same rounding conventions as linear_w4a8_msq."""
    x = np.asarray(x, dtype=np.float32)
    r = fwht_blocks(x, rot_block, np.float32)
    qx, s_rows = quantize_act_int8_dynamic(r)
    acc = int_gemm(qx, qw)
    y64 = dequant(acc, s_rows, s_w, bias, np.float64)
    y32 = dequant(acc, s_rows, s_w, bias, np.float32)
    return {"rotated": r, "s_rows": s_rows, "qx": qx, "acc": acc, "y64": y64, "y32": y32,
            "y_bf16": bf16_rne(y32)}


# ----------------------------------------------------------------------------- glue of a decoder block (checker only)
def rmsnorm(x, gain, eps: float = 1e-6) -> np.ndarray:
    """RMSNorm (App. A.14: x / sqrt(||x||^2 / d + eps)), times the per-channel gain; float64."""
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gain, dtype=np.float64)


def swiglu(gate, up) -> np.ndarray:
    """SiLU(gate) * up, the activation in front of the down-projection; float64."""
    gate = np.asarray(gate, dtype=np.float64)
    return gate / (1.0 + np.exp(-gate)) * np.asarray(up, dtype=np.float64)


def gqa_attention(q, k, v, allowed, n_q_heads: int, n_kv_heads: int) -> np.ndarray:
    """Grouped-query attention: q [L, n_q_heads*D], k, v [L, n_kv_heads*D]; query head h reads
    key/value head h // (n_q_heads / n_kv_heads); every head is attention() above."""
    q = np.asarray(q, dtype=np.float64)
    L = q.shape[0]
    D = q.shape[1] // n_q_heads
    group = n_q_heads // n_kv_heads
    out = np.empty_like(q)
    for h in range(n_q_heads):
        g = h // group
        out[:, h * D:(h + 1) * D] = attention(q[:, h * D:(h + 1) * D], np.asarray(k)[:, g * D:(g + 1) * D],
                                              np.asarray(v)[:, g * D:(g + 1) * D], allowed)
    return out
