"""CPU oracle for the W4A8-dINT linear layer: numpy front end of w4a8_oracle.c.

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the bench's CPU-baseline
leg compare the CUDA library against these functions; the product never calls
them.  The arithmetic lives in w4a8_oracle.c (plain C, one rounded binary32
operation per written operation); this module only marshals numpy arrays.

Paper passages: dINT quantize / dequantize are Eq. 5 / Eq. 6 (Section 4.2);
the operand scaling is Eq. 1 (Section 3.2); the quantizer granularities
(token-wise activations, output-channel-wise weights, Min-Max asymmetric) are
Appendix A.1 "Quantization Settings".
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w4a8_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

# No value-changing optimisation: no fast-math, no FMA contraction.
CFLAGS = ["-O2", "-fPIC", "-shared", "-std=c11", "-ffp-contract=off",
          "-fno-fast-math", "-fopenmp"]


def build(force: bool = False) -> str:
    """Compile w4a8_oracle.c to liboracle.so (gcc) when missing or stale."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < os.path.getmtime(_SRC))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_half_to_float.restype = ctypes.c_float
        _lib.oracle_half_to_float.argtypes = [ctypes.c_uint16]
        _lib.oracle_float_to_bf16.restype = ctypes.c_uint16
        _lib.oracle_float_to_bf16.argtypes = [ctypes.c_float]
        _lib.oracle_dint_p.restype = ctypes.c_int
        _lib.oracle_dint_p.argtypes = [ctypes.c_int]
        _lib.oracle_dint_quantize.restype = ctypes.c_int
        _lib.oracle_dint_quantize.argtypes = [ctypes.c_float, ctypes.c_float,
                                              ctypes.c_int, ctypes.c_int]
        _lib.oracle_dint_dequantize.restype = ctypes.c_float
        _lib.oracle_dint_dequantize.argtypes = [ctypes.c_int, ctypes.c_float,
                                                ctypes.c_int, ctypes.c_int]
        _lib.oracle_get_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


def set_threads(n: int) -> None:
    lib().oracle_set_threads(ctypes.c_int(n))


def get_threads() -> int:
    return int(lib().oracle_get_threads())


# ---------------------------------------------------------------------------
# scalar format routines (Eq. 5, Eq. 6)
# ---------------------------------------------------------------------------

def dint_p(b: int = 4) -> int:
    """Number of uniform steps p = 2^b - 3 (Section 4.2)."""
    return int(lib().oracle_dint_p(b))


def dint_quantize(x: float, s: float, z: int, b: int = 4) -> int:
    """Eq. 5: real value -> dINT code (0..p integer levels, p+1 = c1, p+2 = c2)."""
    return int(lib().oracle_dint_quantize(np.float32(x), np.float32(s), z, b))


def dint_dequantize(code: int, s: float, z: int, b: int = 4) -> float:
    """Eq. 6: dINT code -> real value (binary32)."""
    return float(lib().oracle_dint_dequantize(code, np.float32(s), z, b))


def dint_table2(z: int, b: int = 4) -> np.ndarray:
    """Eq. 6 in units of s/2: 2(code - z) for integer levels, +1 / -1 for c1 / c2."""
    t = np.zeros(1 << b, dtype=np.int8)
    lib().oracle_dint_table2(ctypes.c_int(z), ctypes.c_int(b), _p(t))
    return t


def half_to_float(bits: int) -> float:
    return float(lib().oracle_half_to_float(bits))


def float_to_bf16(f: float) -> int:
    return int(lib().oracle_float_to_bf16(np.float32(f)))


# ---------------------------------------------------------------------------
# the three calls of the path, on host arrays
# ---------------------------------------------------------------------------

def pack_weights(W: np.ndarray, s_in: np.ndarray | None = None, group: int = 0,
                 clip: float = 1.0):
    """Q(W diag(s)) of Eq. 1 in dINT4.  W is [N, K] float16.

    Returns (codes [N, K/2] uint8, scales [G, N] float32, zeros [G, N] uint8).
    """
    W = _c(W, np.float16)
    N, K = W.shape
    if K % 2 or (group and K % group):
        raise ValueError("K must be even and a multiple of the group size")
    G = K // group if group else 1
    if s_in is not None:
        s_in = _c(s_in, np.float32)
        assert s_in.shape == (K,)
    codes = np.empty((N, K // 2), dtype=np.uint8)
    scales = np.empty((G, N), dtype=np.float32)
    zeros = np.empty((G, N), dtype=np.uint8)
    lib().oracle_pack_weights(_p(W.view(np.uint16)), _p(s_in) if s_in is not None else None,
                              ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group),
                              ctypes.c_float(clip), _p(codes), _p(scales), _p(zeros))
    return codes, scales, zeros


def quantize_act(X: np.ndarray, inv_s_in: np.ndarray | None = None):
    """Q(diag(s)^-1 X) of Eq. 1, token-wise INT8.  X is [M, K] float16.

    Returns (Xq [M, K] int8, tok_scale [M] float32).
    """
    X = _c(X, np.float16)
    M, K = X.shape
    if inv_s_in is not None:
        inv_s_in = _c(inv_s_in, np.float32)
        assert inv_s_in.shape == (K,)
    Xq = np.empty((M, K), dtype=np.int8)
    tok = np.empty((M,), dtype=np.float32)
    lib().oracle_quantize_act(_p(X.view(np.uint16)),
                              _p(inv_s_in) if inv_s_in is not None else None,
                              ctypes.c_int(M), ctypes.c_int(K), _p(Xq), _p(tok))
    return Xq, tok


def norm_quantize_act(X: np.ndarray, weight: np.ndarray, bias: np.ndarray | None = None,
                      kind: str = "rms", eps: float = 1e-5):
    """Token-wise INT8 quantizer behind an RMSNorm ("rms") or LayerNorm ("layer") whose weight
    and bias carry the reciprocal Eq. 1 scale (Fig. 1(a), Section 3.1).  X is [M, K] float16.

    Returns (Xq [M, K] int8, tok_scale [M] float32).
    """
    X = _c(X, np.float16)
    M, K = X.shape
    weight = _c(weight, np.float32)
    assert weight.shape == (K,)
    if bias is not None:
        bias = _c(bias, np.float32)
        assert bias.shape == (K,)
    Xq = np.empty((M, K), dtype=np.int8)
    tok = np.empty((M,), dtype=np.float32)
    lib().oracle_norm_quantize_act(_p(X.view(np.uint16)), _p(weight),
                                   _p(bias) if bias is not None else None,
                                   ctypes.c_int({"rms": 0, "layer": 1}[kind]), ctypes.c_float(eps),
                                   ctypes.c_int(M), ctypes.c_int(K), _p(Xq), _p(tok))
    return Xq, tok


def _shape(Xq, codes, zeros, group):
    M, K = Xq.shape
    N = codes.shape[0]
    assert codes.shape == (N, K // 2)
    G = K // group if group else 1
    assert zeros.shape == (G, N)
    return M, N, K, G


def linear_acc(Xq, codes, zeros, group: int = 0, wide: bool = False) -> np.ndarray:
    """Integer accumulators [G, M, N]; int64 when `wide`, else int32."""
    Xq = _c(Xq, np.int8)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    M, N, K, G = _shape(Xq, codes, zeros, group)
    acc = np.empty((G, M, N), dtype=np.int64 if wide else np.int32)
    fn = lib().oracle_linear_acc_i64 if wide else lib().oracle_linear_acc_i32
    fn(_p(Xq), _p(codes), _p(zeros), ctypes.c_int(M), ctypes.c_int(N),
       ctypes.c_int(K), ctypes.c_int(group), _p(acc))
    return acc


def linear(Xq, tok_scale, codes, scales, zeros, bias=None, group: int = 0) -> np.ndarray:
    """BF16 output bits [M, N] (uint16) of the quantized linear layer."""
    Xq = _c(Xq, np.int8)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    tok_scale = _c(tok_scale, np.float32)
    M, N, K, G = _shape(Xq, codes, zeros, group)
    if bias is not None:
        bias = _c(bias, np.float32)
    Y = np.empty((M, N), dtype=np.uint16)
    lib().oracle_linear(_p(Xq), _p(tok_scale), _p(codes), _p(scales), _p(zeros),
                        _p(bias) if bias is not None else None, ctypes.c_int(M),
                        ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group), _p(Y))
    return Y


def linear_f64(Xq, tok_scale, codes, scales, zeros, bias=None, group: int = 0) -> np.ndarray:
    """The same output in binary64, not rounded to BF16."""
    Xq = _c(Xq, np.int8)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    tok_scale = _c(tok_scale, np.float32)
    M, N, K, G = _shape(Xq, codes, zeros, group)
    if bias is not None:
        bias = _c(bias, np.float32)
    Y = np.empty((M, N), dtype=np.float64)
    lib().oracle_linear_f64(_p(Xq), _p(tok_scale), _p(codes), _p(scales), _p(zeros),
                            _p(bias) if bias is not None else None, ctypes.c_int(M),
                            ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group), _p(Y))
    return Y


def quantize_act_asym(X: np.ndarray, inv_s_in: np.ndarray | None = None):
    """Asymmetric token-wise Min-Max activation quantizer (App. A.1).  X is [M, K] float16.

    Returns (Q [M, K] uint8, tok_scale [M] float32, tok_zero [M] int32) with
    x' ~ tok_scale * (Q - tok_zero).
    """
    X = _c(X, np.float16)
    M, K = X.shape
    if inv_s_in is not None:
        inv_s_in = _c(inv_s_in, np.float32)
        assert inv_s_in.shape == (K,)
    Q = np.empty((M, K), dtype=np.uint8)
    tok = np.empty((M,), dtype=np.float32)
    zx = np.empty((M,), dtype=np.int32)
    lib().oracle_quantize_act_asym(_p(X.view(np.uint16)),
                                   _p(inv_s_in) if inv_s_in is not None else None,
                                   ctypes.c_int(M), ctypes.c_int(K), _p(Q), _p(tok), _p(zx))
    return Q, tok, zx


def linear_asym_acc(Q, tok_zero, codes, zeros) -> np.ndarray:
    """int64 sums [M, N] of (Q - tok_zero) times the doubled weight levels; per-channel weights."""
    Q = _c(Q, np.uint8)
    tok_zero = _c(tok_zero, np.int32)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    M, K = Q.shape
    N = codes.shape[0]
    assert codes.shape == (N, K // 2) and zeros.shape == (1, N) and tok_zero.shape == (M,)
    acc = np.empty((M, N), dtype=np.int64)
    lib().oracle_linear_asym_acc_i64(_p(Q), _p(tok_zero), _p(codes), _p(zeros), ctypes.c_int(M),
                                     ctypes.c_int(N), ctypes.c_int(K), _p(acc))
    return acc


def linear_asym(Q, tok_scale, tok_zero, codes, scales, zeros, bias=None, wide: bool = False):
    """BF16 output bits [M, N] of the layer with asymmetric activations; with `wide` also the
    unrounded binary64 values."""
    Q = _c(Q, np.uint8)
    tok_scale = _c(tok_scale, np.float32)
    tok_zero = _c(tok_zero, np.int32)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    M, K = Q.shape
    N = codes.shape[0]
    assert codes.shape == (N, K // 2) and zeros.shape == (1, N) and scales.shape == (1, N)
    if bias is not None:
        bias = _c(bias, np.float32)
    Y = np.empty((M, N), dtype=np.uint16)
    W = np.empty((M, N), dtype=np.float64) if wide else None
    lib().oracle_linear_asym(_p(Q), _p(tok_scale), _p(tok_zero), _p(codes), _p(scales), _p(zeros),
                             _p(bias) if bias is not None else None, ctypes.c_int(M),
                             ctypes.c_int(N), ctypes.c_int(K), _p(Y),
                             _p(W) if wide else None)
    return (Y, W) if wide else Y


def linear_asym_group(Q, tok_scale, tok_zero, codes, scales, zeros, bias, group: int):
    """Asymmetric activations with group-wise weight steps: (acc int64 [G, M, N], Y BF16 bits
    [M, N], Y binary64 [M, N])."""
    Q = _c(Q, np.uint8)
    tok_scale = _c(tok_scale, np.float32)
    tok_zero = _c(tok_zero, np.int32)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    M, K = Q.shape
    N = codes.shape[0]
    G = K // group
    assert codes.shape == (N, K // 2) and zeros.shape == (G, N) and scales.shape == (G, N)
    if bias is not None:
        bias = _c(bias, np.float32)
    acc = np.empty((G, M, N), dtype=np.int64)
    Y = np.empty((M, N), dtype=np.uint16)
    wide = np.empty((M, N), dtype=np.float64)
    lib().oracle_linear_asym_group(_p(Q), _p(tok_scale), _p(tok_zero), _p(codes), _p(scales), _p(zeros),
                                   _p(bias) if bias is not None else None, ctypes.c_int(M),
                                   ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group), _p(acc),
                                   _p(Y), _p(wide))
    return acc, Y, wide


# ---- special value s / 2^shift (App. A.5): shift = 1 is Eq. 5 / Eq. 6 --------------------

def dint_quantize_fmt(x: float, s: float, z: int, shift: int, b: int = 4) -> int:
    fn = lib().oracle_dint_quantize_fmt
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_int]
    return int(fn(x, s, z, b, shift))


def dint_dequantize_fmt(code: int, s: float, z: int, shift: int, b: int = 4) -> float:
    fn = lib().oracle_dint_dequantize_fmt
    fn.restype = ctypes.c_float
    fn.argtypes = [ctypes.c_int, ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_int]
    return float(fn(code, s, z, b, shift))


def dint_table_fmt(z: int, shift: int, b: int = 4) -> np.ndarray:
    t = np.zeros(1 << b, dtype=np.int8)
    lib().oracle_dint_table_fmt(ctypes.c_int(z), ctypes.c_int(b), ctypes.c_int(shift), _p(t))
    return t


def pack_weights_fmt(W, s_in, group: int, shift: int, clip: float = 1.0):
    """pack_weights with the special value step / 2^shift."""
    W = _c(W, np.float16)
    N, K = W.shape
    if s_in is not None:
        s_in = _c(s_in, np.float32)
    G = K // group if group else 1
    codes = np.empty((N, K // 2), dtype=np.uint8)
    scales = np.empty((G, N), dtype=np.float32)
    zeros = np.empty((G, N), dtype=np.uint8)
    lib().oracle_pack_weights_fmt(_p(W.view(np.uint16)), _p(s_in) if s_in is not None else None,
                                  ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group),
                                  ctypes.c_float(clip), ctypes.c_int(shift), _p(codes), _p(scales),
                                  _p(zeros))
    return codes, scales, zeros


def linear_fmt(Xq, tok_scale, codes, scales, zeros, bias, group: int, shift: int):
    """(acc int64 [G, M, N], Y bf16 bits [M, N], Y binary64 [M, N]) with levels in units of
    step / 2^shift."""
    Xq = _c(Xq, np.int8)
    tok_scale = _c(tok_scale, np.float32)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    M, N, K, G = _shape(Xq, codes, zeros, group)
    if bias is not None:
        bias = _c(bias, np.float32)
    acc = np.empty((G, M, N), dtype=np.int64)
    Y = np.empty((M, N), dtype=np.uint16)
    wide = np.empty((M, N), dtype=np.float64)
    lib().oracle_linear_fmt(_p(Xq), _p(tok_scale), _p(codes), _p(scales), _p(zeros),
                            _p(bias) if bias is not None else None, ctypes.c_int(M),
                            ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group),
                            ctypes.c_int(shift), _p(acc), _p(Y), _p(wide))
    return acc, Y, wide


def pack_weights_bits(W, s_in, group: int, bits: int, shift: int = 1, clip: float = 1.0):
    """pack_weights for the b-bit format (b = 3: integer codes 0..5, code 6 = +c, code 7 = -c),
    special value step / 2^shift.  Codes come two per byte whatever the width."""
    W = _c(W, np.float16)
    N, K = W.shape
    if s_in is not None:
        s_in = _c(s_in, np.float32)
    G = K // group if group else 1
    codes = np.empty((N, K // 2), dtype=np.uint8)
    scales = np.empty((G, N), dtype=np.float32)
    zeros = np.empty((G, N), dtype=np.uint8)
    lib().oracle_pack_weights_bits(_p(W.view(np.uint16)), _p(s_in) if s_in is not None else None,
                                   ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group),
                                   ctypes.c_float(clip), ctypes.c_int(bits), ctypes.c_int(shift),
                                   _p(codes), _p(scales), _p(zeros))
    return codes, scales, zeros


def linear_bits(Xq, tok_scale, codes, scales, zeros, bias, group: int, bits: int, shift: int = 1):
    """(acc int64 [G, M, N], Y bf16 bits [M, N], Y binary64 [M, N]) for b-bit codes."""
    Xq = _c(Xq, np.int8)
    tok_scale = _c(tok_scale, np.float32)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    M, N, K, G = _shape(Xq, codes, zeros, group)
    if bias is not None:
        bias = _c(bias, np.float32)
    acc = np.empty((G, M, N), dtype=np.int64)
    Y = np.empty((M, N), dtype=np.uint16)
    wide = np.empty((M, N), dtype=np.float64)
    lib().oracle_linear_bits(_p(Xq), _p(tok_scale), _p(codes), _p(scales), _p(zeros),
                             _p(bias) if bias is not None else None, ctypes.c_int(M),
                             ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group),
                             ctypes.c_int(bits), ctypes.c_int(shift), _p(acc), _p(Y), _p(wide))
    return acc, Y, wide


def linear_swiglu(Xq, tok_scale, codes, scales, zeros, bias=None, group: int = 0):
    """Gate / up projections (rows interleaved: 2 i gate, 2 i + 1 up) and h = silu(g) * u.
    Returns (H binary64 [M, F], the layer's FP32 values [M, 2 F])."""
    Xq = _c(Xq, np.int8)
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.uint8)
    scales = _c(scales, np.float32)
    tok_scale = _c(tok_scale, np.float32)
    M, N, K, G = _shape(Xq, codes, zeros, group)
    assert N % 2 == 0
    if bias is not None:
        bias = _c(bias, np.float32)
    H = np.empty((M, N // 2), dtype=np.float64)
    T = np.empty((M, N), dtype=np.float32)
    lib().oracle_linear_swiglu(_p(Xq), _p(tok_scale), _p(codes), _p(scales), _p(zeros),
                               _p(bias) if bias is not None else None, ctypes.c_int(M),
                               ctypes.c_int(N // 2), ctypes.c_int(K), ctypes.c_int(group), _p(H), _p(T))
    return H, T


def pack_value(V: np.ndarray, clip: float = 1.0):
    """Channel-wise dINT4 quantization of the attention values (Appendix A.1, "W4A8V4"):
    V is [S, H, D] float16; a channel is one (h, d), its Min-Max range is taken over the S
    positions (the dimension the attention map sums over).  Returns (codes [H*D, S/2],
    scales [1, H*D], zeros [1, H*D]) as pack_weights does for the matrix V^T."""
    V = _c(V, np.float16)
    S, H, D = V.shape
    return pack_weights(np.ascontiguousarray(V.reshape(S, H * D).T), None, 0, clip)


def attn_pv(Pq: np.ndarray, p_scale: np.ndarray, codes, scales, zeros, D: int) -> np.ndarray:
    """O[t, h, d] = (float(sum_s Pq[h, t, s] * t2(code[h*D + d, s])) * p_scale[h, t]) * (0.5 * step[h*D + d]),
    BF16 bits [T, H, D]: Eq. 1 once per head with the channels (h, d) as output features."""
    Pq = _c(Pq, np.int8)
    p_scale = _c(p_scale, np.float32)
    H, T, S = Pq.shape
    out = np.empty((T, H, D), dtype=np.uint16)
    for h in range(H):
        sl = slice(h * D, (h + 1) * D)
        out[:, h, :] = linear(Pq[h], p_scale[h], np.ascontiguousarray(codes[sl]),
                              np.ascontiguousarray(scales[:, sl]), np.ascontiguousarray(zeros[:, sl]), None, 0)
    return out


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    """Widen BF16 bit patterns (uint16) to float32 values (exact)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)
