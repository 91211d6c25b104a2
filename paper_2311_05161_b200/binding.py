"""ctypes binding of libw4a8.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/w4a8.h) minus the
`w4a8_` prefix.  torch supplies device memory and the current stream; all arithmetic of
the path runs in the library's CUDA kernels.  There is no fallback: a missing library or a
non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libw4a8.so")

STATUS_NAMES = {
    0: "W4A8_OK", 1: "W4A8_ERR_NULL", 2: "W4A8_ERR_SHAPE", 3: "W4A8_ERR_ALIGN",
    4: "W4A8_ERR_BUFFER_TOO_SMALL", 5: "W4A8_ERR_UNSUPPORTED_ARCH", 6: "W4A8_ERR_CUDA",
    7: "W4A8_ERR_TIMEOUT", 8: "W4A8_ERR_BAD_BLOB",
}
PATH_AUTO, PATH_SIMPLE, PATH_TCGEN05, PATH_GEMV = 0, 1, 2, 3

EXPORTS = (
    "w4a8_packed_bytes", "w4a8_pack_weights", "w4a8_quantize_act",
    "w4a8_linear_workspace_bytes", "w4a8_linear_workspace_bytes_ex", "w4a8_workspace_init",
    "w4a8_linear", "w4a8_linear_ex", "w4a8_linear_static", "w4a8_static_poll_status", "w4a8_linear_acc_i32",
    "w4a8_unpack_codes",
    "w4a8_poll_status", "w4a8_dint4_table", "w4a8_version",
    "w4a8_quantize_act_asym", "w4a8_weight_rowsum", "w4a8_linear_asym",
    "w4a8_pack_weights_fmt", "w4a8_dint4_table_fmt",
    "w4a8_quantize_linear", "w4a8_quantize_linear_workspace_bytes", "w4a8_linear_plan", "w4a8_norm_quantize_act",
    "w4a8_packed_bytes_bits", "w4a8_pack_weights_bits", "w4a8_unpack_codes_bits", "w4a8_dint_table_bits",
    "w4a8_pack_value", "w4a8_attn_pv", "w4a8_attn_pv_workspace_bytes",
    "w4a8_linear_swiglu", "w4a8_linear_swiglu_workspace_bytes", "w4a8_linear_asym_group",
)


class W4A8Error(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}")


class Opts(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int), ("split_k", ctypes.c_int), ("tok_tile", ctypes.c_int),
                ("decode_warps", ctypes.c_int), ("level_shift", ctypes.c_int),
                ("cluster", ctypes.c_int), ("debug_wait_ms", ctypes.c_int), ("debug_skip_load", ctypes.c_int),
                ("bits", ctypes.c_int), ("offset_tables", ctypes.c_int),
                ("tok_run", ctypes.c_int)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python __graft_entry__.py` "
            "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, sz, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_float
    op = ctypes.POINTER(Opts)
    lib.w4a8_packed_bytes.restype = sz
    lib.w4a8_packed_bytes.argtypes = [ci, ci, ci]
    lib.w4a8_pack_weights.restype = ci
    lib.w4a8_pack_weights.argtypes = [vp, vp, ci, ci, ci, cf, vp, sz, vp]
    lib.w4a8_quantize_act.restype = ci
    lib.w4a8_quantize_act.argtypes = [vp, vp, ci, ci, vp, vp, vp]
    lib.w4a8_norm_quantize_act.restype = ci
    lib.w4a8_norm_quantize_act.argtypes = [vp, vp, vp, ci, cf, ci, ci, vp, vp, vp]
    lib.w4a8_linear_workspace_bytes.restype = sz
    lib.w4a8_linear_workspace_bytes.argtypes = [ci, ci, ci, ci]
    lib.w4a8_linear_workspace_bytes_ex.restype = sz
    lib.w4a8_linear_workspace_bytes_ex.argtypes = [ci, ci, ci, ci, op]
    lib.w4a8_linear_plan.restype = ci
    lib.w4a8_linear_plan.argtypes = [ci, ci, ci, ci, op, vp]
    lib.w4a8_workspace_init.restype = ci
    lib.w4a8_workspace_init.argtypes = [vp, sz, vp]
    lib.w4a8_linear.restype = ci
    lib.w4a8_linear.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, sz, vp]
    lib.w4a8_linear_ex.restype = ci
    lib.w4a8_linear_ex.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, sz, vp, op]
    lib.w4a8_linear_static.restype = ci
    lib.w4a8_linear_static.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp]
    lib.w4a8_static_poll_status.restype = ci
    lib.w4a8_static_poll_status.argtypes = [vp]
    lib.w4a8_quantize_linear_workspace_bytes.restype = sz
    lib.w4a8_quantize_linear_workspace_bytes.argtypes = [ci, ci, ci, ci]
    lib.w4a8_quantize_linear.restype = ci
    lib.w4a8_quantize_linear.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, sz, vp]
    lib.w4a8_packed_bytes_bits.restype = sz
    lib.w4a8_packed_bytes_bits.argtypes = [ci, ci, ci, ci]
    lib.w4a8_pack_weights_bits.restype = ci
    lib.w4a8_pack_weights_bits.argtypes = [vp, vp, ci, ci, ci, cf, ci, ci, vp, sz, vp]
    lib.w4a8_unpack_codes_bits.restype = ci
    lib.w4a8_unpack_codes_bits.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp]
    lib.w4a8_dint_table_bits.restype = None
    lib.w4a8_dint_table_bits.argtypes = [ci, ci, ci, vp]
    lib.w4a8_linear_swiglu_workspace_bytes.restype = sz
    lib.w4a8_linear_swiglu_workspace_bytes.argtypes = [ci, ci, ci, ci]
    lib.w4a8_linear_swiglu.restype = ci
    lib.w4a8_linear_swiglu.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, sz, vp]
    lib.w4a8_pack_value.restype = ci
    lib.w4a8_pack_value.argtypes = [vp, ci, ci, ci, cf, vp, sz, vp]
    lib.w4a8_attn_pv_workspace_bytes.restype = sz
    lib.w4a8_attn_pv_workspace_bytes.argtypes = [ci, ci, ci, ci]
    lib.w4a8_attn_pv.restype = ci
    lib.w4a8_attn_pv.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, vp, sz, vp]
    lib.w4a8_pack_weights_fmt.restype = ci
    lib.w4a8_pack_weights_fmt.argtypes = [vp, vp, ci, ci, ci, cf, ci, vp, sz, vp]
    lib.w4a8_quantize_act_asym.restype = ci
    lib.w4a8_quantize_act_asym.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp]
    lib.w4a8_weight_rowsum.restype = ci
    lib.w4a8_weight_rowsum.argtypes = [vp, ci, ci, ci, vp, vp]
    lib.w4a8_linear_asym.restype = ci
    lib.w4a8_linear_asym.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, vp, vp, vp, sz, vp, op]
    lib.w4a8_linear_asym_group.restype = ci
    lib.w4a8_linear_asym_group.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, vp, sz, vp, op]
    lib.w4a8_linear_acc_i32.restype = ci
    lib.w4a8_linear_acc_i32.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, sz, vp, op]
    lib.w4a8_unpack_codes.restype = ci
    lib.w4a8_unpack_codes.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp]
    lib.w4a8_poll_status.restype = ci
    lib.w4a8_poll_status.argtypes = [vp, vp]
    lib.w4a8_dint4_table.restype = None
    lib.w4a8_dint4_table.argtypes = [ci, vp]
    lib.w4a8_version.restype = ctypes.c_char_p
    lib.w4a8_version.argtypes = []
    return lib


lib = _load()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, what: str):
    if status != 0:
        raise W4A8Error(status, what)


def _dev(t, dtype, what):
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{what}: expected a contiguous CUDA tensor of {dtype}")
    return t


def make_opts(path: int = PATH_AUTO, split_k: int = 0, tok_tile: int = 0,
              decode_warps: int = 0, level_shift: int = 0, cluster: int = 0,
              debug_wait_ms: int = 0, debug_skip_load: int = 0, bits: int = 0,
              offset_tables: int = 0, tok_run: int = 0) -> Opts:
    o = Opts()
    o.path, o.split_k, o.tok_tile, o.decode_warps = path, split_k, tok_tile, decode_warps
    o.level_shift = level_shift
    o.cluster = cluster
    o.debug_wait_ms, o.debug_skip_load = debug_wait_ms, debug_skip_load
    o.bits = bits
    o.offset_tables = offset_tables
    o.tok_run = tok_run
    return o


def version() -> str:
    return lib.w4a8_version().decode()


def dint4_table(z: int):
    buf = (ctypes.c_int8 * 16)()
    lib.w4a8_dint4_table(z, buf)
    return list(buf)


def packed_bytes(N: int, K: int, group: int = 0, bits: int = 4) -> int:
    return int(lib.w4a8_packed_bytes_bits(N, K, group, bits))


def dint_table(z: int, bits: int = 4, level_shift: int = 1):
    buf = (ctypes.c_int8 * 16)()
    lib.w4a8_dint_table_bits(z, bits, level_shift, buf)
    return list(buf)[: 1 << bits]


def pack_weights(W, s_in=None, group: int = 0, clip: float = 1.0, out=None, level_shift: int = 1,
                 bits: int = 4):
    """W [N, K] float16 (CUDA) -> packed blob (uint8 CUDA tensor); `bits`-bit dINT codes,
    special value step / 2^level_shift."""
    W = _dev(W, torch.float16, "W")
    s_in = _dev(s_in, torch.float32, "s_in")
    N, K = W.shape
    nbytes = packed_bytes(N, K, group, bits)
    if nbytes == 0:
        raise W4A8Error(2, "w4a8_packed_bytes")
    if out is None:
        out = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    _check(lib.w4a8_pack_weights_bits(_ptr(W), _ptr(s_in), N, K, group, clip, bits, level_shift,
                                      _ptr(out), out.numel(), _stream()), "w4a8_pack_weights")
    return out


def quantize_act(X, inv_s_in=None, out=None):
    """X [M, K] float16 (CUDA) -> (Xq [M, K] int8, tok_scale [M] float32)."""
    X = _dev(X, torch.float16, "X")
    inv_s_in = _dev(inv_s_in, torch.float32, "inv_s_in")
    M, K = X.shape
    if out is None:
        out = (torch.empty((M, K), dtype=torch.int8, device=X.device),
               torch.empty((M,), dtype=torch.float32, device=X.device))
    Xq, tok = out
    _check(lib.w4a8_quantize_act(_ptr(X), _ptr(inv_s_in), M, K, _ptr(Xq), _ptr(tok), _stream()),
           "w4a8_quantize_act")
    return Xq, tok


NORM_RMS, NORM_LAYER = 0, 1


def norm_quantize_act(X, norm_weight, norm_bias=None, kind: int = NORM_RMS, eps: float = 1e-5, out=None):
    """RMSNorm / LayerNorm (weight and bias carry the reciprocal Eq. 1 scale) and the token-wise
    INT8 quantizer in one pass: X [M, K] float16 (CUDA) -> (Xq [M, K] int8, tok_scale [M] float32)."""
    X = _dev(X, torch.float16, "X")
    norm_weight = _dev(norm_weight, torch.float32, "norm_weight")
    norm_bias = _dev(norm_bias, torch.float32, "norm_bias")
    M, K = X.shape
    if out is None:
        out = (torch.empty((M, K), dtype=torch.int8, device=X.device),
               torch.empty((M,), dtype=torch.float32, device=X.device))
    Xq, tok = out
    _check(lib.w4a8_norm_quantize_act(_ptr(X), _ptr(norm_weight), _ptr(norm_bias), kind, eps, M, K,
                                      _ptr(Xq), _ptr(tok), _stream()), "w4a8_norm_quantize_act")
    return Xq, tok


def linear_workspace_bytes(M: int, N: int, K: int, group: int = 0, opts: Opts | None = None) -> int:
    if opts is None:
        return int(lib.w4a8_linear_workspace_bytes(M, N, K, group))
    return int(lib.w4a8_linear_workspace_bytes_ex(M, N, K, group, ctypes.byref(opts)))


def linear_plan(M: int, N: int, K: int, group: int = 0, opts: Opts | None = None) -> dict:
    """What w4a8_linear(_ex) would run for this shape: kernel, token tile, K slices, warps."""
    out = (ctypes.c_int * 5)()
    _check(lib.w4a8_linear_plan(M, N, K, group, ctypes.byref(opts) if opts is not None else None,
                                out), "w4a8_linear_plan")
    names = {PATH_SIMPLE: "simple", PATH_TCGEN05: "tcgen05", PATH_GEMV: "weight-streaming"}
    return {"kernel": names.get(out[0], str(out[0])), "tok_tile": out[1], "split_k": out[2],
            "warps": out[3], "cluster": out[4]}


def workspace_init(ws):
    _check(lib.w4a8_workspace_init(_ptr(ws), ws.numel(), _stream()), "w4a8_workspace_init")


def new_workspace(M: int, N: int, K: int, group: int = 0, opts: Opts | None = None, device="cuda"):
    nbytes = linear_workspace_bytes(M, N, K, group, opts)
    if nbytes == 0:
        raise W4A8Error(2, "w4a8_linear_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def linear(Xq, tok_scale, packed, bias, N: int, group: int, workspace, opts: Opts | None = None,
           out=None):
    """Quantized linear layer: returns Y [M, N] bfloat16."""
    Xq = _dev(Xq, torch.int8, "Xq")
    tok_scale = _dev(tok_scale, torch.float32, "tok_scale")
    bias = _dev(bias, torch.float32, "bias")
    M, K = Xq.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=Xq.device)
    if opts is None:
        st = lib.w4a8_linear(_ptr(Xq), _ptr(tok_scale), _ptr(packed), _ptr(bias), M, N, K, group,
                             _ptr(out), _ptr(workspace), workspace.numel(), _stream())
    else:
        st = lib.w4a8_linear_ex(_ptr(Xq), _ptr(tok_scale), _ptr(packed), _ptr(bias), M, N, K,
                                group, _ptr(out), _ptr(workspace), workspace.numel(), _stream(),
                                ctypes.byref(opts))
    _check(st, "w4a8_linear")
    return out


def quantize_linear_workspace_bytes(M: int, N: int, K: int, group: int = 0) -> int:
    return int(lib.w4a8_quantize_linear_workspace_bytes(M, N, K, group))


def new_quantize_linear_workspace(M: int, N: int, K: int, group: int = 0, device="cuda"):
    nbytes = quantize_linear_workspace_bytes(M, N, K, group)
    if nbytes == 0:
        raise W4A8Error(2, "w4a8_quantize_linear_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def quantize_linear(X, inv_s_in, packed, bias, N: int, group: int, workspace, out=None):
    """Decode form, one to four tokens: activation quantizer and quantized linear layer in one
    launch.  X [M, K] float16 (CUDA) -> Y [M, N] bfloat16."""
    X = _dev(X, torch.float16, "X")
    inv_s_in = _dev(inv_s_in, torch.float32, "inv_s_in")
    bias = _dev(bias, torch.float32, "bias")
    M, K = X.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    _check(lib.w4a8_quantize_linear(_ptr(X), _ptr(inv_s_in), _ptr(packed), _ptr(bias), M, N, K,
                                    group, _ptr(out), _ptr(workspace), workspace.numel(),
                                    _stream()), "w4a8_quantize_linear")
    return out


def quantize_act_asym(X, inv_s_in=None, out=None):
    """Asymmetric token-wise quantizer: X [M, K] float16 (CUDA) ->
    (Xq [M, K] int8 = code - 128, tok_scale [M] float32, tok_zero [M] int32 = zero-point - 128)."""
    X = _dev(X, torch.float16, "X")
    inv_s_in = _dev(inv_s_in, torch.float32, "inv_s_in")
    M, K = X.shape
    if out is None:
        out = (torch.empty((M, K), dtype=torch.int8, device=X.device),
               torch.empty((M,), dtype=torch.float32, device=X.device),
               torch.empty((M,), dtype=torch.int32, device=X.device))
    Xq, tok, zero = out
    _check(lib.w4a8_quantize_act_asym(_ptr(X), _ptr(inv_s_in), M, K, _ptr(Xq), _ptr(tok),
                                      _ptr(zero), _stream()), "w4a8_quantize_act_asym")
    return Xq, tok, zero


def weight_rowsum(packed, N: int, K: int, group: int = 0):
    """Row sums of the doubled weight levels: int32 [G, N]."""
    G = K // group if group else 1
    out = torch.empty((G, N), dtype=torch.int32, device=packed.device)
    _check(lib.w4a8_weight_rowsum(_ptr(packed), N, K, group, _ptr(out), _stream()),
           "w4a8_weight_rowsum")
    return out


def linear_asym_group(Xq, tok_scale, tok_zero, packed, rowsum, bias, N: int, group: int, workspace,
                      opts: Opts | None = None, out=None, want_acc: bool = False):
    """linear_asym for group-wise weight steps: rowsum is [G, N]; returns Y [M, N] bfloat16, or
    (Y, acc [G, M, N] int32) with `want_acc`."""
    Xq = _dev(Xq, torch.int8, "Xq")
    tok_scale = _dev(tok_scale, torch.float32, "tok_scale")
    tok_zero = _dev(tok_zero, torch.int32, "tok_zero")
    rowsum = _dev(rowsum, torch.int32, "rowsum")
    bias = _dev(bias, torch.float32, "bias")
    M, K = Xq.shape
    G = K // group if group else 1
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=Xq.device)
    acc = torch.empty((G, M, N), dtype=torch.int32, device=Xq.device) if want_acc else None
    st = lib.w4a8_linear_asym_group(_ptr(Xq), _ptr(tok_scale), _ptr(tok_zero), _ptr(packed), _ptr(rowsum),
                                    _ptr(bias), M, N, K, group, _ptr(out), _ptr(acc), _ptr(workspace),
                                    workspace.numel(), _stream(),
                                    ctypes.byref(opts) if opts is not None else None)
    _check(st, "w4a8_linear_asym_group")
    return (out, acc) if want_acc else out


def linear_asym(Xq, tok_scale, tok_zero, packed, rowsum, bias, N: int, workspace,
                opts: Opts | None = None, out=None, want_acc: bool = False):
    """Quantized linear layer with asymmetric activations (per-channel weights): returns
    Y [M, N] bfloat16, or (Y, acc [M, N] int32) with `want_acc`."""
    Xq = _dev(Xq, torch.int8, "Xq")
    tok_scale = _dev(tok_scale, torch.float32, "tok_scale")
    tok_zero = _dev(tok_zero, torch.int32, "tok_zero")
    rowsum = _dev(rowsum, torch.int32, "rowsum")
    bias = _dev(bias, torch.float32, "bias")
    M, K = Xq.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=Xq.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=Xq.device) if want_acc else None
    st = lib.w4a8_linear_asym(_ptr(Xq), _ptr(tok_scale), _ptr(tok_zero), _ptr(packed), _ptr(rowsum),
                              _ptr(bias), M, N, K, _ptr(out), _ptr(acc), _ptr(workspace),
                              workspace.numel(), _stream(),
                              ctypes.byref(opts) if opts is not None else None)
    _check(st, "w4a8_linear_asym")
    return (out, acc) if want_acc else out


def interleave_gate_up(Wg, Wu):
    """[F, K] gate and up weights -> [2 F, K] with row 2 i = gate row i, row 2 i + 1 = up row i."""
    F, K = Wg.shape
    return torch.stack((Wg, Wu), dim=1).reshape(2 * F, K).contiguous()


def new_linear_swiglu_workspace(M: int, F: int, K: int, group: int = 0, device="cuda"):
    nbytes = int(lib.w4a8_linear_swiglu_workspace_bytes(M, F, K, group))
    if nbytes == 0:
        raise W4A8Error(2, "w4a8_linear_swiglu_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def linear_swiglu(Xq, tok_scale, packed_gate_up, bias_gate_up, F: int, group: int, workspace, out=None):
    """Gate and up projections (rows interleaved in one blob) with silu(gate) * up in the epilogue:
    returns H [M, F] float16."""
    Xq = _dev(Xq, torch.int8, "Xq")
    tok_scale = _dev(tok_scale, torch.float32, "tok_scale")
    bias_gate_up = _dev(bias_gate_up, torch.float32, "bias_gate_up")
    M, K = Xq.shape
    if out is None:
        out = torch.empty((M, F), dtype=torch.float16, device=Xq.device)
    _check(lib.w4a8_linear_swiglu(_ptr(Xq), _ptr(tok_scale), _ptr(packed_gate_up), _ptr(bias_gate_up), M, F,
                                  K, group, _ptr(out), _ptr(workspace), workspace.numel(), _stream()),
           "w4a8_linear_swiglu")
    return out


def pack_value(V, clip: float = 1.0, out=None):
    """Attention values V [S, H, D] float16 (CUDA) -> dINT4 blob, one step per channel (h, d)."""
    V = _dev(V, torch.float16, "V")
    S, H, D = V.shape
    nbytes = packed_bytes(H * D, S, 0)
    if nbytes == 0:
        raise W4A8Error(2, "w4a8_packed_bytes")
    if out is None:
        out = torch.empty(nbytes, dtype=torch.uint8, device=V.device)
    _check(lib.w4a8_pack_value(_ptr(V), S, H, D, clip, _ptr(out), out.numel(), _stream()), "w4a8_pack_value")
    return out


def new_attn_pv_workspace(T: int, S: int, H: int, D: int, device="cuda"):
    nbytes = int(lib.w4a8_attn_pv_workspace_bytes(T, S, H, D))
    if nbytes == 0:
        raise W4A8Error(2, "w4a8_attn_pv_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def attn_pv(Pq, p_scale, packed, D: int, workspace, out=None):
    """Pq [H, T, S] int8, p_scale [H, T] float32, packed values -> O [T, H, D] bfloat16."""
    Pq = _dev(Pq, torch.int8, "Pq")
    p_scale = _dev(p_scale, torch.float32, "p_scale")
    H, T, S = Pq.shape
    if out is None:
        out = torch.empty((T, H, D), dtype=torch.bfloat16, device=Pq.device)
    _check(lib.w4a8_attn_pv(_ptr(Pq), _ptr(p_scale), _ptr(packed), T, S, H, D, _ptr(out),
                            _ptr(workspace), workspace.numel(), _stream()), "w4a8_attn_pv")
    return out


def linear_static(Xq, tok_scale, packed, bias, N: int, group: int, out):
    """w4a8_linear without a workspace: the library's built-in scratch array is used, and
    nothing is allocated here either, so the caller passes the output tensor `out`
    ([M, N] bfloat16).  For callers that may not allocate device memory."""
    Xq = _dev(Xq, torch.int8, "Xq")
    tok_scale = _dev(tok_scale, torch.float32, "tok_scale")
    bias = _dev(bias, torch.float32, "bias")
    out = _dev(out, torch.bfloat16, "out")
    M, K = Xq.shape
    _check(lib.w4a8_linear_static(_ptr(Xq), _ptr(tok_scale), _ptr(packed), _ptr(bias), M, N, K,
                                  group, _ptr(out), _stream()), "w4a8_linear_static")
    return out


def static_poll_status() -> int:
    """Status the kernel of the last linear_static call on this device reported (0 = none)."""
    return int(lib.w4a8_static_poll_status(_stream()))


def linear_acc_i32(Xq, packed, N: int, group: int, workspace, opts: Opts | None = None, out=None):
    """INT32 accumulators [G, M, N] of the contraction (test export)."""
    Xq = _dev(Xq, torch.int8, "Xq")
    M, K = Xq.shape
    G = K // group if group else 1
    acc = out if out is not None else torch.empty((G, M, N), dtype=torch.int32, device=Xq.device)
    _check(lib.w4a8_linear_acc_i32(_ptr(Xq), _ptr(packed), M, N, K, group, _ptr(acc),
                                   _ptr(workspace), workspace.numel(), _stream(),
                                   ctypes.byref(opts) if opts is not None else None),
           "w4a8_linear_acc_i32")
    return acc


def unpack_codes(packed, N: int, K: int, group: int = 0, bits: int = 4):
    """Blob -> (codes [N, K/2] uint8, scales [G, N] float32, zeros [G, N] uint8)."""
    G = K // group if group else 1
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=packed.device)
    scales = torch.empty((G, N), dtype=torch.float32, device=packed.device)
    zeros = torch.empty((G, N), dtype=torch.uint8, device=packed.device)
    _check(lib.w4a8_unpack_codes_bits(_ptr(packed), N, K, group, bits, _ptr(codes), _ptr(scales),
                                      _ptr(zeros), _stream()), "w4a8_unpack_codes")
    return codes, scales, zeros


def poll_status(workspace) -> int:
    return int(lib.w4a8_poll_status(_ptr(workspace), _stream()))


def check_status(workspace):
    _check(poll_status(workspace), "w4a8_poll_status")
