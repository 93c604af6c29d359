"""Thin ctypes binding over ``libbitnet_a48.so`` (argument marshalling only).

Every function has the name of the C entry point it calls (see
``include/bitnet_a48.h``) minus the ``bitnet_a48_`` prefix.  Tensors are torch
CUDA tensors used purely as device buffers; streams are torch streams.  There
is no fallback: if the shared library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_float, c_int, c_size_t, c_uint, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbitnet_a48.so")

ACT_INT4, ACT_TOPK_INT8, ACT_FP4 = 0, 1, 2
LAYOUT_GEMM, LAYOUT_DECODE, LAYOUT_SPARSE, LAYOUT_ALL, LAYOUT_I8, LAYOUT_TRIT5 = 1, 2, 4, 7, 8, 16
ALGO_AUTO, ALGO_SIMPLE, ALGO_GEMM_TCGEN05, ALGO_DECODE, ALGO_DECODE_SPARSE, ALGO_GEMM_TCGEN05_I8 = 0, 1, 2, 3, 4, 5
ALGO_GEMM_TCGEN05_PAIR = 6
ALGO_DECODE_TRIT5 = 7

EXPORTS = [
    "bitnet_a48_status_string", "bitnet_a48_pack_ternary", "bitnet_a48_weight_unpack",
    "bitnet_a48_weight_unpack_layout", "bitnet_a48_weight_dims", "bitnet_a48_weight_packed_bytes",
    "bitnet_a48_weight_free", "bitnet_a48_quant_int4", "bitnet_a48_topk_quant_int8", "bitnet_a48_quant_fp4",
    "bitnet_a48_compact_codes",
    "bitnet_a48_linear", "bitnet_a48_linear_ex", "bitnet_a48_linear_workspace_bytes",
    "bitnet_a48_bitlinear_host", "bitnet_a48_bitlinear_host_workspace_bytes", "bitnet_a48_block_create",
    "bitnet_a48_block_free", "bitnet_a48_block_workspace_bytes", "bitnet_a48_block_forward",
    "bitnet_a48_kernel_status", "bitnet_a48_linear_decode_static", "bitnet_a48_linear_multi",
    "bitnet_a48_linear_multi_workspace_bytes", "bitnet_a48_bitlinear_host_async",
    "bitnet_a48_ffn_gate_first", "bitnet_a48_ffn_gate_first_workspace_bytes",
    "bitnet_a48_ffn_dense", "bitnet_a48_kv_cache_bytes", "bitnet_a48_weight_layout_bytes",
    "bitnet_a48_quant_int4_bf16", "bitnet_a48_topk_quant_int8_bf16", "bitnet_a48_linear_bf16",
    "bitnet_a48_attention_prefill", "bitnet_a48_attention_prefill_workspace_bytes",
]


class A48Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: status {code} ({status_string(code)})")


class BlockConfig(ctypes.Structure):
    _fields_ = [("hidden", c_int), ("n_heads", c_int), ("ffn", c_int), ("k_o", c_int), ("k_down", c_int),
                ("ctx_cap", c_int), ("norm_eps", c_float), ("quant_eps", c_float), ("rope_base", c_float),
                ("act_fp4", c_int), ("q_bits", c_int), ("kv_bits", c_int)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run paper_2411_04965_b200/build.py (there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.bitnet_a48_status_string.restype = ctypes.c_char_p
        L.bitnet_a48_status_string.argtypes = [c_int]
        for name in ("bitnet_a48_weight_packed_bytes", "bitnet_a48_linear_workspace_bytes",
                     "bitnet_a48_bitlinear_host_workspace_bytes", "bitnet_a48_block_workspace_bytes"):
            getattr(L, name).restype = c_size_t
        L.bitnet_a48_weight_packed_bytes.argtypes = [c_void_p]
        L.bitnet_a48_weight_layout_bytes.restype = c_size_t
        L.bitnet_a48_weight_layout_bytes.argtypes = [c_void_p, c_uint]
        L.bitnet_a48_linear_workspace_bytes.argtypes = [c_void_p, c_int]
        L.bitnet_a48_bitlinear_host_workspace_bytes.argtypes = [c_void_p, c_int]
        L.bitnet_a48_block_workspace_bytes.argtypes = [c_void_p, c_int, c_int]
        L.bitnet_a48_pack_ternary.argtypes = [c_void_p, c_int, c_int, c_float, c_uint, POINTER(c_void_p), c_void_p]
        L.bitnet_a48_weight_unpack.argtypes = [c_void_p, c_void_p, POINTER(c_float), c_void_p]
        L.bitnet_a48_weight_unpack_layout.argtypes = [c_void_p, c_uint, c_void_p, c_void_p]
        L.bitnet_a48_weight_dims.argtypes = [c_void_p, POINTER(c_int), POINTER(c_int), POINTER(c_uint)]
        L.bitnet_a48_weight_free.argtypes = [c_void_p]
        L.bitnet_a48_weight_free.restype = None
        L.bitnet_a48_quant_int4.argtypes = [c_void_p, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p]
        L.bitnet_a48_topk_quant_int8.argtypes = [c_void_p, c_int, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p,
                                                 c_void_p]
        L.bitnet_a48_quant_fp4.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p]
        L.bitnet_a48_compact_codes.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
        L.bitnet_a48_linear.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p,
                                        c_size_t, c_void_p]
        L.bitnet_a48_linear_ex.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p,
                                           c_void_p, c_size_t, c_void_p]
        L.bitnet_a48_bitlinear_host.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_float, c_void_p, c_void_p,
                                                c_size_t, c_void_p]
        L.bitnet_a48_bitlinear_host_async.argtypes = L.bitnet_a48_bitlinear_host.argtypes
        L.bitnet_a48_block_create.argtypes = [POINTER(BlockConfig), POINTER(c_void_p), c_void_p, c_void_p,
                                              POINTER(c_void_p)]
        L.bitnet_a48_block_free.argtypes = [c_void_p]
        L.bitnet_a48_block_free.restype = None
        L.bitnet_a48_block_forward.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p,
                                               c_void_p, c_size_t, c_void_p]
        L.bitnet_a48_kernel_status.argtypes = [POINTER(c_uint)]
        L.bitnet_a48_quant_int4_bf16.argtypes = [c_void_p, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p]
        L.bitnet_a48_topk_quant_int8_bf16.argtypes = [c_void_p, c_int, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p]
        L.bitnet_a48_linear_bf16.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_size_t,
                                             c_void_p]
        L.bitnet_a48_attention_prefill_workspace_bytes.restype = c_size_t
        L.bitnet_a48_attention_prefill_workspace_bytes.argtypes = [c_int, c_int, c_int, c_int, c_int]
        L.bitnet_a48_attention_prefill.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int, c_int,
                                                   c_void_p, c_void_p, c_size_t, c_void_p]
        L.bitnet_a48_kv_cache_bytes.restype = c_size_t
        L.bitnet_a48_kv_cache_bytes.argtypes = [c_void_p, c_int]
        L.bitnet_a48_linear_multi.argtypes = [c_int, POINTER(c_void_p), c_void_p, c_void_p, c_int, c_int, POINTER(c_void_p),
                                              c_void_p, c_size_t, c_void_p]
        L.bitnet_a48_linear_multi_workspace_bytes.restype = c_size_t
        L.bitnet_a48_linear_multi_workspace_bytes.argtypes = [c_int, POINTER(c_void_p), c_int]
        L.bitnet_a48_linear_decode_static.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p]
        L.bitnet_a48_ffn_gate_first.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_float, c_void_p,
                                                c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.bitnet_a48_ffn_dense.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_float, c_void_p, c_void_p,
                                           c_size_t, c_void_p]
        L.bitnet_a48_ffn_gate_first_workspace_bytes.restype = c_size_t
        L.bitnet_a48_ffn_gate_first_workspace_bytes.argtypes = [c_void_p, c_void_p, c_void_p, c_int]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().bitnet_a48_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise A48Error(code, where)


def _ptr(t):
    return c_void_p(t.data_ptr()) if t is not None else c_void_p(0)


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return c_void_p(s.cuda_stream)


class Weight:
    """Owns a ``bitnet_a48_weight`` handle."""

    def __init__(self, handle: int, N: int, K: int, layouts: int):
        self.handle, self.N, self.K, self.layouts = handle, N, K, layouts

    def free(self):
        if self.handle:
            lib().bitnet_a48_weight_free(c_void_p(self.handle))
            self.handle = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    @property
    def packed_bytes(self) -> int:
        return int(lib().bitnet_a48_weight_packed_bytes(c_void_p(self.handle)))

    def layout_bytes(self, layout: int) -> int:
        return int(lib().bitnet_a48_weight_layout_bytes(c_void_p(self.handle), layout))


def pack_ternary(W: torch.Tensor, eps: float = 1e-5, layouts: int = LAYOUT_ALL, stream=None) -> Weight:
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    N, K = W.shape
    out = c_void_p(0)
    _check(lib().bitnet_a48_pack_ternary(_ptr(W), N, K, eps, layouts, byref(out), _stream(stream)), "pack_ternary")
    return Weight(out.value, N, K, layouts)


def weight_unpack(w: Weight, stream=None):
    """Returns (codes int8 [N,K] on the device, alpha as a Python float)."""
    codes = torch.empty(w.N, w.K, dtype=torch.int8, device="cuda")
    alpha = c_float(0.0)
    _check(lib().bitnet_a48_weight_unpack(c_void_p(w.handle), _ptr(codes), byref(alpha), _stream(stream)),
           "weight_unpack")
    return codes, alpha.value


def weight_unpack_layout(w: Weight, layout: int, stream=None) -> torch.Tensor:
    codes = torch.full((w.N, w.K), 99, dtype=torch.int8, device="cuda")
    _check(lib().bitnet_a48_weight_unpack_layout(c_void_p(w.handle), layout, _ptr(codes), _stream(stream)),
           "weight_unpack_layout")
    return codes


def quant_int4(X: torch.Tensor, eps: float = 1e-5, codes=None, scale=None, stream=None):
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.dim() == 2
    M, K = X.shape
    codes = codes if codes is not None else torch.empty(M, K, dtype=torch.int8, device=X.device)
    scale = scale if scale is not None else torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().bitnet_a48_quant_int4(_ptr(X), M, K, eps, _ptr(codes), _ptr(scale), _stream(stream)), "quant_int4")
    return codes, scale


def topk_quant_int8(X: torch.Tensor, k: int, eps: float = 1e-5, codes=None, scale=None, mask_bits=None,
                    want_mask: bool = False, stream=None):
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.dim() == 2
    M, K = X.shape
    codes = codes if codes is not None else torch.empty(M, K, dtype=torch.int8, device=X.device)
    scale = scale if scale is not None else torch.empty(M, dtype=torch.float32, device=X.device)
    if want_mask and mask_bits is None:
        mask_bits = torch.zeros(M, (K + 31) // 32, dtype=torch.int32, device=X.device)
    _check(lib().bitnet_a48_topk_quant_int8(_ptr(X), M, K, k, eps, _ptr(codes), _ptr(scale), _ptr(mask_bits),
                                            _stream(stream)), "topk_quant_int8")
    return codes, scale, mask_bits


def quant_int4_bf16(X: torch.Tensor, eps: float = 1e-5, codes=None, scale=None, stream=None):
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous() and X.dim() == 2
    M, K = X.shape
    codes = codes if codes is not None else torch.empty(M, K, dtype=torch.int8, device=X.device)
    scale = scale if scale is not None else torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().bitnet_a48_quant_int4_bf16(_ptr(X), M, K, eps, _ptr(codes), _ptr(scale), _stream(stream)),
           "quant_int4_bf16")
    return codes, scale


def topk_quant_int8_bf16(X: torch.Tensor, k: int, eps: float = 1e-5, codes=None, scale=None, stream=None):
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous() and X.dim() == 2
    M, K = X.shape
    codes = codes if codes is not None else torch.empty(M, K, dtype=torch.int8, device=X.device)
    scale = scale if scale is not None else torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().bitnet_a48_topk_quant_int8_bf16(_ptr(X), M, K, k, eps, _ptr(codes), _ptr(scale), _stream(stream)),
           "topk_quant_int8_bf16")
    return codes, scale


def linear_bf16(w: Weight, codes: torch.Tensor, scale: torch.Tensor, kind: int = ACT_INT4, Y=None, workspace=None,
                stream=None):
    """BitLinear with a bf16 output (round-to-nearest-even of the fp32 result)."""
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.is_contiguous() and codes.shape[1] == w.K
    M = codes.shape[0]
    Y = Y if Y is not None else torch.empty(M, w.N, dtype=torch.bfloat16, device=codes.device)
    assert Y.dtype == torch.bfloat16 and Y.is_contiguous()
    need = linear_workspace_bytes(w, M)
    if workspace is None and need:
        workspace = torch.zeros(need, dtype=torch.uint8, device=codes.device)
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().bitnet_a48_linear_bf16(c_void_p(w.handle), _ptr(codes), _ptr(scale), M, kind, _ptr(Y), _ptr(workspace),
                                        ws_bytes, _stream(stream)), "linear_bf16")
    return Y


def quant_fp4(X: torch.Tensor, codes=None, scale=None, stream=None):
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.dim() == 2
    M, K = X.shape
    codes = codes if codes is not None else torch.empty(M, K, dtype=torch.int8, device=X.device)
    scale = scale if scale is not None else torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().bitnet_a48_quant_fp4(_ptr(X), M, K, _ptr(codes), _ptr(scale), _stream(stream)), "quant_fp4")
    return codes, scale


def compact_codes(codes: torch.Tensor, cap: int, stream=None):
    """Non-zero codes of every row as (channel index uint16, code int8) lists [M, cap] plus counts [M] (int32)."""
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.is_contiguous() and codes.dim() == 2
    M, K = codes.shape
    idx = torch.zeros(M, cap, dtype=torch.uint16, device=codes.device)
    val = torch.zeros(M, cap, dtype=torch.int8, device=codes.device)
    count = torch.empty(M, dtype=torch.int32, device=codes.device)
    _check(lib().bitnet_a48_compact_codes(_ptr(codes), M, K, cap, _ptr(idx), _ptr(val), _ptr(count), _stream(stream)),
           "compact_codes")
    return idx, val, count


def linear_workspace_bytes(w: Weight, M: int) -> int:
    return int(lib().bitnet_a48_linear_workspace_bytes(c_void_p(w.handle), M))


def linear(w: Weight, codes: torch.Tensor, scale: torch.Tensor, kind: int = ACT_INT4, algo: int = ALGO_AUTO,
           Y=None, want_acc: bool = False, acc=None, workspace=None, stream=None):
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.is_contiguous() and codes.shape[1] == w.K
    assert scale.dtype == torch.float32
    M = codes.shape[0]
    Y = Y if Y is not None else torch.empty(M, w.N, dtype=torch.float32, device=codes.device)
    if want_acc and acc is None:
        acc = torch.empty(M, w.N, dtype=torch.int32, device=codes.device)
    need = linear_workspace_bytes(w, M)
    if workspace is None and need:
        workspace = torch.zeros(need, dtype=torch.uint8, device=codes.device)  # the decode scratch starts zeroed
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().bitnet_a48_linear_ex(c_void_p(w.handle), _ptr(codes), _ptr(scale), M, kind, algo, _ptr(Y), _ptr(acc),
                                      _ptr(workspace), ws_bytes, _stream(stream)), "linear")
    return (Y, acc) if want_acc else Y


def linear_multi_workspace_bytes(ws, M: int) -> int:
    arr = (c_void_p * len(ws))(*[c_void_p(w.handle) for w in ws])
    return int(lib().bitnet_a48_linear_multi_workspace_bytes(len(ws), arr, M))


def linear_multi(ws, codes: torch.Tensor, scale: torch.Tensor, kind: int = ACT_INT4, Ys=None, workspace=None, stream=None):
    """Several BitLinears (one K) on the same codes; one fused launch for M <= 8.  Returns the list of outputs."""
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.is_contiguous() and codes.shape[1] == ws[0].K
    M = codes.shape[0]
    if Ys is None:
        Ys = [torch.empty(M, w.N, dtype=torch.float32, device=codes.device) for w in ws]
    need = linear_multi_workspace_bytes(ws, M)
    if workspace is None and need:
        workspace = torch.zeros(need, dtype=torch.uint8, device=codes.device)
    warr = (c_void_p * len(ws))(*[c_void_p(w.handle) for w in ws])
    yarr = (c_void_p * len(ws))(*[_ptr(y) for y in Ys])
    _check(lib().bitnet_a48_linear_multi(len(ws), warr, _ptr(codes), _ptr(scale), M, kind, yarr, _ptr(workspace),
                                         workspace.numel() if workspace is not None else 0, _stream(stream)), "linear_multi")
    return Ys


def linear_decode_static(w: Weight, codes: torch.Tensor, scale: torch.Tensor, Y: torch.Tensor, stream=None):
    """Decode BitLinear with the library's built-in scratch: allocates nothing, Y must be passed in."""
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.is_contiguous() and codes.shape[1] == w.K
    assert Y.is_cuda and Y.dtype == torch.float32 and Y.is_contiguous() and tuple(Y.shape) == (codes.shape[0], w.N)
    _check(lib().bitnet_a48_linear_decode_static(c_void_p(w.handle), _ptr(codes), _ptr(scale), codes.shape[0], _ptr(Y),
                                                 _stream(stream)), "linear_decode_static")
    return Y


def ffn_gate_first(gate: Weight, up: Weight, down: Weight, X: torch.Tensor, k_down: int, eps: float = 1e-5, Y=None,
                   want_inter: bool = False, want_rows: bool = False, workspace=None, stream=None):
    """Gate-first feed-forward sub-layer for up to 8 tokens.  Returns Y, or (Y, inter, rows_fetched) parts on request."""
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.shape[1] == gate.K
    M = X.shape[0]
    Y = Y if Y is not None else torch.empty(M, down.N, dtype=torch.float32, device=X.device)
    inter = torch.empty(M, gate.N, dtype=torch.float32, device=X.device) if want_inter else None
    rows = torch.zeros(4, dtype=torch.int32, device=X.device) if want_rows else None
    if workspace is None:
        need = int(lib().bitnet_a48_ffn_gate_first_workspace_bytes(c_void_p(gate.handle), c_void_p(up.handle),
                                                                   c_void_p(down.handle), M))
        workspace = torch.empty(need, dtype=torch.uint8, device=X.device)
    _check(lib().bitnet_a48_ffn_gate_first(c_void_p(gate.handle), c_void_p(up.handle), c_void_p(down.handle), _ptr(X), M,
                                           k_down, eps, _ptr(Y), _ptr(inter), _ptr(rows), _ptr(workspace),
                                           workspace.numel(), _stream(stream)), "ffn_gate_first")
    if want_inter or want_rows:
        return Y, inter, rows
    return Y


def ffn_workspace_bytes(gate: Weight, up: Weight, down: Weight, M: int) -> int:
    return int(lib().bitnet_a48_ffn_gate_first_workspace_bytes(c_void_p(gate.handle), c_void_p(up.handle),
                                                               c_void_p(down.handle), M))


def ffn_dense(gate: Weight, up: Weight, down: Weight, X: torch.Tensor, k_down: int, eps: float = 1e-5, Y=None,
              workspace=None, stream=None):
    """The feed-forward sub-layer for up to 8 tokens evaluated densely (the comparison point of ffn_gate_first)."""
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.shape[1] == gate.K
    M = X.shape[0]
    Y = Y if Y is not None else torch.empty(M, down.N, dtype=torch.float32, device=X.device)
    if workspace is None:
        workspace = torch.empty(ffn_workspace_bytes(gate, up, down, M), dtype=torch.uint8, device=X.device)
    _check(lib().bitnet_a48_ffn_dense(c_void_p(gate.handle), c_void_p(up.handle), c_void_p(down.handle), _ptr(X), M,
                                      k_down, eps, _ptr(Y), _ptr(workspace), workspace.numel(), _stream(stream)),
           "ffn_dense")
    return Y


def bitlinear_host_workspace_bytes(w: Weight, M: int) -> int:
    return int(lib().bitnet_a48_bitlinear_host_workspace_bytes(c_void_p(w.handle), M))


def bitlinear_host(w: Weight, X_host: torch.Tensor, Y_host: torch.Tensor, kind: int, k: int, eps: float,
                   workspace: torch.Tensor, stream=None):
    """X_host / Y_host: CPU fp32 tensors (ideally pinned)."""
    assert not X_host.is_cuda and not Y_host.is_cuda and X_host.is_contiguous() and Y_host.is_contiguous()
    M = X_host.shape[0]
    _check(lib().bitnet_a48_bitlinear_host(c_void_p(w.handle), _ptr(X_host), M, kind, k, eps, _ptr(Y_host),
                                           _ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _stream(stream)), "bitlinear_host")
    return Y_host


def bitlinear_host_async(w: Weight, X_host: torch.Tensor, Y_host: torch.Tensor, kind: int, k: int, eps: float,
                         workspace: torch.Tensor, stream=None):
    """As bitlinear_host, but only enqueues: synchronise the stream before reading Y_host."""
    assert not X_host.is_cuda and not Y_host.is_cuda and X_host.is_contiguous() and Y_host.is_contiguous()
    _check(lib().bitnet_a48_bitlinear_host_async(c_void_p(w.handle), _ptr(X_host), X_host.shape[0], kind, k, eps,
                                                 _ptr(Y_host), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                 _stream(stream)), "bitlinear_host_async")
    return Y_host


class Block:
    """Owns a ``bitnet_a48_block`` handle and keeps its borrowed weights and gains alive."""

    ORDER = ("q", "k", "v", "o", "gate", "up", "down")

    def __init__(self, weights: dict, g_attn: torch.Tensor, g_ffn: torch.Tensor, *, n_heads: int, k_o: int,
                 k_down: int, ctx_cap: int = 0, norm_eps: float = 1e-5, quant_eps: float = 1e-5,
                 rope_base: float = 10000.0, act_fp4: bool = False, q_bits: int = 0, kv_bits: int = 0):
        self.weights, self.g_attn, self.g_ffn = weights, g_attn, g_ffn
        H, F = weights["q"].N, weights["gate"].N
        self.cfg = BlockConfig(H, n_heads, F, k_o, k_down, ctx_cap, norm_eps, quant_eps, rope_base, int(act_fp4),
                               q_bits, kv_bits)
        arr = (c_void_p * 7)(*[c_void_p(weights[n].handle) for n in self.ORDER])
        out = c_void_p(0)
        _check(lib().bitnet_a48_block_create(byref(self.cfg), arr, _ptr(g_attn), _ptr(g_ffn), byref(out)),
               "block_create")
        self.handle = out.value

    def free(self):
        if self.handle:
            lib().bitnet_a48_block_free(c_void_p(self.handle))
            self.handle = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    def kv_cache_bytes(self, B: int) -> int:
        """Bytes of one cache buffer (keys or values) for B sequences; packed when kv_bits != 0."""
        return int(lib().bitnet_a48_kv_cache_bytes(c_void_p(self.handle), B))

    def workspace_bytes(self, B: int, T: int) -> int:
        return int(lib().bitnet_a48_block_workspace_bytes(c_void_p(self.handle), B, T))

    def forward(self, X: torch.Tensor, B: int, T: int, pos0: int = 0, kcache=None, vcache=None, Y=None,
                workspace=None, stream=None) -> torch.Tensor:
        assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.shape[0] == B * T
        Y = Y if Y is not None else torch.empty_like(X)
        if workspace is None:
            workspace = torch.empty(self.workspace_bytes(B, T), dtype=torch.uint8, device=X.device)
        _check(lib().bitnet_a48_block_forward(c_void_p(self.handle), _ptr(X), B, T, pos0, _ptr(kcache), _ptr(vcache),
                                              _ptr(Y), _ptr(workspace), workspace.numel(), _stream(stream)),
               "block_forward")
        return Y


def attention_prefill_workspace_bytes(B: int, n_heads: int, head_dim: int, T: int, n_keys: int) -> int:
    return int(lib().bitnet_a48_attention_prefill_workspace_bytes(B, n_heads, head_dim, T, n_keys))


def attention_prefill(q: torch.Tensor, kcache: torch.Tensor, vcache: torch.Tensor, B: int, T: int, pos0: int = 0, out=None,
                      workspace=None, stream=None) -> torch.Tensor:
    """Causal softmax attention of a prefill.  q fp32 [B*T, n_heads*head_dim] (rotated), caches fp32 [B, n_heads, cap, head_dim]."""
    _, n_heads, cap, hd = kcache.shape
    if out is None:
        out = torch.empty_like(q)
    need = attention_prefill_workspace_bytes(B, n_heads, hd, T, pos0 + T)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    _check(lib().bitnet_a48_attention_prefill(_ptr(q), _ptr(kcache), _ptr(vcache), B, T, n_heads, hd, pos0, cap, _ptr(out),
                                              _ptr(workspace), workspace.numel(), _stream(stream)), "attention_prefill")
    return out


def kernel_status():
    words = (c_uint * 4)()
    _check(lib().bitnet_a48_kernel_status(words), "kernel_status")
    return list(words)
