"""ctypes front end of the CPU oracle (test infrastructure, not the product).

Compiles ``oracle_a48.cpp`` with g++ on first use and exposes its entry points
on numpy arrays.  Only tests, the smoke check and the benchmark's CPU-baseline
leg may import this module; the CUDA library never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_a48.cpp")
_LIB = os.path.join(_HERE, "liboracle_a48.so")
_lib = None

_i64 = ctypes.c_int64
_f64 = ctypes.c_double


class BlockParams(ctypes.Structure):
    _fields_ = [
        ("hidden", _i64), ("n_heads", _i64), ("head_dim", _i64), ("ffn", _i64),
        ("B", _i64), ("T", _i64), ("pos0", _i64), ("ctx_cap", _i64),
        ("k_o", _i64), ("k_down", _i64),
        ("norm_eps", _f64), ("quant_eps", _f64), ("rope_base", _f64),
        ("act_fp4", _i64), ("q_bits", _i64), ("kv_bits", _i64),
    ]


def build(force: bool = False) -> str:
    """Compile the oracle shared library (g++ only); returns its path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", "-ffp-contract=off", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty)) if a is not None else None


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def ternarise(W, eps=1e-5):
    """Eq. 2.  Returns (codes int8 [N,K], alpha float64)."""
    W = _f32(W)
    N, K = W.shape
    t = np.empty((N, K), np.int8)
    alpha = _f64(0.0)
    rc = _load().oracle_a48_ternarise(_p(W, ctypes.c_float), _i64(N), _i64(K), _f64(eps), _p(t, ctypes.c_int8),
                                      ctypes.byref(alpha))
    assert rc == 0, rc
    return t, alpha.value


def quant_int4(X, eps=1e-5, nthreads=1):
    """Eq. 7.  Returns (codes int8 [M,K] in [-8,7], scale float64 [M] = beta/sqrt7)."""
    X = _f32(X)
    M, K = X.shape
    q = np.empty((M, K), np.int8)
    d = np.empty(M, np.float64)
    rc = _load().oracle_a48_quant_int4(_p(X, ctypes.c_float), _i64(M), _i64(K), _f64(eps), _p(q, ctypes.c_int8),
                                       _p(d, _f64), ctypes.c_int(nthreads))
    assert rc == 0, rc
    return q, d


def topk_quant_int8(X, k, eps=1e-5, nthreads=1):
    """Eq. 1 and 3.  Returns (codes int8 [M,K], scale float64 [M] = gamma/127, mask uint8 [M,K])."""
    X = _f32(X)
    M, K = X.shape
    c = np.empty((M, K), np.int8)
    d = np.empty(M, np.float64)
    mask = np.empty((M, K), np.uint8)
    rc = _load().oracle_a48_topk_quant_int8(_p(X, ctypes.c_float), _i64(M), _i64(K), _i64(k), _f64(eps),
                                            _p(c, ctypes.c_int8), _p(d, _f64), _p(mask, ctypes.c_uint8),
                                            ctypes.c_int(nthreads))
    assert rc == 0, rc
    return c, d, mask


def quant_fp4(X, nthreads=1):
    """Eq. 8-9 (E2M1).  Returns (grid codes int8 in {0,±1,±2,±3,±4,±6,±8,±12}, scale float64 [M] = |x|max/12)."""
    X = _f32(X)
    M, K = X.shape
    g = np.empty((M, K), np.int8)
    d = np.empty(M, np.float64)
    rc = _load().oracle_a48_quant_fp4(_p(X, ctypes.c_float), _i64(M), _i64(K), _p(g, ctypes.c_int8), _p(d, _f64),
                                      ctypes.c_int(nthreads))
    assert rc == 0, rc
    return g, d


def compact_codes(codes):
    """Section 2.1 / Eq. 1: per row the channels whose code is non-zero, ascending, with their codes.

    Returns a list of (idx int64 array, val int8 array), one pair per row.  The definition written out."""
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    out = []
    for row in codes:
        idx = np.flatnonzero(row != 0)
        out.append((idx.astype(np.int64), row[idx].copy()))
    return out


def linear_from_lists(lists, scale, t, alpha):
    """Eq. 1 evaluated over the compacted rows only: acc[m, n] = sum over listed channels of code * t[n, channel]."""
    t = np.ascontiguousarray(t, dtype=np.int8).astype(np.int64)
    scale = np.ascontiguousarray(scale, dtype=np.float64)
    acc = np.zeros((len(lists), t.shape[0]), np.int64)
    for m, (idx, val) in enumerate(lists):
        for j, c in zip(idx.tolist(), val.tolist()):
            acc[m] += int(c) * t[:, j]
    return acc, acc.astype(np.float64) * scale[:, None] * float(alpha)


def linear(codes, scale, t, alpha, nthreads=1, want_acc=True, want_y=True):
    """Eq. 1 / Eq. 6.  Returns (acc int64 [M,N] or None, y float64 [M,N] or None)."""
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    t = np.ascontiguousarray(t, dtype=np.int8)
    scale = np.ascontiguousarray(scale, dtype=np.float64)
    M, K = codes.shape
    N, K2 = t.shape
    assert K == K2
    acc = np.empty((M, N), np.int64) if want_acc else None
    y = np.empty((M, N), np.float64) if want_y else None
    rc = _load().oracle_a48_linear(_p(codes, ctypes.c_int8), _p(scale, _f64), _i64(M), _p(t, ctypes.c_int8),
                                   _f64(alpha), _i64(N), _i64(K), _p(acc, _i64), _p(y, _f64),
                                   ctypes.c_int(nthreads))
    assert rc == 0, rc
    return acc, y


def quant_heads(X, bits, eps=1e-5):
    """Section 3, low-bit attention: absmax quantisation of head vectors (rows of X) to `bits` bits.

    Returns (codes int8 [M, n] in [-(L+1), L] with L = 2^(bits-1) - 1, scale float64 [M] = gamma / L); the stored
    unsigned integer is code + L + 1."""
    X = _f32(X)
    M, n = X.shape
    q = np.empty((M, n), np.int8)
    d = np.empty(M, np.float64)
    rc = _load().oracle_a48_quant_heads(_p(X, ctypes.c_float), _i64(M), _i64(n), ctypes.c_int(bits), _f64(eps),
                                        _p(q, ctypes.c_int8), _p(d, _f64))
    assert rc == 0, rc
    return q, d


def ffn_gate_first(X, tg, ag, tu, au, td, ad, k_down, eps=1e-5):
    """Section 2.1 (after Eq. 5): gate projection first, up projection only where ReLU²(gate) != 0.

    X fp32 [M, H]; tg, tu int8 [F, H]; td int8 [H, F].  Returns (y float64 [M, H], active uint8 [M, F])."""
    X = _f32(X)
    M, H = X.shape
    F = tg.shape[0]
    tg, tu, td = (np.ascontiguousarray(t, dtype=np.int8) for t in (tg, tu, td))
    y = np.empty((M, H), np.float64)
    active = np.empty((M, F), np.uint8)
    rc = _load().oracle_a48_ffn_gate_first(_p(X, ctypes.c_float), _i64(M), _i64(H), _i64(F), _p(tg, ctypes.c_int8),
                                           _f64(ag), _p(tu, ctypes.c_int8), _f64(au), _p(td, ctypes.c_int8), _f64(ad),
                                           _i64(k_down), _f64(eps), _p(y, _f64), _p(active, ctypes.c_uint8))
    assert rc == 0, rc
    return y, active


def attention_causal(q, kcache, vcache, *, B, T, n_heads, pos0=0):
    """Causal softmax attention of the block (Section 2.1: the attention between the q/k/v BitLinears and the output
    BitLinear is the ordinary one), written out as its definition in float64.

    q [B*T, n_heads*head_dim] (already rotated); kcache, vcache [B, n_heads, cap, head_dim] holding positions
    0 .. pos0+T-1.  Token t of a sequence sits at position pos0 + t and sees positions 0 .. pos0 + t:
    out[t] = sum_j softmax_j(q[t] . k[j] / sqrt(head_dim)) v[j].  Returns float64 [B*T, n_heads*head_dim].
    """
    q = np.asarray(q, np.float64)
    kcache = np.asarray(kcache, np.float64)
    vcache = np.asarray(vcache, np.float64)
    H = q.shape[1]
    hd = H // n_heads
    assert q.shape[0] == B * T and kcache.shape[:2] == (B, n_heads) and kcache.shape[3] == hd
    out = np.empty((B * T, H), np.float64)
    position = pos0 + np.arange(T)[:, None]      # of each query
    key_index = np.arange(pos0 + T)[None, :]
    for b in range(B):
        for h in range(n_heads):
            Q = q[b * T:(b + 1) * T, h * hd:(h + 1) * hd]
            K = kcache[b, h, :pos0 + T]
            V = vcache[b, h, :pos0 + T]
            S = (Q @ K.T) / np.sqrt(float(hd))
            S = np.where(key_index <= position, S, -np.inf)
            P = np.exp(S - S.max(axis=1, keepdims=True))
            P /= P.sum(axis=1, keepdims=True)
            out[b * T:(b + 1) * T, h * hd:(h + 1) * hd] = P @ V
    return out


def block_forward(X, weights, g1, g2, *, n_heads, B, T, pos0=0, ctx_cap=0, kcache=None, vcache=None,
                  k_o, k_down, norm_eps=1e-5, quant_eps=1e-5, rope_base=10000.0, nthreads=1, act_fp4=False,
                  q_bits=0, kv_bits=0):
    """One transformer block.  ``weights`` = dict with fp32 latents q,k,v,o [H,H], gate,up [F,H], down [H,F].

    Returns (out float64 [B*T,H], k_new, v_new float64 [B,n_heads,T,head_dim]).
    act_fp4: the floating-point variant of Section 2.3.  q_bits / kv_bits: low-bit attention of Section 3 (k_new and
    v_new are then the dequantised heads; kcache / vcache hold dequantised values as well).
    """
    X = _f32(X)
    M, H = X.shape
    assert M == B * T
    F = weights["gate"].shape[0]
    w = {n: _f32(weights[n]) for n in ("q", "k", "v", "o", "gate", "up", "down")}
    g1 = _f32(g1)
    g2 = _f32(g2)
    hd = H // n_heads
    p = BlockParams(H, n_heads, hd, F, B, T, pos0, ctx_cap, k_o, k_down, norm_eps, quant_eps, rope_base,
                    int(act_fp4), q_bits, kv_bits)
    out = np.empty((M, H), np.float64)
    k_new = np.empty((B, n_heads, T, hd), np.float64)
    v_new = np.empty((B, n_heads, T, hd), np.float64)
    kc = _f32(kcache) if kcache is not None else None
    vc = _f32(vcache) if vcache is not None else None
    cf = ctypes.c_float
    rc = _load().oracle_a48_block_forward(ctypes.byref(p), _p(X, cf), _p(w["q"], cf), _p(w["k"], cf), _p(w["v"], cf),
                                          _p(w["o"], cf), _p(w["gate"], cf), _p(w["up"], cf), _p(w["down"], cf),
                                          _p(g1, cf), _p(g2, cf), _p(kc, cf), _p(vc, cf), _p(out, _f64),
                                          _p(k_new, _f64), _p(v_new, _f64), ctypes.c_int(nthreads))
    assert rc == 0, rc
    return out, k_new, v_new
