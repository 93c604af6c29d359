"""Pins for the oracle's transformer block (Section 2.1 layout, Eq. 5).

The paper fixes the sub-layer order, which projections take which quantiser,
and the ReLU²GLU formula; norm type, RoPE pairing and cache layout are this
build's reading (parity unpinned by the paper).  These tests check what is
fixed, plus invariants any correct block has (causality, cache consistency,
residual identity) and an independent dequantise-then-float-matmul derivation.
"""
import math

import numpy as np
import pytest

from paper_2411_04965_b200 import synth

H, NH, F, T = 64, 4, 96, 6
HD = H // NH


def _weights(seed=0, scale=1.0):
    names = (("q", H, H), ("k", H, H), ("v", H, H), ("o", H, H), ("gate", F, H), ("up", F, H), ("down", H, F))
    return {n: synth.latent_weights(a, b, seed=seed * 10 + i).numpy() * scale for i, (n, a, b) in enumerate(names)}


def _inputs(seed=0, B=1, T_=T):
    x = synth.gaussian_outlier_activations(B * T_, H, seed=seed, count=2).numpy()
    return x, synth.norm_gains(H, seed + 1).numpy(), synth.norm_gains(H, seed + 2).numpy()


def _rmsnorm(x, g, eps=1e-5):
    x = x.astype(np.float64)
    return (x / np.sqrt((x * x).mean(-1, keepdims=True) + eps) * g.astype(np.float64)).astype(np.float32)


def _bitlinear(oracle, a, W, kind, k=None):
    """BitLinear as dequantise-then-float-matmul (Eq. 1 / Eq. 6 read literally)."""
    t, alpha = oracle.ternarise(W)
    if kind == "int4":
        c, d = oracle.quant_int4(a)
    else:
        c, d, _ = oracle.topk_quant_int8(a, k)
    return (d[:, None] * c.astype(np.float64)) @ (alpha * t.astype(np.float64)).T


def _rope(z, pos):
    # z [T, NH, HD]; pairs (i, i+HD/2), angle pos * 10000^(-2i/HD)
    i = np.arange(HD // 2)
    ang = pos[:, None, None] * (10000.0 ** (-2.0 * i / HD))[None, None, :]
    lo, hi = z[..., : HD // 2], z[..., HD // 2:]
    return np.concatenate([lo * np.cos(ang) - hi * np.sin(ang), hi * np.cos(ang) + lo * np.sin(ang)], -1)


def _numpy_block(oracle, x, w, g1, g2, k_o, k_down):
    a = _rmsnorm(x, g1)
    q = _bitlinear(oracle, a, w["q"], "int4").reshape(T, NH, HD)
    k = _bitlinear(oracle, a, w["k"], "int4").reshape(T, NH, HD)
    v = _bitlinear(oracle, a, w["v"], "int4").reshape(T, NH, HD)
    pos = np.arange(T, dtype=np.float64)
    q, k = _rope(q, pos), _rope(k, pos)
    att = np.zeros((T, NH, HD))
    for h in range(NH):
        s = q[:, h] @ k[:, h].T / math.sqrt(HD)
        s = np.where(np.tril(np.ones((T, T), bool)), s, -np.inf)
        p = np.exp(s - s.max(-1, keepdims=True))
        att[:, h] = (p / p.sum(-1, keepdims=True)) @ v[:, h]
    att = att.reshape(T, H).astype(np.float32)
    h1 = x.astype(np.float64) + _bitlinear(oracle, att, w["o"], "topk", k_o)
    f = _rmsnorm(h1, g2)
    gate = _bitlinear(oracle, f, w["gate"], "int4")
    up = _bitlinear(oracle, f, w["up"], "int4")
    inter = (up * np.maximum(gate, 0.0) ** 2).astype(np.float32)  # Eq. 5
    return h1 + _bitlinear(oracle, inter, w["down"], "topk", k_down)


def test_block_matches_float_derivation(oracle):
    # weights scaled up so that every sub-layer contributes visibly to the output
    w = _weights(1, scale=25.0)
    x, g1, g2 = _inputs(1)
    out, _, _ = oracle.block_forward(x, w, g1, g2, n_heads=NH, B=1, T=T, k_o=H // 2, k_down=F // 2)
    ref = _numpy_block(oracle, x, w, g1, g2, H // 2, F // 2)
    assert np.abs(out - x).max() > 0.1 * np.abs(x).max()  # the sub-layers are not negligible
    assert np.abs(out - ref).max() <= 1e-9 * np.abs(ref).max()


def test_block_zero_output_projections_is_identity(oracle):
    w = _weights(2)
    w["o"] = np.zeros_like(w["o"])
    w["down"] = np.zeros_like(w["down"])
    x, g1, g2 = _inputs(2)
    out, _, _ = oracle.block_forward(x, w, g1, g2, n_heads=NH, B=1, T=T, k_o=H // 2, k_down=F // 2)
    assert np.array_equal(out, x.astype(np.float64))


def test_block_single_token_attention_is_value(oracle):
    # T = 1, no cache: softmax over one key is 1, RoPE at position 0 is the identity,
    # so the attention output equals the v projection and k_new the k projection.
    w = _weights(3, scale=25.0)
    x, g1, g2 = _inputs(3, T_=1)
    out, k_new, v_new = oracle.block_forward(x, w, g1, g2, n_heads=NH, B=1, T=1, k_o=H // 2, k_down=F // 2)
    a = _rmsnorm(x, g1)
    v = _bitlinear(oracle, a, w["v"], "int4")
    k = _bitlinear(oracle, a, w["k"], "int4")
    assert np.allclose(v_new.reshape(1, H), v, rtol=1e-12, atol=1e-15)
    assert np.allclose(k_new.reshape(1, H), k, rtol=1e-12, atol=1e-15)
    h1 = x + _bitlinear(oracle, v.astype(np.float32), w["o"], "topk", H // 2)
    f = _rmsnorm(h1, g2)
    inter = _bitlinear(oracle, f, w["up"], "int4") * np.maximum(_bitlinear(oracle, f, w["gate"], "int4"), 0) ** 2
    ref = h1 + _bitlinear(oracle, inter.astype(np.float32), w["down"], "topk", F // 2)
    assert np.abs(out - ref).max() <= 1e-9 * np.abs(ref).max()


def test_block_is_causal_and_batched(oracle):
    w = _weights(4, scale=25.0)
    x, g1, g2 = _inputs(4, B=2)
    kw = dict(n_heads=NH, k_o=H // 2, k_down=F // 2)
    out, _, _ = oracle.block_forward(x, w, g1, g2, B=2, T=T, **kw)
    # batches are independent
    o0, _, _ = oracle.block_forward(x[:T], w, g1, g2, B=1, T=T, **kw)
    o1, _, _ = oracle.block_forward(x[T:], w, g1, g2, B=1, T=T, **kw)
    assert np.array_equal(out[:T], o0) and np.array_equal(out[T:], o1)
    # changing later tokens leaves earlier outputs untouched
    x2 = x[:T].copy()
    x2[4:] += 3.0
    o2, _, _ = oracle.block_forward(x2, w, g1, g2, B=1, T=T, **kw)
    assert np.array_equal(o2[:4], o0[:4]) and not np.array_equal(o2[4:], o0[4:])


def test_block_cache_consistency(oracle):
    # Prefill T tokens, then redo the last token alone against the cache of the first T-1.
    w = _weights(5, scale=25.0)
    x, g1, g2 = _inputs(5)
    kw = dict(n_heads=NH, k_o=H // 2, k_down=F // 2)
    out, k_new, v_new = oracle.block_forward(x, w, g1, g2, B=1, T=T, **kw)
    cap = 8
    kc = np.zeros((1, NH, cap, HD), np.float32)
    vc = np.zeros((1, NH, cap, HD), np.float32)
    kc[:, :, : T - 1] = k_new[:, :, : T - 1]
    vc[:, :, : T - 1] = v_new[:, :, : T - 1]
    o_last, k1, v1 = oracle.block_forward(x[T - 1:], w, g1, g2, B=1, T=1, pos0=T - 1, ctx_cap=cap, kcache=kc,
                                          vcache=vc, **kw)
    assert np.allclose(k1[0, :, 0], k_new[0, :, T - 1], rtol=1e-12, atol=1e-15)
    # the cache is fp32, so agreement is to fp32 rounding of k/v (a quantiser flip would show as ~1e-2)
    assert np.abs(o_last[0] - out[T - 1]).max() <= 2e-4 * np.abs(out[T - 1]).max()
