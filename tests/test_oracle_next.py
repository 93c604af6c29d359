"""Pins for the oracle functions of the rows beyond the first BitLinear path: the floating-point variant of the
block (Section 2.3), low-bit attention (Section 3) and gate-first evaluation of the feed-forward sub-layer
(Section 2.1, paragraph after Eq. 5).  The paper prints no formula for the head quantiser beyond "unsigned integers
using the absmax function", so its pins are what any absmax quantiser of b bits must satisfy; the other two are
pinned to independent derivations."""
import math

import numpy as np
import pytest

from conftest import golden
from paper_2411_04965_b200 import synth
from test_oracle_block import F, H, HD, NH, T, _bitlinear, _inputs, _rmsnorm, _rope, _weights


# ---------------------------------------------------------------------------------------------- low-bit attention
@pytest.mark.parametrize("bits", [3, 4, 8])
def test_head_quantiser_is_absmax_with_nearest_levels(oracle, bits):
    L = 2 ** (bits - 1) - 1
    x = synth.student_t3(64, 128, seed=bits).numpy()
    q, d = oracle.quant_heads(x, bits, eps=0.0)
    assert q.min() >= -L and q.max() <= L  # the clip at -(L+1) never fires
    gamma = np.abs(x).max(1).astype(np.float64)
    assert np.allclose(d, gamma / L, rtol=1e-15)
    assert (np.abs(q).max(1) == L).all()  # the maximum takes the top code
    # brute force: every code is the nearest of the 2L+1 levels gamma/L * j (ties aside)
    levels = (d[:, None] * np.arange(-L, L + 1)[None, :])  # [M, 2L+1]
    nearest = np.abs(x[:, :, None].astype(np.float64) - levels[:, None, :]).argmin(-1) - L
    frac = x.astype(np.float64) / d[:, None]
    tie = np.abs(np.abs(frac - np.floor(frac)) - 0.5) < 1e-9
    assert np.array_equal(q[~tie], nearest[~tie])
    # error bound of a uniform quantiser with step gamma/L
    assert (np.abs(x - d[:, None] * q) <= d[:, None] / 2 * (1 + 1e-12)).all()
    # as unsigned integers (code + L + 1) they fit `bits` bits
    stored = q.astype(np.int64) + L + 1
    assert stored.min() >= 1 and stored.max() <= 2 ** bits - 1


def test_head_quantiser_is_eq3_at_eight_bits(oracle):
    # with 8 bits the head quantiser is Eq. 3 itself: same codes and scale as the INT8 quantiser with every entry kept
    x = synth.student_t3(16, 96, seed=1).numpy()
    q, d = oracle.quant_heads(x, 8, eps=1e-5)
    c, d8, _ = oracle.topk_quant_int8(x, 96, eps=1e-5)
    assert np.array_equal(q, c) and np.array_equal(d, d8)


def test_head_quantiser_scale_invariance_and_zero(oracle):
    x = synth.student_t3(8, 64, seed=2).numpy()
    q1, d1 = oracle.quant_heads(x, 4, eps=0.0)
    q2, d2 = oracle.quant_heads(x * 8.0, 4, eps=0.0)  # a power of two: exact
    assert np.array_equal(q1, q2) and np.array_equal(d1 * 8.0, d2)
    q0, d0 = oracle.quant_heads(np.zeros((1, 64), np.float32), 3)
    assert not q0.any() and d0[0] == 0.0


def _numpy_block_lowbit(oracle, x, w, g1, g2, k_o, k_down, q_bits, kv_bits, fp4):
    """Independent derivation of the block with the options: dequantise-then-float matmuls, numpy attention."""
    def dense(a, W):
        if not fp4:
            return _bitlinear(oracle, a, W, "int4")
        t, alpha = oracle.ternarise(W)
        g, d = oracle.quant_fp4(a)
        return (d[:, None] * g.astype(np.float64)) @ (alpha * t.astype(np.float64)).T

    def heads(z, bits, bos_rule):  # z [T, NH, HD]
        out = np.empty_like(z)
        for t_ in range(z.shape[0]):
            use = 4 if (bos_rule and bits == 3 and t_ == 0) else bits
            L = 2 ** (use - 1) - 1
            gamma = np.abs(z[t_]).max(-1, keepdims=True)
            codes = np.clip(np.rint(z[t_] * (L / (gamma + 1e-5))), -(L + 1), L)
            out[t_] = codes * (gamma / L)
        return out

    a = _rmsnorm(x, g1)
    q = dense(a, w["q"]).reshape(T, NH, HD)
    k = dense(a, w["k"]).reshape(T, NH, HD)
    v = dense(a, w["v"]).reshape(T, NH, HD)
    pos = np.arange(T, dtype=np.float64)
    q, k = _rope(q, pos), _rope(k, pos)
    if q_bits:
        q = heads(q, q_bits, False)
    if kv_bits:
        k, v = heads(k, kv_bits, True), heads(v, kv_bits, True)
    att = np.zeros((T, NH, HD))
    for h in range(NH):
        s = q[:, h] @ k[:, h].T / math.sqrt(HD)
        s = np.where(np.tril(np.ones((T, T), bool)), s, -np.inf)
        p = np.exp(s - s.max(-1, keepdims=True))
        att[:, h] = (p / p.sum(-1, keepdims=True)) @ v[:, h]
    att = att.reshape(T, H).astype(np.float32)
    o = dense(att, w["o"]) if fp4 else _bitlinear(oracle, att, w["o"], "topk", k_o)
    h1 = x.astype(np.float64) + o
    f = _rmsnorm(h1, g2)
    inter = (dense(f, w["up"]) * np.maximum(dense(f, w["gate"]), 0.0) ** 2).astype(np.float32)
    return h1 + _bitlinear(oracle, inter, w["down"], "topk", k_down), k, v


@pytest.mark.parametrize("q_bits,kv_bits,fp4", [(0, 4, False), (4, 4, False), (4, 3, False), (0, 0, True), (4, 3, True)])
def test_block_options_match_float_derivation(oracle, q_bits, kv_bits, fp4):
    w = _weights(7, scale=25.0)
    x, g1, g2 = _inputs(7)
    out, k_new, v_new = oracle.block_forward(x, w, g1, g2, n_heads=NH, B=1, T=T, k_o=H // 2, k_down=F // 2,
                                             q_bits=q_bits, kv_bits=kv_bits, act_fp4=fp4)
    ref, k_ref, v_ref = _numpy_block_lowbit(oracle, x, w, g1, g2, H // 2, F // 2, q_bits, kv_bits, fp4)
    assert np.abs(out - ref).max() <= 1e-9 * np.abs(ref).max()
    assert np.allclose(k_new[0].transpose(1, 0, 2), k_ref, rtol=1e-12, atol=1e-15)
    assert np.allclose(v_new[0].transpose(1, 0, 2), v_ref, rtol=1e-12, atol=1e-15)
    plain, _, _ = oracle.block_forward(x, w, g1, g2, n_heads=NH, B=1, T=T, k_o=H // 2, k_down=F // 2)
    assert not np.array_equal(out, plain)  # the option is not a no-op


def test_three_bit_cache_keeps_the_bos_heads_at_four_bits(oracle):
    w = _weights(8, scale=25.0)
    x, g1, g2 = _inputs(8)
    kw = dict(n_heads=NH, B=1, T=T, k_o=H // 2, k_down=F // 2)
    _, k3, v3 = oracle.block_forward(x, w, g1, g2, kv_bits=3, **kw)
    _, k4, v4 = oracle.block_forward(x, w, g1, g2, kv_bits=4, **kw)
    assert np.array_equal(k3[:, :, 0], k4[:, :, 0]) and np.array_equal(v3[:, :, 0], v4[:, :, 0])  # position 0
    assert not np.array_equal(k3[:, :, 1:], k4[:, :, 1:])
    # 3-bit heads take at most 7 distinct values per head vector, 4-bit ones at most 15
    assert max(len(np.unique(k3[0, h, t])) for h in range(NH) for t in range(1, T)) <= 7
    assert max(len(np.unique(k4[0, h, t])) for h in range(NH) for t in range(T)) <= 15


# ---------------------------------------------------------------------------------------------- gate-first FFN
def test_gate_first_ffn_equals_the_dense_evaluation(oracle):
    Hs, Fs, M = 96, 160, 5
    lat = {n: synth.latent_weights(a, b, seed=40 + i).numpy() * 25.0
           for i, (n, a, b) in enumerate((("gate", Fs, Hs), ("up", Fs, Hs), ("down", Hs, Fs)))}
    (tg, ag), (tu, au), (td, ad) = (oracle.ternarise(lat[n]) for n in ("gate", "up", "down"))
    x = synth.gaussian_outlier_activations(M, Hs, seed=41, count=2).numpy()
    y, active = oracle.ffn_gate_first(x, tg, ag, tu, au, td, ad, Fs // 2)
    # dense evaluation from the separately pinned pieces: Eq. 7, Eq. 6, Eq. 5, Eq. 1 + 3
    q, d = oracle.quant_int4(x)
    _, gate = oracle.linear(q, d, tg, ag)
    _, up = oracle.linear(q, d, tu, au)
    inter = (up * np.maximum(gate, 0.0) ** 2).astype(np.float32)
    c, d8, _ = oracle.topk_quant_int8(inter, Fs // 2)
    _, y_dense = oracle.linear(c, d8, td, ad)
    assert np.array_equal(y, y_dense)  # skipping rows whose gate is zero changes nothing, bit for bit
    assert np.array_equal(active.astype(bool), np.maximum(gate, 0.0) ** 2 != 0.0)
    assert 0.2 < active.mean() < 0.8  # random gates: about half of the up rows are needed
    # a gate that is never positive needs no up row at all and gives an exact zero
    y1, a1 = oracle.ffn_gate_first(np.abs(x), -np.abs(tg), ag, tu, au, td, ad, Fs // 2)
    assert not a1.any() and not y1.any()


def test_up_projection_sparsity_identity_of_the_paper():
    # Section 3 "Sparsity": rows of W_up are skipped where the gate is zero, columns where the INT4 input is zero
    g = golden("sparsity_text.txt")
    assert abs(100 * (1 - (1 - g["up_in"][0] / 100) * (1 - g["gate_out"][0] / 100)) - g["up"][0]) < 0.06
