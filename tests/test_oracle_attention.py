"""Pins of the oracle's stand-alone attention (Section 2.1): closed forms and invariants, no GPU."""
import numpy as np



def _random_case(B, T, NH, hd, pos0, cap, seed):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B * T, NH * hd))
    kc = rng.standard_normal((B, NH, cap, hd))
    vc = rng.standard_normal((B, NH, cap, hd))
    return q, kc, vc


def test_two_keys_closed_form(oracle):
    # q = sqrt(d) e1, k1 = a e1, k2 = b e1: the scaled scores are exactly a and b, so the weights are the logistic
    # function of a - b; with a - b = ln 3 they are 3/4 and 1/4.  (A missing 1/sqrt(d), a transposed product or a
    # sign error all move them.)
    hd = 16
    q = np.zeros((2, hd)); q[1, 0] = np.sqrt(hd); q[0, 0] = 1.0
    kc = np.zeros((1, 1, 2, hd)); kc[0, 0, 0, 0] = np.log(3.0) + 0.5; kc[0, 0, 1, 0] = 0.5
    vc = np.zeros((1, 1, 2, hd)); vc[0, 0, 0] = np.arange(hd); vc[0, 0, 1] = -2.0 * np.arange(hd)
    out = oracle.attention_causal(q, kc, vc, B=1, T=2, n_heads=1)
    np.testing.assert_allclose(out[0], vc[0, 0, 0], rtol=0, atol=1e-14)  # the first token sees only itself
    np.testing.assert_allclose(out[1], 0.75 * vc[0, 0, 0] + 0.25 * vc[0, 0, 1], rtol=1e-14, atol=1e-14)


def test_equal_keys_give_running_mean_of_values(oracle):
    B, T, NH, hd, pos0, cap = 2, 5, 3, 8, 4, 12
    q, kc, vc = _random_case(B, T, NH, hd, pos0, cap, 1)
    kc[:] = kc[:, :, :1]  # every position has the same key: uniform weights over the visible positions
    out = oracle.attention_causal(q, kc, vc, B=B, T=T, n_heads=NH, pos0=pos0)
    for b in range(B):
        for h in range(NH):
            for t in range(T):
                want = vc[b, h, :pos0 + t + 1].mean(axis=0)
                np.testing.assert_allclose(out[b * T + t, h * hd:(h + 1) * hd], want, rtol=1e-13, atol=1e-13)


def test_causal_mask_and_unused_cache_rows(oracle):
    B, T, NH, hd, pos0, cap = 1, 6, 2, 4, 3, 16
    q, kc, vc = _random_case(B, T, NH, hd, pos0, cap, 2)
    base = oracle.attention_causal(q, kc, vc, B=B, T=T, n_heads=NH, pos0=pos0)
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[:, :, pos0 + 3:] += 5.0  # positions after the fourth new token, and the rows past pos0 + T
    vc2[:, :, pos0 + 3:] -= 7.0
    moved = oracle.attention_causal(q, kc2, vc2, B=B, T=T, n_heads=NH, pos0=pos0)
    assert np.array_equal(base[:3], moved[:3])      # tokens 0..2 do not see positions >= pos0 + 3
    assert not np.allclose(base[3:], moved[3:])


def test_cached_prefix_equals_the_tail_of_a_full_pass(oracle):
    B, NH, hd, full, pos0 = 2, 2, 8, 9, 5
    T = full - pos0
    rng = np.random.default_rng(3)
    q_full = rng.standard_normal((B * full, NH * hd))
    kc = rng.standard_normal((B, NH, full, hd)); vc = rng.standard_normal((B, NH, full, hd))
    whole = oracle.attention_causal(q_full, kc, vc, B=B, T=full, n_heads=NH).reshape(B, full, -1)
    q_tail = q_full.reshape(B, full, -1)[:, pos0:].reshape(B * T, -1)
    tail = oracle.attention_causal(q_tail, kc, vc, B=B, T=T, n_heads=NH, pos0=pos0).reshape(B, T, -1)
    np.testing.assert_allclose(tail, whole[:, pos0:], rtol=1e-13, atol=1e-13)


def test_saturated_scores_pick_the_best_key(oracle):
    # keys far apart along q: the weights collapse onto the largest score, the output is that key's value
    hd, n = 8, 6
    q = np.zeros((n, hd)); q[:, 0] = 1.0
    kc = np.zeros((1, 1, n, hd)); kc[0, 0, :, 0] = np.array([3.0, -1.0, 7.0, 2.0, 9.0, 0.0]) * 400.0
    vc = np.arange(n * hd, dtype=np.float64).reshape(1, 1, n, hd)
    out = oracle.attention_causal(q, kc, vc, B=1, T=n, n_heads=1)
    best = [0, 0, 2, 2, 4, 4]
    for t in range(n):
        np.testing.assert_allclose(out[t], vc[0, 0, best[t]], rtol=1e-12, atol=1e-12)


def test_heads_and_sequences_are_independent(oracle):
    B, T, NH, hd = 2, 4, 3, 4
    q, kc, vc = _random_case(B, T, NH, hd, 0, T, 4)
    out = oracle.attention_causal(q, kc, vc, B=B, T=T, n_heads=NH)
    b, h = 1, 2
    alone = oracle.attention_causal(q[b * T:(b + 1) * T, h * hd:(h + 1) * hd], kc[b:b + 1, h:h + 1], vc[b:b + 1, h:h + 1],
                                    B=1, T=T, n_heads=1)
    np.testing.assert_allclose(out[b * T:(b + 1) * T, h * hd:(h + 1) * hd], alone, rtol=1e-14, atol=1e-14)
