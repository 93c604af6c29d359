"""Pins the CPU oracle to what the paper and the mathematics fix (no GPU needed).

Each test states the passage it checks.  The checks use closed forms, the
paper's printed Table 2 rates, brute force on tiny inputs and library routines
(numpy matmul / sort) that the oracle itself does not call.
"""
import math

import numpy as np
import pytest
import torch

from conftest import golden
from paper_2411_04965_b200 import synth


def _phi(z):  # standard normal CDF
    return 0.5 * (1.0 + math.erf(z / math.sqrt(2.0)))


# ----------------------------------------------------------------------------- Eq. 2 (ternary weights)
def test_ternarise_hand_vector(oracle):
    # alpha = (0.3+0.1+0.04+0.5)/4 = 0.235; W/alpha = 1.277, -0.426, 0.170, -2.128 -> 1, 0, 0, -1 (clipped)
    t, alpha = oracle.ternarise(np.array([[0.3, -0.1, 0.04, -0.5]], np.float32), eps=1e-5)
    assert t.tolist() == [[1, 0, 0, -1]]
    assert alpha == pytest.approx(0.235, rel=1e-6)


def test_ternarise_ties_round_half_to_even(oracle):
    # eps = 0 and mean|W| = 1 exactly, so W/alpha hits the exact ties 0.5, -0.5, 1.5
    W = np.array([[0.5, -0.5, 1.5, 1.5]], np.float32)  # mean|W| = 1.0
    t, alpha = oracle.ternarise(W, eps=0.0)
    assert alpha == 1.0
    assert t.tolist() == [[0, 0, 1, 1]]  # 0.5 -> 0 (even), 1.5 -> 2 -> clipped to 1
    # a strict round-half-away implementation would give [1, -1, 1, 1]


def test_ternarise_gaussian_rates(oracle):
    # For W ~ N(0, s^2): alpha = s*sqrt(2/pi); code 0 <=> |z| < 0.5*sqrt(2/pi)  =>  P(0) = 0.3101
    W = synth.latent_weights(1024, 1024, seed=11).numpy()
    t, alpha = oracle.ternarise(W)
    assert set(np.unique(t)) <= {-1, 0, 1}
    p0 = 2 * _phi(0.5 * math.sqrt(2 / math.pi)) - 1
    assert p0 == pytest.approx(0.3101, abs=2e-4)
    assert (t == 0).mean() == pytest.approx(p0, abs=2e-3)
    assert (t == 1).mean() == pytest.approx((1 - p0) / 2, abs=2e-3)
    assert alpha == pytest.approx(0.02 * math.sqrt(2 / math.pi), rel=5e-3)


def test_ternary_latents_survive(oracle):
    W = synth.ternary_latents(64, 96, seed=3).numpy()
    t, alpha = oracle.ternarise(W)
    assert np.array_equal(t, np.rint(W / 0.024).astype(np.int8))
    assert alpha == pytest.approx(0.016, rel=0.05)


# ----------------------------------------------------------------------------- Eq. 7 (INT4 absmean)
def test_int4_hand_vector(oracle):
    # beta = 1.5, sqrt7/beta = 1.7638: 1.76 -> 2, 3.53 -> 4; scale = 1.5/sqrt7
    q, d = oracle.quant_int4(np.array([[1, -1, 2, -2]], np.float32), eps=0.0)
    assert q.tolist() == [[2, -2, 4, -4]]
    assert d[0] == pytest.approx(1.5 / math.sqrt(7.0), rel=1e-15)


def test_int4_range_and_clip(oracle):
    x = synth.gaussian_outlier_activations(64, 1024, seed=1).numpy()
    q, d = oracle.quant_int4(x)
    assert q.min() == -8 and q.max() == 7  # the x20 outliers clip on both sides
    beta = np.abs(x.astype(np.float64)).mean(1)
    assert np.allclose(d, beta / math.sqrt(7.0), rtol=1e-14)


def test_int4_zero_rate_matches_table2(oracle):
    # Table 2 prints 12.0-12.1 % zeros for the INT4 inputs (QKV and Gate columns).  For Gaussian
    # inputs the quantiser of Eq. 7 gives P(code 0) = P(|z| < 0.5/(sqrt7*sqrt(2/pi)^-1)) = 0.1199.
    rows = golden("table2_sparsity.txt")
    printed = [rows[m][0] for m in rows] + [rows[m][3] for m in rows]
    assert min(printed) == 12.0 and max(printed) == 12.1
    thr = 0.5 * math.sqrt(2 / math.pi) / math.sqrt(7.0)
    closed = 2 * _phi(thr) - 1
    assert closed == pytest.approx(0.1199, abs=1e-4)
    g = torch.Generator().manual_seed(5)
    x = torch.randn(512, 4096, generator=g).numpy()
    q, _ = oracle.quant_int4(x, nthreads=4)
    rate = (q == 0).mean()
    assert rate == pytest.approx(closed, abs=1e-3)
    assert 0.1185 <= rate <= 0.1215  # rounds to the printed 12.0-12.1 %
    # tails: code +7 <=> z >= 6.5*thr*2; code -8 <=> z <= -7.5*thr*2
    assert (q == 7).mean() == pytest.approx(1 - _phi(6.5 * 2 * thr), abs=5e-4)
    assert (q == -8).mean() == pytest.approx(_phi(-7.5 * 2 * thr), abs=5e-4)
    assert 1 - _phi(6.5 * 2 * thr) == pytest.approx(0.0250, abs=1e-4)


def test_int4_error_bound_and_scale_invariance(oracle):
    g = torch.Generator().manual_seed(6)
    x = torch.randn(32, 512, generator=g).numpy()
    q, d = oracle.quant_int4(x, eps=0.0)
    inside = (q > -8) & (q < 7)
    err = np.abs(x.astype(np.float64) - d[:, None] * q)
    assert (err[inside] <= d[:, None].repeat(512, 1)[inside] * 0.5 * (1 + 1e-12)).all()
    for j in (-3, 1, 5):  # powers of two scale x exactly: codes unchanged, scale multiplied
        q2, d2 = oracle.quant_int4(x * np.float32(2.0 ** j), eps=0.0)
        assert np.array_equal(q, q2)
        assert np.allclose(d2, d * 2.0 ** j, rtol=1e-15)


def test_int4_all_zero_token(oracle):
    q, d = oracle.quant_int4(np.zeros((2, 16), np.float32))
    assert not q.any() and not d.any()


# ----------------------------------------------------------------------------- Eq. 1, 3 (top-K + INT8 absmax)
def _bruteforce_mask(x, k):
    a = np.abs(x.astype(np.float64))
    K = a.shape[0]
    m = np.zeros(K, np.uint8)
    for j in range(K):
        rank = sum(1 for i in range(K) if a[i] > a[j] or (a[i] == a[j] and i < j))
        m[j] = 1 if rank < k else 0
    return m


def test_topk_bruteforce_small(oracle):
    rng = np.random.default_rng(2)
    for K, k in ((8, 1), (8, 8), (33, 16), (64, 32), (64, 63)):
        x = rng.standard_normal((5, K)).astype(np.float32)
        x[1, :] = np.round(x[1, :])  # many ties, including zeros
        x[2, ::2] = 0.0
        x[3, :] = -0.0
        x[3, 5] = 0.0
        c, d, mask = oracle.topk_quant_int8(x, k, eps=0.0)
        for r in range(5):
            assert np.array_equal(mask[r], _bruteforce_mask(x[r], k)), (K, k, r)
        assert (mask.sum(1) == k).all()


def test_topk_ties_lowest_index(oracle):
    x = np.array([[1, -1, 1, 0.5, -1, 1, 0.25, 1]], np.float32)
    _, _, mask = oracle.topk_quant_int8(x, 3, eps=0.0)
    assert mask.tolist() == [[1, 1, 1, 0, 0, 0, 0, 0]]
    _, _, mask = oracle.topk_quant_int8(x, 7, eps=0.0)
    assert mask.tolist() == [[1, 1, 1, 1, 1, 1, 0, 1]]


def test_int8_rounding_ties_and_range(oracle):
    # gamma = 127, eps = 0: 127/gamma * x = x, so 0.5, 1.5, 2.5, -3.5 hit exact ties
    x = np.array([[127.0, 0.5, 1.5, 2.5, -3.5, -127.0, 64.49, 0.0]], np.float32)
    c, d, mask = oracle.topk_quant_int8(x, 8, eps=0.0)
    assert c.tolist() == [[127, 0, 2, 2, -4, -127, 64, 0]]
    assert d[0] == 1.0
    # the printed lower clip of -128 can never fire: |127 x / (gamma+eps)| <= 127
    y = synth.student_t3(64, 2048, seed=9).numpy()
    c, d, mask = oracle.topk_quant_int8(y, 2048)
    assert c.min() >= -127 and c.max() <= 127
    assert (np.abs(c).max(1) == 127).all()  # the arg-max is always coded +-127


def test_topk_half_is_table2_out_column(oracle):
    # Section 3: "topK as 50 %" for the attention output projection; Table 2 "Out" column = 50.0
    rows = golden("table2_sparsity.txt")
    assert all(rows[m][1] == 50.0 for m in rows)
    y = synth.student_t3(16, 4096, seed=10).numpy()
    c, d, mask = oracle.topk_quant_int8(y, 2048)
    assert (mask.sum(1) == 2048).all()
    assert ((c != 0) <= (mask == 1)).all()
    ay = np.abs(y)
    for r in range(16):  # every kept magnitude >= every dropped magnitude
        assert ay[r][mask[r] == 1].min() >= ay[r][mask[r] == 0].max()
    # gamma comes from the full row and the arg-max is kept
    assert np.allclose(d * 127.0, ay.max(1).astype(np.float64), rtol=1e-15)
    # median of |t_3| is 0.7649: the 50 % threshold of a long Student-t(3) row sits there
    z = synth.student_t3(1, 200000, seed=12).numpy()
    _, _, m = oracle.topk_quant_int8(z, 100000)
    assert np.abs(z[0])[m[0] == 1].min() == pytest.approx(0.7649, abs=0.01)


def test_mask_then_quantise_equals_quantise_then_mask(oracle):
    y = synth.student_t3(8, 512, seed=13).numpy()
    c, d, mask = oracle.topk_quant_int8(y, 256)
    c2, d2, mask2 = oracle.topk_quant_int8(y * mask, 256)  # sparsify first, then quantise
    assert np.array_equal(c, c2) and np.array_equal(d, d2) and np.array_equal(mask, mask2)
    cfull, dfull, _ = oracle.topk_quant_int8(y, 512)  # plain Q_INT8, then multiply by M
    assert np.array_equal(c, cfull * mask.astype(np.int8)) and np.array_equal(d, dfull)
    # error bound of Eq. 3 on the kept entries
    err = np.abs(y.astype(np.float64) - d[:, None] * cfull)
    assert (err <= d[:, None] * 0.5 * (1 + 1e-9) + 1e-5).all()


# ----------------------------------------------------------------------------- Eq. 1 / Eq. 6 (contraction)
def test_linear_matches_dequantised_float_matmul(oracle):
    M, N, K = 7, 13, 40
    x = synth.gaussian_outlier_activations(M, K, seed=4, count=2).numpy()
    W = synth.latent_weights(N, K, seed=5).numpy()
    t, alpha = oracle.ternarise(W)
    for codes, d in (oracle.quant_int4(x), oracle.topk_quant_int8(x, K // 2)[:2]):
        acc, y = oracle.linear(codes, d, t, alpha)
        assert np.array_equal(acc, codes.astype(np.int64) @ t.astype(np.int64).T)
        deq_x = d[:, None] * codes.astype(np.float64)  # Q_a(X)
        deq_w = alpha * t.astype(np.float64)  # Q_w(W)
        ref = deq_x @ deq_w.T
        bound = 1e-12 * (np.abs(deq_x) @ np.abs(deq_w).T)  # float-matmul rounding scales with sum |terms|
        assert (np.abs(y - ref) <= bound).all()
        assert (y[acc == 0] == 0.0).all()
        assert np.abs(acc).max() <= 128 * K
    # column permutation of the contraction index leaves the result unchanged
    perm = np.random.default_rng(0).permutation(K)
    acc2, _ = oracle.linear(codes[:, perm], d, t[:, perm], alpha)
    assert np.array_equal(acc, acc2)


def test_linear_threads_agree(oracle):
    x = synth.gaussian_outlier_activations(9, 64, seed=4, count=1).numpy()
    t, alpha = oracle.ternarise(synth.latent_weights(11, 64, seed=5).numpy())
    q, d = oracle.quant_int4(x)
    q3, d3 = oracle.quant_int4(x, nthreads=3)
    assert np.array_equal(q, q3) and np.array_equal(d, d3)
    a1, y1 = oracle.linear(q, d, t, alpha)
    a3, y3 = oracle.linear(q, d, t, alpha, nthreads=3)
    assert np.array_equal(a1, a3) and np.array_equal(y1, y3)


# ----------------------------------------------------------------------------- Eq. 8-9 (FP4 E2M1, MinMax)
def test_fp4_grid(oracle):
    x = synth.student_t3(32, 1024, seed=14).numpy()
    g, d = oracle.quant_fp4(x)
    grid = np.array([0, 1, 2, 3, 4, 6, 8, 12])
    assert set(np.unique(np.abs(g))) <= set(grid.tolist())
    assert (np.abs(g).max(1) == 12).all()  # |x|max maps to the top code exactly
    assert np.allclose(d * 12.0, np.abs(x).max(1).astype(np.float64), rtol=1e-15)
    # textbook E2M1 values {0,.5,1,1.5,2,3,4,6} times |x|max/6
    e2m1 = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0}
    assert set(np.unique(np.abs(g) / 2.0)) <= e2m1
    # each output is the nearest grid point to the scaled input (brute force over the grid)
    xp = x.astype(np.float64) / d[:, None]
    full = np.concatenate([-grid[::-1], grid[1:]]).astype(np.float64)
    dist = np.abs(xp[..., None] - full)
    best = dist.min(-1)
    assert np.allclose(np.abs(xp - g), best, rtol=0, atol=1e-9)
    # monotone
    order = np.argsort(x[0])
    assert (np.diff(g[0][order].astype(int)) >= 0).all()
    gz, dz = oracle.quant_fp4(np.zeros((1, 8), np.float32))
    assert not gz.any() and dz[0] == 0.0


def test_compacted_rows_reproduce_the_dense_contraction(oracle):
    # Section 2.1: masked channels contribute nothing to Eq. 1, so the contraction over the listed channels
    # alone equals the dense one; the list itself is pinned by hand on a small row and by its invariants.
    row = np.array([[0, 5, 0, 0, -3, 0, 127, 0, -128, 0, 0, 1]], np.int8)
    (idx, val), = oracle.compact_codes(row)
    assert idx.tolist() == [1, 4, 6, 8, 11] and val.tolist() == [5, -3, 127, -128, 1]
    rng = np.random.default_rng(5)
    X = rng.standard_t(3, size=(6, 96)).astype(np.float32)
    codes, d, mask = oracle.topk_quant_int8(X, 48, 1e-5)
    lists = oracle.compact_codes(codes)
    for m, (idx, val) in enumerate(lists):
        assert np.all(np.diff(idx) > 0) and np.all(val != 0)           # ascending, no zero entries
        assert len(idx) <= 48 and np.all(mask[m, idx] == 1)            # only kept channels, at most k of them
        dense = np.zeros(96, np.int8)
        dense[idx] = val
        assert np.array_equal(dense, codes[m])                         # scatter gives the row back
    W = rng.normal(0, 0.02, size=(10, 96)).astype(np.float32)
    t, alpha = oracle.ternarise(W, 1e-5)
    acc_dense, y_dense = oracle.linear(codes, d, t, alpha)
    acc_list, y_list = oracle.linear_from_lists(lists, d, t, alpha)
    assert np.array_equal(acc_dense, acc_list) and np.array_equal(y_dense, y_list)


def test_five_codes_per_byte_is_the_base3_number_of_the_codes():
    # the densest whole-byte packing of ternary codes (Section 1 counts log2(3) = 1.58 bits per weight): 3^5 = 243
    # values fit a byte, so five codes cost 8 bits = 1.6 bits each, and the packing is invertible
    import itertools
    import math
    seen = set()
    for t in itertools.product((-1, 0, 1), repeat=5):
        b = sum((ti + 1) * 3 ** i for i, ti in enumerate(t))
        assert 0 <= b <= 242
        back = tuple((b // 3 ** i) % 3 - 1 for i in range(5))
        assert back == t
        seen.add(b)
    assert len(seen) == 243 and 3 ** 5 <= 256 < 3 ** 6
    assert 8 / 5 == 1.6 and math.log2(3) < 1.6
