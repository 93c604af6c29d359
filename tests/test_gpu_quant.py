"""CUDA quantisers and weight packer against the CPU oracle (bit-exact codes, masks and scales to fp32)."""
import math

import numpy as np
import pytest
import torch

from parity import assert_codes_match, unpack_mask_bits
from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5
# K values: 256 (one warp per row), 1536/3200/4096 (wider groups), 8640/11008 (12 vectors per thread,
# ragged tail), 250 and 13004 (generic path: unaligned / beyond the register-resident limit)
SHAPES = [(32, 256), (37, 768), (19, 1536), (13, 3200), (21, 4096), (9, 8640), (11, 11008), (7, 250), (3, 13004),
          (300, 512)]


def _inputs(kind, M, K, seed):
    if kind == "gauss":
        return synth.gaussian_outlier_activations(M, K, seed)
    return synth.student_t3(M, K, seed)


@pytest.mark.parametrize("M,K", SHAPES)
def test_quant_int4_matches_oracle(a48, oracle, cuda_dev, M, K):
    x = _inputs("gauss", M, K, seed=M + K)
    x[M // 2] = 0.0  # an all-zero token
    codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
    q_ref, d_ref = oracle.quant_int4(x.numpy(), EPS, nthreads=4)
    beta = d_ref * math.sqrt(7.0)
    n_bad = assert_codes_match(codes.cpu().numpy(), q_ref, x.numpy(), math.sqrt(7.0) / (beta + EPS), "int4")
    assert n_bad == 0 or n_bad < 1e-6 * M * K
    assert np.array_equal(scale.cpu().numpy(), d_ref.astype(np.float32))
    assert codes.min() >= -8 and codes.max() <= 7


@pytest.mark.parametrize("M,K", SHAPES)
@pytest.mark.parametrize("kfrac", [0.5, 0.0, 1.0])
def test_topk_quant_int8_matches_oracle(a48, oracle, cuda_dev, M, K, kfrac):
    k = max(1, min(K, int(round(kfrac * K))))
    x = _inputs("t3", M, K, seed=2 * M + K)
    x[0] = 0.0  # all-zero token: the first k indices win the tie
    if M > 2:
        x[1] = torch.round(x[1])  # many equal magnitudes, ties straddle the k-th place
        x[2] = torch.relu(x[2]) ** 2  # ReLU²-like: about half exact zeros
    codes, scale, bits = a48.topk_quant_int8(x.to(cuda_dev), k, EPS, want_mask=True)
    c_ref, d_ref, m_ref = oracle.topk_quant_int8(x.numpy(), k, EPS, nthreads=4)
    mask = unpack_mask_bits(bits.cpu().numpy(), K)
    assert np.array_equal(mask, m_ref), "top-k mask differs"
    assert (mask.sum(1) == k).all()
    gamma = d_ref * 127.0
    assert_codes_match(codes.cpu().numpy(), c_ref, x.numpy(), 127.0 / (gamma + EPS), "int8")
    assert np.array_equal(scale.cpu().numpy(), d_ref.astype(np.float32))
    assert np.array_equal(codes.cpu().numpy() != 0, (c_ref != 0))
    # the same call without the bitmap takes the kernel that keeps the row in registers: identical codes and scales
    codes2, scale2, _ = a48.topk_quant_int8(x.to(cuda_dev), k, EPS)
    assert torch.equal(codes2, codes) and torch.equal(scale2, scale)


@pytest.mark.parametrize("K", [512, 1536, 3200, 4096, 8640, 11008])
def test_topk_rows_that_leave_the_common_path(a48, oracle, cuda_dev, K):
    # Rows built to miss the interpolated window or to overflow the ranking list of the register kernel, next to
    # ordinary ones: two far-apart clusters (the k-th entry sits at a cluster's edge), one value repeated over most
    # of the row (more ties than the list holds), values that differ in the last bits only, tiny magnitudes
    # (denormals), huge ones, and mostly-zero rows whose k-th entry is zero or the smallest non-zero one.
    g = torch.Generator().manual_seed(K)
    rows = []
    r = torch.randn(K, generator=g)
    rows.append(torch.where(torch.arange(K) % 2 == 0, r * 1e-3, 1.0 + 1e-4 * r))          # two clusters, k = K/2 at the gap
    rows.append(torch.where(torch.arange(K) % 3 == 0, r, torch.full((K,), 0.75)))           # two thirds equal 0.75
    rows.append(1.0 + torch.randint(0, 50, (K,), generator=g).float() * 2.0 ** -23)         # last-bit differences, many ties
    rows.append(r * 1e-41)                                                                  # denormals only
    rows.append(r * 1e37)                                                                   # near the top of the range
    z = torch.relu(torch.randn(K, generator=g)) ** 2
    rows.append(z)                                                                          # about half zeros
    rows.append(torch.where(torch.rand(K, generator=g) < 0.9, torch.zeros(K), z + 0.1))     # 90 % zeros
    rows.append(torch.sign(r) * torch.exp(8.0 * torch.randn(K, generator=g)))               # log-normal over many binades
    rows.append(synth.student_t3(1, K, seed=K)[0])
    x = torch.stack(rows).float().contiguous()
    for k in (K // 2, K // 8, K - 3, 1):
        codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), k, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), k, EPS, nthreads=4)
        assert np.array_equal(codes.cpu().numpy(), c_ref), f"k={k}: rows {np.unique(np.argwhere(codes.cpu().numpy() != c_ref)[:, 0])}"
        assert np.array_equal(scale.cpu().numpy(), d_ref.astype(np.float32))


def test_topk_without_mask_output(a48, oracle, cuda_dev):
    x = synth.student_t3(5, 1024, seed=3)
    codes, scale, bits = a48.topk_quant_int8(x.to(cuda_dev), 512, EPS)
    assert bits is None
    c_ref, _, _ = oracle.topk_quant_int8(x.numpy(), 512, EPS)
    assert np.array_equal(codes.cpu().numpy(), c_ref)


@pytest.mark.parametrize("M,K", [(16, 512), (5, 250), (3, 4096), (9, 1536), (4, 3200), (6, 8640), (5, 11008), (2, 13004)])
def test_quant_fp4_matches_oracle(a48, oracle, cuda_dev, M, K):
    x = synth.student_t3(M, K, seed=M * K)
    x[0] = 0.0
    codes, scale = a48.quant_fp4(x.to(cuda_dev))
    g_ref, d_ref = oracle.quant_fp4(x.numpy())
    assert np.array_equal(codes.cpu().numpy(), g_ref)
    assert np.array_equal(scale.cpu().numpy(), d_ref.astype(np.float32))


@pytest.mark.parametrize("N,K", [(256, 256), (768, 256), (100, 250), (130, 384), (1536, 4096), (257, 129)])
def test_pack_ternary_matches_oracle_in_every_layout(a48, oracle, cuda_dev, N, K):
    W = synth.latent_weights(N, K, seed=N + K)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_ALL)
    codes, alpha = a48.weight_unpack(w)
    t_ref, a_ref = oracle.ternarise(W.numpy(), EPS)
    assert np.array_equal(codes.cpu().numpy(), t_ref)
    assert alpha == np.float32(a_ref)
    for layout in (a48.LAYOUT_GEMM, a48.LAYOUT_DECODE, a48.LAYOUT_SPARSE):
        again = a48.weight_unpack_layout(w, layout)
        assert np.array_equal(again.cpu().numpy(), t_ref), f"layout {layout} holds a different matrix"
    assert w.packed_bytes == N * ((K + 3) // 4)
    w.free()


def test_pack_ternary_ties_and_ternary_latents(a48, oracle, cuda_dev):
    W = torch.tensor([[0.5, -0.5, 1.5, 1.5]] * 4, dtype=torch.float32)
    w = a48.pack_ternary(W.to(cuda_dev), 0.0, 0)
    codes, alpha = a48.weight_unpack(w)
    assert codes.cpu().tolist() == [[0, 0, 1, 1]] * 4 and alpha == 1.0
    W = synth.ternary_latents(96, 160, seed=1)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, 0)
    codes, alpha = a48.weight_unpack(w)
    t_ref, a_ref = oracle.ternarise(W.numpy(), EPS)
    assert np.array_equal(codes.cpu().numpy(), t_ref) and alpha == np.float32(a_ref)


@pytest.mark.parametrize("K,kind", [(4096, "int4"), (4096, "topk"), (11008, "topk")])
def test_quantisers_at_benchmark_size_sampled(a48, oracle, cuda_dev, K, kind):
    # The benchmark's launch configuration (16384 tokens of the 7B shape); the oracle recomputes 48 sampled rows,
    # and every row is checked for what holds at any size: code range, at most k survivors, the maximum coded +-127.
    M = 16384
    g = torch.Generator().manual_seed(K)
    rows = torch.cat([torch.tensor([0, 1, M - 1]), torch.randint(0, M, (45,), generator=g)]).to(cuda_dev)
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed=40, device=cuda_dev)
        codes, scale = a48.quant_int4(x, EPS)
        q_ref, d_ref = oracle.quant_int4(x[rows].cpu().numpy(), EPS, nthreads=8)
        assert int(codes.min()) >= -8 and int(codes.max()) <= 7
    else:
        x = synth.student_t3(M, K, seed=41, device=cuda_dev)
        codes, scale, _ = a48.topk_quant_int8(x, K // 2, EPS)
        q_ref, d_ref, _ = oracle.topk_quant_int8(x[rows].cpu().numpy(), K // 2, EPS, nthreads=8)
        nz = (codes != 0).sum(1)
        assert int(nz.max()) <= K // 2  # at most k survivors (kept entries below gamma/254 still code to 0)
        assert bool((codes.abs().amax(1) == 127).all())
    assert np.array_equal(codes[rows].cpu().numpy(), q_ref)
    assert np.array_equal(scale[rows].cpu().numpy(), d_ref.astype(np.float32))


@pytest.mark.parametrize("M,K,kfrac", [(1, 4096, 0.5), (3, 11008, 0.5), (8, 3200, 0.5), (5, 250, 0.3), (2, 65535, 0.1),
                                       (4, 1027, 1.0)])
def test_compact_codes_matches_oracle(a48, oracle, cuda_dev, M, K, kfrac):
    # compacted (channel, code) lists of the top-K codes: same entries, same order, same counts as the oracle's
    x = synth.student_t3(M, K, seed=K + M)
    k = max(1, int(K * kfrac))
    codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), k, EPS)
    c_ref, _, _ = oracle.topk_quant_int8(x.numpy(), k, EPS)
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    idx, val, count = a48.compact_codes(codes, cap=k)
    torch.cuda.synchronize()
    lists = oracle.compact_codes(c_ref)
    idx_h, val_h, cnt_h = idx.cpu().numpy().astype(np.int64), val.cpu().numpy(), count.cpu().numpy()
    for m, (i_ref, v_ref) in enumerate(lists):
        assert cnt_h[m] == len(i_ref) <= k
        assert np.array_equal(idx_h[m, :cnt_h[m]], i_ref) and np.array_equal(val_h[m, :cnt_h[m]], v_ref)
        assert not idx_h[m, cnt_h[m]:].any() and not val_h[m, cnt_h[m]:].any()  # nothing written past the count


def test_compact_codes_capacity_and_arguments(a48, cuda_dev):
    codes = torch.zeros(2, 64, dtype=torch.int8, device=cuda_dev)
    codes[0, ::2] = 7   # 32 non-zero codes, capacity 8: only the first 8 are written, the count says 32
    idx, val, count = a48.compact_codes(codes, cap=8)
    assert count.tolist() == [32, 0]
    assert idx[0].tolist() == list(range(0, 16, 2)) and val[0].tolist() == [7] * 8
    wide = torch.zeros(1, 65536, dtype=torch.int8, device=cuda_dev)  # indices would not fit 16 bits
    with pytest.raises(RuntimeError):
        a48.compact_codes(wide, cap=16)
