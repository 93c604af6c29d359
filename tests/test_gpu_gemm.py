"""tcgen05 prefill kernel (both operand variants) against the oracle: int32 accumulators bit-exact."""
import numpy as np
import pytest
import torch

from parity import max_rel_err
from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5
# (M, N, K): one tile; several k-blocks; ragged M and N tails; K a multiple of 64 but not 128 (like 8640);
# K a multiple of 16 only; several tiles per CTA wave
SHAPES = [(256, 128, 128), (256, 128, 1024), (300, 200, 384), (70, 130, 320), (513, 257, 144), (1, 128, 256),
          (1100, 1536, 1536),
          # 65..128 and 193..256 tokens run on 128-token tiles: ragged second tile, few tiles with the cluster split
          (100, 300, 512), (200, 384, 640), (250, 130, 2048), (100, 256, 4096), (250, 384, 4096), (128, 2048, 1024)]


def _algos(a48):
    return {"tmem": a48.ALGO_GEMM_TCGEN05, "smem_i8": a48.ALGO_GEMM_TCGEN05_I8}


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("variant", ["tmem", "smem_i8"])
@pytest.mark.parametrize("kind", ["int4", "topk"])
def test_gemm_tcgen05_matches_oracle(a48, oracle, cuda_dev, M, N, K, variant, kind):
    W = synth.latent_weights(N, K, seed=N + K)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_ALL | a48.LAYOUT_I8)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed=M)
        codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
        c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS, nthreads=8)
        act = a48.ACT_INT4
    else:
        x = synth.student_t3(M, K, seed=M)
        codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS, nthreads=8)
        act = a48.ACT_TOPK_INT8
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    y, acc = a48.linear(w, codes, scale, act, _algos(a48)[variant], want_acc=True)
    torch.cuda.synchronize()
    assert a48.kernel_status() == [0, 0, 0, 0]
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5


# CTA-pair form (cta_group::2): 256 weight rows per two SMs.  One pair tile, several k-blocks, ragged M (second half
# of the token tile partly or wholly beyond M), several tiles per pair, K = 8640, N with an odd number of 128-row
# tiles (the last pair's second CTA has no rows of its own) and N not a multiple of 128 at all.
PAIR_SHAPES = [(192, 256, 256), (100, 256, 1024), (97, 512, 384), (300, 768, 2048), (1100, 1536, 1536), (200, 256, 8640),
               (250, 384, 512), (130, 128, 256), (400, 3200, 640), (77, 200, 320), (513, 257, 144)]


@pytest.mark.parametrize("M,N,K", PAIR_SHAPES)
@pytest.mark.parametrize("kind", ["int4", "topk"])
def test_gemm_pair_matches_oracle(a48, oracle, cuda_dev, M, N, K, kind):
    W = synth.latent_weights(N, K, seed=N + K + 2)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_GEMM)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed=M + 1)
        codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
        c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS, nthreads=8)
        act = a48.ACT_INT4
    else:
        x = synth.student_t3(M, K, seed=M + 1)
        codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS, nthreads=8)
        act = a48.ACT_TOPK_INT8
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    for _ in range(2):
        y, acc = a48.linear(w, codes, scale, act, a48.ALGO_GEMM_TCGEN05_PAIR, want_acc=True)
        torch.cuda.synchronize()
        assert a48.kernel_status() == [0, 0, 0, 0]
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
        assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5


def test_gemm_extreme_codes_do_not_overflow(a48, oracle, cuda_dev):
    # all codes +-127 against all-(+1) weights: |acc| = 127*K, the largest accumulator this path can see
    M, N, K = 256, 128, 11008
    W = torch.full((N, K), 0.05)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_GEMM)
    codes = torch.full((M, K), 127, dtype=torch.int8)
    codes[1::2] = -127
    scale = torch.ones(M)
    y, acc = a48.linear(w, codes.to(cuda_dev), scale.to(cuda_dev), a48.ACT_TOPK_INT8, a48.ALGO_GEMM_TCGEN05,
                        want_acc=True)
    acc = acc.cpu()
    assert (acc[0::2] == 127 * K).all() and (acc[1::2] == -127 * K).all()


def test_gemm_full_size_sampled(a48, oracle, cuda_dev):
    # The benchmark's launch configuration: 7B gate projection (4096 -> 11008) over 16384 tokens.  The oracle
    # recomputes a sample: 24 whole token rows and 24 whole output columns.
    M, N, K = 16384, 11008, 4096
    W = synth.ternary_latents(N, K, seed=4, device=cuda_dev)
    w = a48.pack_ternary(W, EPS, a48.LAYOUT_GEMM)
    t_dev, alpha = a48.weight_unpack(w)
    x = synth.gaussian_outlier_activations(M, K, seed=40, device=cuda_dev)
    codes, scale = a48.quant_int4(x, EPS)
    # the library's own choice at this size, as in the benchmark: the CTA-pair form
    y, acc = a48.linear(w, codes, scale, a48.ACT_INT4, a48.ALGO_AUTO, want_acc=True)
    y1, acc1 = a48.linear(w, codes, scale, a48.ACT_INT4, a48.ALGO_GEMM_TCGEN05, want_acc=True)
    torch.cuda.synchronize()
    assert a48.kernel_status() == [0, 0, 0, 0]
    assert torch.equal(acc, acc1) and torch.equal(y, y1)  # single-CTA form: the same bits
    del y1, acc1
    g = torch.Generator().manual_seed(0)
    rows = torch.cat([torch.tensor([0, 255, 256, M - 1]), torch.randint(0, M, (20,), generator=g)]).to(cuda_dev)
    cols = torch.cat([torch.tensor([0, 127, 128, N - 1]), torch.randint(0, N, (20,), generator=g)]).to(cuda_dev)
    t_ref, a_ref = oracle.ternarise(W.cpu().numpy(), EPS)
    assert np.array_equal(t_dev.cpu().numpy(), t_ref) and alpha == np.float32(a_ref)
    x_rows = x[rows].cpu().numpy()
    q_ref, d_ref = oracle.quant_int4(x_rows, EPS, nthreads=8)
    assert np.array_equal(codes[rows].cpu().numpy(), q_ref)
    acc_ref, y_ref = oracle.linear(q_ref, d_ref, t_ref, a_ref, nthreads=8)
    assert np.array_equal(acc[rows].cpu().numpy().astype(np.int64), acc_ref)
    assert max_rel_err(y[rows].cpu().numpy(), y_ref) <= 1e-5
    # whole columns: every token against 24 weight rows (codes already checked on the sampled rows; here the
    # GPU codes feed the oracle contraction, which checks the contraction at every token)
    codes_h, scale_h = codes.cpu().numpy(), scale.cpu().numpy().astype(np.float64)
    acc_c, _ = oracle.linear(codes_h, scale_h, t_ref[cols.cpu().numpy()], a_ref, nthreads=8, want_y=False)
    assert np.array_equal(acc[:, cols].cpu().numpy().astype(np.int64), acc_c)


# Few tokens: the 64-token tile and the split of a tile's channels over the CTAs of a cluster.  (M, N, K) cover one and
# several weight-row tiles, a ragged N tail, K = 3200 / 8640 (padded to whole pipeline units), M around the
# 64-token boundary and a two-tile M of the wide kernel.
SKINNY = [(9, 128, 512), (16, 384, 2048), (33, 200, 3200), (64, 1024, 8640), (65, 256, 2048), (100, 640, 4096),
          (191, 130, 1536), (40, 3200, 3200), (32, 1000, 4096), (17, 130, 11008), (31, 4096, 1024)]


@pytest.mark.parametrize("M,N,K", SKINNY)
@pytest.mark.parametrize("variant", ["tmem", "smem_i8"])
def test_gemm_few_tokens_split_k(a48, oracle, cuda_dev, M, N, K, variant):
    W = synth.latent_weights(N, K, seed=N + K + 1)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_GEMM | a48.LAYOUT_I8)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    x = synth.student_t3(M, K, seed=M + 7)
    codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
    c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS, nthreads=8)
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    algo = _algos(a48)[variant]
    for _ in range(2):
        y, acc = a48.linear(w, codes, scale, a48.ACT_TOPK_INT8, algo, want_acc=True)
        torch.cuda.synchronize()
        assert a48.kernel_status() == [0, 0, 0, 0]
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
        assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5


@pytest.mark.parametrize("Ns,K,M", [((512, 256), 1536, 12), ((3200, 3200, 3200), 3200, 64), ((130, 257, 64, 1000), 400, 33),
                                    ((1024, 1024), 2048, 100), ((640, 384, 128), 512, 300)])
def test_gemm_grouped_launch_matches_oracle(a48, oracle, cuda_dev, Ns, K, M):
    # q/k/v-like and gate/up-like groups beyond the decode kernel's token count: one tensor-core launch walks the
    # tiles of all matrices (with and without the cluster split); every output against the oracle
    Ws = [synth.latent_weights(N, K, seed=3 * N + i) for i, N in enumerate(Ns)]
    ws = [a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_GEMM) for W in Ws]
    x = synth.gaussian_outlier_activations(M, K, seed=M)
    codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
    c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS, nthreads=8)
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    fused = a48.linear_multi(ws, codes, scale, a48.ACT_INT4)
    torch.cuda.synchronize()
    assert a48.kernel_status() == [0, 0, 0, 0]
    for W, w, y in zip(Ws, ws, fused):
        t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
        _, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
        assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5
        assert torch.equal(y, a48.linear(w, codes, scale, a48.ACT_INT4, a48.ALGO_GEMM_TCGEN05))


@pytest.mark.parametrize("M", [32, 64])
def test_gemm_decode_batch_3b_layer(a48, oracle, cuda_dev, M):
    # The 3B decode configuration at 32 and 64 tokens, in the launch form the benchmark's chain uses: q/k/v and
    # gate/up as grouped launches, o and down as single (cluster split-K) launches; int32-exact against the oracle
    H, F = 3200, 8640
    def make(n, k, seed):
        W = synth.ternary_latents(n, k, seed=seed)
        return W, a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_GEMM)
    x4 = synth.gaussian_outlier_activations(M, H, seed=5)
    c4, d4 = a48.quant_int4(x4.to(cuda_dev), EPS)
    c4_ref, d4_ref = oracle.quant_int4(x4.numpy(), EPS, nthreads=8)
    assert np.array_equal(c4.cpu().numpy(), c4_ref)
    for Ns, K, codes, scale, c_ref, d_ref, act in [((H, H, H), H, c4, d4, c4_ref, d4_ref, a48.ACT_INT4),
                                                   ((F, F), H, c4, d4, c4_ref, d4_ref, a48.ACT_INT4)]:
        pairs = [make(n, K, 70 + i) for i, n in enumerate(Ns)]
        ys = a48.linear_multi([w for _, w in pairs], codes, scale, act)
        torch.cuda.synchronize()
        assert a48.kernel_status() == [0, 0, 0, 0]
        for (W, w), y in zip(pairs, ys):
            t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
            _, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
            assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5
    for n, k in [(H, H), (H, F)]:
        xs = synth.student_t3(M, k, seed=k)
        c8, d8, _ = a48.topk_quant_int8(xs.to(cuda_dev), k // 2, EPS)
        c8_ref, d8_ref, _ = oracle.topk_quant_int8(xs.numpy(), k // 2, EPS, nthreads=8)
        assert np.array_equal(c8.cpu().numpy(), c8_ref)
        W, w = make(n, k, 90 + n % 7)
        y, acc = a48.linear(w, c8, d8, a48.ACT_TOPK_INT8, want_acc=True)
        torch.cuda.synchronize()
        assert a48.kernel_status() == [0, 0, 0, 0]
        t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
        acc_ref, y_ref = oracle.linear(c8_ref, d8_ref, t_ref, alpha, nthreads=8)
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
        assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5
