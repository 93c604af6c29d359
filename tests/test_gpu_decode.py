"""Decode kernel (up to 8 tokens, weight-streaming) against the oracle: int32 accumulators bit-exact,
fp32 outputs within 1e-5 relative (Eq. 1 / Eq. 6)."""
import numpy as np
import pytest
import torch

from parity import max_rel_err
from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5
# (N, K): tiny; ragged N (not a multiple of 16) with K a multiple of 16 only; one, two and four CTAs per cluster;
# the 3B and 7B projection shapes
SHAPES = [(16, 128), (130, 144), (257, 400), (256, 512), (768, 2048), (3200, 3200), (8640, 3200), (3200, 8640),
          (4096, 4096), (11008, 4096), (4096, 11008)]


@pytest.mark.parametrize("N,K", SHAPES)
@pytest.mark.parametrize("M", [1, 3, 8])
@pytest.mark.parametrize("kind", ["int4", "topk"])
def test_decode_matches_oracle(a48, oracle, cuda_dev, N, K, M, kind):
    if N * K > 2e7 and M == 3:
        pytest.skip("large shapes run at M = 1 and M = 8")
    W = synth.latent_weights(N, K, seed=N + K)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed=M + K)
        codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
        c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS)
        act = a48.ACT_INT4
    else:
        x = synth.student_t3(M, K, seed=M + K)
        codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS)
        act = a48.ACT_TOPK_INT8
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    y, acc = a48.linear(w, codes, scale, act, a48.ALGO_DECODE, want_acc=True)
    torch.cuda.synchronize()
    assert a48.kernel_status() == [0, 0, 0, 0]
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5
    y2 = a48.linear(w, codes, scale, act, a48.ALGO_AUTO)  # AUTO takes the same kernel: identical bits
    assert torch.equal(y, y2)
    w.free()


def test_decode_extreme_codes(a48, cuda_dev):
    # every code -127 against all-(+1) weights, then all-(-1) weights: the largest accumulators this path can see
    N, K = 64, 11008
    for sign in (1.0, -1.0):
        w = a48.pack_ternary(torch.full((N, K), 0.05 * sign).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
        codes = torch.full((8, K), -127, dtype=torch.int8, device=cuda_dev)
        scale = torch.ones(8, device=cuda_dev)
        _, acc = a48.linear(w, codes, scale, a48.ACT_TOPK_INT8, a48.ALGO_DECODE, want_acc=True)
        assert (acc.cpu() == int(-127 * K * sign)).all()


def test_decode_rejects_more_than_eight_tokens(a48, cuda_dev):
    w = a48.pack_ternary(synth.latent_weights(64, 128, seed=1).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    codes = torch.zeros(9, 128, dtype=torch.int8, device=cuda_dev)
    scale = torch.ones(9, device=cuda_dev)
    with pytest.raises(a48.A48Error) as e:
        a48.linear(w, codes, scale, a48.ACT_INT4, a48.ALGO_DECODE)
    assert e.value.code == 4  # BITNET_A48_ERR_UNSUPPORTED


def test_decode_leaves_its_scratch_zeroed(a48, oracle, cuda_dev):
    # one scratch buffer, zeroed once, serves several calls in a row (different tokens, different matrices of one shape)
    N, K = 1100, 1536
    Ws = [synth.latent_weights(N, K, seed=70 + i) for i in range(2)]
    ws = [a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_DECODE) for W in Ws]
    scratch = torch.zeros(a48.linear_workspace_bytes(ws[0], 5), dtype=torch.uint8, device=cuda_dev)
    assert scratch.numel() > 0
    for rep in range(4):
        W, w = Ws[rep % 2], ws[rep % 2]
        M = 1 + rep
        x = synth.gaussian_outlier_activations(M, K, seed=80 + rep)
        codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
        c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS)
        t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
        acc_ref, _ = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8, want_y=False)
        _, acc = a48.linear(w, codes, scale, a48.ACT_INT4, a48.ALGO_DECODE, want_acc=True, workspace=scratch)
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
        assert int(scratch.count_nonzero()) == 0


@pytest.mark.parametrize("Ns,K,M", [((4096, 4096, 4096), 4096, 1), ((11008, 11008), 4096, 3), ((130, 257, 64, 1000), 400, 8),
                                    ((512, 256), 1536, 12)])
def test_linear_multi_equals_separate_calls(a48, cuda_dev, Ns, K, M):
    # q/k/v-like and gate/up-like groups on shared codes: the fused launch gives the bits of the separate calls
    # (which the tests above pin to the oracle); M = 12 takes the one-after-the-other route
    ws = [a48.pack_ternary(synth.latent_weights(N, K, seed=N + i).to(cuda_dev), EPS, a48.LAYOUT_ALL) for i, N in enumerate(Ns)]
    x = synth.gaussian_outlier_activations(M, K, seed=9).to(cuda_dev)
    codes, scale = a48.quant_int4(x, EPS)
    fused = a48.linear_multi(ws, codes, scale, a48.ACT_INT4)
    for w, y in zip(ws, fused):
        assert torch.equal(y, a48.linear(w, codes, scale, a48.ACT_INT4))
    assert a48.kernel_status() == [0, 0, 0, 0]


@pytest.mark.parametrize("N,K", [(16, 128), (130, 144), (1000, 250), (3200, 3200), (4096, 11008), (11008, 4096)])
@pytest.mark.parametrize("kfrac", [0.5, 0.05, 1.0])
def test_decode_sparse_matches_oracle(a48, oracle, cuda_dev, N, K, kfrac):
    # zero-skipping kernel: one token, top-K codes (about kfrac of the channels survive)
    W = synth.latent_weights(N, K, seed=N + K)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_SPARSE)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    x = synth.student_t3(1, K, seed=K)
    k = max(1, int(K * kfrac))
    codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), k, EPS)
    c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), k, EPS)
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    scratch = torch.zeros(a48.linear_workspace_bytes(w, 1), dtype=torch.uint8, device=cuda_dev)
    for _ in range(2):  # twice on one scratch: it is left zeroed
        y, acc = a48.linear(w, codes, scale, a48.ACT_TOPK_INT8, a48.ALGO_DECODE_SPARSE, want_acc=True, workspace=scratch)
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
        assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5
        assert int(scratch.count_nonzero()) == 0
    w.free()


def test_decode_sparse_segment_bound(a48, oracle, cuda_dev):
    # the segments of an output meet in one 64-bit word that has room for 255 of them (512 channels each): the widest
    # supported row is exact, one channel more is declined before anything is launched
    N, K = 48, 255 * 512
    W = synth.latent_weights(N, K, seed=77)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_SPARSE)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    x = synth.student_t3(1, K, seed=78)
    codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
    c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS)
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, _ = oracle.linear(c_ref, d_ref, t_ref, alpha)
    _, acc = a48.linear(w, codes, scale, a48.ACT_TOPK_INT8, a48.ALGO_DECODE_SPARSE, want_acc=True)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    wide = a48.pack_ternary(synth.latent_weights(16, K + 16, seed=79).to(cuda_dev), EPS, a48.LAYOUT_SPARSE)
    with pytest.raises(a48.A48Error) as e:
        a48.linear(wide, torch.zeros(1, K + 16, dtype=torch.int8, device=cuda_dev), torch.ones(1, device=cuda_dev),
                   a48.ACT_TOPK_INT8, a48.ALGO_DECODE_SPARSE)
    assert e.value.code == 4


@pytest.mark.parametrize("N,K", [(16, 128), (130, 144), (1000, 250), (3200, 3200), (4096, 11008), (11008, 4096), (257, 129)])
@pytest.mark.parametrize("M", [1, 3, 8])
def test_decode_trit5_matches_oracle(a48, oracle, cuda_dev, N, K, M):
    # five ternary codes per byte (1.6 bits per weight): the packed bytes are the base-3 numbers of the oracle's codes,
    # the layout unpacks to the same matrix, and the kernel that reads it gives the oracle's accumulators
    W = synth.latent_weights(N, K, seed=N + K + 5)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_TRIT5)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    assert np.array_equal(a48.weight_unpack_layout(w, a48.LAYOUT_TRIT5).cpu().numpy(), t_ref)
    row = ((K + 4) // 5 + 15) // 16 * 16
    assert w.layout_bytes(a48.LAYOUT_TRIT5) == N * row and row * 8 <= 1.6 * K + 16 * 8 + 8
    kind = "int4" if M != 3 else "topk"
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed=N)
        codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
        c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS)
        act = a48.ACT_INT4
    else:
        x = synth.student_t3(M, K, seed=N)
        codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS)
        act = a48.ACT_TOPK_INT8
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    y, acc = a48.linear(w, codes, scale, act, a48.ALGO_DECODE_TRIT5, want_acc=True)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert max_rel_err(y.cpu().numpy(), y_ref) <= 1e-5
    y2 = a48.linear(w, codes, scale, act, a48.ALGO_AUTO)  # the handle carries nothing else: AUTO takes this kernel
    assert torch.equal(y, y2)
    w.free()
