"""BitLinear contraction on the GPU against the oracle: int32 accumulators bit-exact,
fp32 outputs within 1e-5 relative (Eq. 1 / Eq. 6)."""
import numpy as np
import pytest
import torch

from parity import max_rel_err
from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5
REL_TOL = 1e-5  # max relative error per BitLinear output


def _case(a48, oracle, dev, M, N, K, kind, seed):
    W = synth.latent_weights(N, K, seed=seed)
    w = a48.pack_ternary(W.to(dev), EPS, a48.LAYOUT_ALL)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    if kind == "int4":
        x = synth.gaussian_outlier_activations(M, K, seed + 1)
        codes, scale = a48.quant_int4(x.to(dev), EPS)
        c_ref, d_ref = oracle.quant_int4(x.numpy(), EPS, nthreads=8)
        act = a48.ACT_INT4
    else:
        x = synth.student_t3(M, K, seed + 1)
        codes, scale, _ = a48.topk_quant_int8(x.to(dev), K // 2, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(x.numpy(), K // 2, EPS, nthreads=8)
        act = a48.ACT_TOPK_INT8
    assert np.array_equal(codes.cpu().numpy(), c_ref)
    acc_ref, y_ref = oracle.linear(c_ref, d_ref, t_ref, alpha, nthreads=8)
    return w, codes, scale, act, acc_ref, y_ref


SIMPLE_SHAPES = [(32, 256, 256), (32, 768, 256), (32, 256, 768), (45, 200, 250), (70, 130, 1536), (1, 257, 129),
                 (5, 1536, 4096)]


@pytest.mark.parametrize("M,N,K", SIMPLE_SHAPES)
@pytest.mark.parametrize("kind", ["int4", "topk"])
def test_linear_simple_matches_oracle(a48, oracle, cuda_dev, M, N, K, kind):
    w, codes, scale, act, acc_ref, y_ref = _case(a48, oracle, cuda_dev, M, N, K, kind, seed=M + N + K)
    y, acc = a48.linear(w, codes, scale, act, a48.ALGO_SIMPLE, want_acc=True)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert max_rel_err(y.cpu().numpy(), y_ref) <= REL_TOL
    y2 = a48.linear(w, codes, scale, act, a48.ALGO_AUTO)  # whatever AUTO picks must agree bit for bit
    assert torch.equal(y, y2)


@pytest.mark.parametrize("M", [5, 300])
def test_host_buffer_entry_points_match_the_device_path(a48, cuda_dev, M):
    # bitnet_a48_bitlinear_host and its asynchronous form: upload, quantise, contract, download
    N, K = 384, 512
    w = a48.pack_ternary(synth.latent_weights(N, K, seed=3).to(cuda_dev), EPS, a48.LAYOUT_ALL)
    x = synth.student_t3(M, K, seed=4)
    codes, scale, _ = a48.topk_quant_int8(x.to(cuda_dev), K // 2, EPS)
    expected = a48.linear(w, codes, scale, a48.ACT_TOPK_INT8).cpu()
    ws = torch.zeros(a48.bitlinear_host_workspace_bytes(w, M), dtype=torch.uint8, device=cuda_dev)
    xp = x.pin_memory()
    y1 = torch.empty(M, N).pin_memory()
    a48.bitlinear_host(w, xp, y1, a48.ACT_TOPK_INT8, K // 2, EPS, ws)
    assert torch.equal(y1, expected)
    y2 = torch.full((M, N), float("nan")).pin_memory()
    side = torch.cuda.Stream()
    a48.bitlinear_host_async(w, xp, y2, a48.ACT_TOPK_INT8, K // 2, EPS, ws, stream=side)
    side.synchronize()
    assert torch.equal(y2, expected)


# Eq. 8-9: the FP4 quantiser's codes are integers on the doubled E2M1 grid {0, ±1, ±2, ±3, ±4, ±6, ±8, ±12}, so they
# go through the same int8 contraction exactly.  Every kernel the dispatcher can pick is covered: decode (M <= 8),
# the tensor-core forms (64-token tile, 192-token tile, CTA pairs from 1024 tokens on) and the simple kernel.
@pytest.mark.parametrize("M,N,K", [(1, 512, 1024), (7, 384, 512), (40, 640, 768), (300, 384, 512), (1100, 512, 256),
                                   (33, 130, 250)])
def test_fp4_codes_through_the_contraction(a48, oracle, cuda_dev, M, N, K):
    W = synth.latent_weights(N, K, seed=N + K + 1)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_ALL)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    x = synth.gaussian_outlier_activations(M, K, seed=M + 2)
    codes, scale = a48.quant_fp4(x.to(cuda_dev))
    g_ref, d_ref = oracle.quant_fp4(x.numpy(), nthreads=8)
    assert np.array_equal(codes.cpu().numpy(), g_ref)
    acc_ref, y_ref = oracle.linear(g_ref, d_ref, t_ref, alpha, nthreads=8)
    y, acc = a48.linear(w, codes, scale, a48.ACT_FP4, a48.ALGO_AUTO, want_acc=True)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert max_rel_err(y.cpu().numpy(), y_ref) <= REL_TOL
    y2, acc2 = a48.linear(w, codes, scale, a48.ACT_FP4, a48.ALGO_SIMPLE, want_acc=True)
    assert torch.equal(acc, acc2)
