"""bf16 activations at the boundary: the quantisers read bf16 rows (widened exactly to fp32, then Eq. 7 / Eq. 1 + 3),
the contraction writes the round-to-nearest-even bf16 of its fp32 result (Eq. 1 / Eq. 6)."""
import numpy as np
import pytest
import torch

from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5


@pytest.mark.parametrize("M,K", [(7, 256), (33, 1536), (5, 3200), (19, 4096), (6, 8640), (9, 11008)])
def test_bf16_quantisers_match_oracle_on_the_widened_values(a48, oracle, cuda_dev, M, K):
    xg = synth.gaussian_outlier_activations(M, K, seed=K).to(torch.bfloat16)
    xs = synth.student_t3(M, K, seed=K + 1).to(torch.bfloat16)
    xs[0] = torch.relu(xs[0]) ** 2  # many zeros
    codes, scale = a48.quant_int4_bf16(xg.to(cuda_dev), EPS)
    q_ref, d_ref = oracle.quant_int4(xg.float().numpy(), EPS)  # bf16 -> fp32 is exact
    assert np.array_equal(codes.cpu().numpy(), q_ref) and np.array_equal(scale.cpu().numpy(), d_ref.astype(np.float32))
    for k in (K // 2, K // 7):
        codes, scale = a48.topk_quant_int8_bf16(xs.to(cuda_dev), k, EPS)
        c_ref, d_ref, _ = oracle.topk_quant_int8(xs.float().numpy(), k, EPS)
        # bf16 values repeat often: ties at the k-th place are common, and the lowest index must still win
        assert np.array_equal(codes.cpu().numpy(), c_ref)
        assert np.array_equal(scale.cpu().numpy(), d_ref.astype(np.float32))
    # the same codes as the fp32 entry points give on the widened values
    c32, s32 = a48.quant_int4(xg.float().to(cuda_dev), EPS)
    c16, s16 = a48.quant_int4_bf16(xg.to(cuda_dev), EPS)
    assert torch.equal(c32, c16) and torch.equal(s32, s16)


@pytest.mark.parametrize("M,N,K", [(1, 512, 1024), (7, 384, 512), (40, 640, 768), (300, 384, 512), (1100, 512, 256),
                                   (33, 130, 250)])
def test_bf16_output_is_the_rounded_fp32_output(a48, oracle, cuda_dev, M, N, K):
    W = synth.latent_weights(N, K, seed=N + K + 2)
    w = a48.pack_ternary(W.to(cuda_dev), EPS, a48.LAYOUT_ALL)
    t_ref, alpha = oracle.ternarise(W.numpy(), EPS)
    x = synth.gaussian_outlier_activations(M, K, seed=M + 3)
    codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
    y32 = a48.linear(w, codes, scale, a48.ACT_INT4)
    y16 = a48.linear_bf16(w, codes, scale, a48.ACT_INT4)
    assert y16.dtype == torch.bfloat16 and torch.equal(y16, y32.to(torch.bfloat16))  # torch rounds to nearest even
    # against the oracle: one bf16 rounding (2^-9 relative) on top of the fp32 tolerance
    q_ref, d_ref = oracle.quant_int4(x.numpy(), EPS)
    _, y_ref = oracle.linear(q_ref, d_ref, t_ref, alpha)
    got = y16.float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - y_ref) <= (2.0 ** -8) * np.abs(y_ref) + 1e-30).all()
    assert (got[y_ref == 0] == 0).all()
