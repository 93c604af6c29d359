"""Gate-first feed-forward sub-layer on the GPU against the oracle (Section 2.1, paragraph after Eq. 5)."""
import numpy as np
import pytest
import torch

from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5


@pytest.mark.parametrize("H,F,M", [(256, 768, 1), (256, 768, 5), (1536, 4096, 2), (3200, 8640, 1), (4096, 11008, 1),
                                   (4096, 11008, 8), (320, 1000, 3)])
def test_ffn_gate_first_matches_oracle(a48, oracle, cuda_dev, H, F, M):
    lat = {n: synth.latent_weights(a, b, seed=50 + i) * 25.0
           for i, (n, a, b) in enumerate((("gate", F, H), ("up", F, H), ("down", H, F)))}
    w = {n: a48.pack_ternary(v.to(cuda_dev), EPS, a48.LAYOUT_ALL) for n, v in lat.items()}
    (tg, ag), (tu, au), (td, ad) = (oracle.ternarise(lat[n].numpy(), EPS) for n in ("gate", "up", "down"))
    x = synth.gaussian_outlier_activations(M, H, seed=51, count=max(2, H // 100))
    y, inter, rows = a48.ffn_gate_first(w["gate"], w["up"], w["down"], x.to(cuda_dev), F // 2, EPS, want_inter=True,
                                        want_rows=True)
    y_ref, active = oracle.ffn_gate_first(x.numpy(), tg, ag, tu, au, td, ad, F // 2, EPS)
    # the rows of W_up that were read: exactly those some token needs
    assert int(rows[0]) == int(active.any(0).sum())
    assert 0.2 * F < int(rows[0]) < (0.8 if M == 1 else 1.0) * F
    # Eq. 5's product: zero exactly where the oracle skipped, else within float32 rounding of the float64 product
    q, d = oracle.quant_int4(x.numpy(), EPS)
    _, gate = oracle.linear(q, d, tg, ag)
    _, up = oracle.linear(q, d, tu, au)
    inter_ref = up * np.maximum(gate, 0.0) ** 2
    got = inter.cpu().numpy().astype(np.float64)
    assert np.array_equal(got != 0, inter_ref.astype(np.float32) != 0)
    nz = inter_ref != 0
    assert (np.abs(got[nz] - inter_ref[nz]) <= 1e-6 * np.abs(inter_ref[nz]) + 1e-37).all()
    # output of the sub-layer: a top-k or rounding tie may fall differently on float32 intermediates
    assert np.abs(y.cpu().numpy() - y_ref).max() <= 2e-3 * np.abs(y_ref).max()
    # and the dense evaluation through the ordinary entry points gives the same bits
    codes, scale = a48.quant_int4(x.to(cuda_dev), EPS)
    g_d, u_d = a48.linear_multi([w["gate"], w["up"]], codes, scale, a48.ACT_INT4)
    prod = u_d * torch.relu(g_d) ** 2
    c8, s8, _ = a48.topk_quant_int8(prod, F // 2, EPS)
    y_dense = a48.linear(w["down"], c8, s8, a48.ACT_TOPK_INT8)
    assert torch.equal(inter, prod) and torch.equal(y, y_dense)
    if F % 4 == 0:
        assert torch.equal(a48.ffn_dense(w["gate"], w["up"], w["down"], x.to(cuda_dev), F // 2, EPS), y)


def test_ffn_gate_first_argument_checks(a48, cuda_dev):
    H, F = 128, 256
    w = {n: a48.pack_ternary(synth.latent_weights(a, b, seed=60 + i).to(cuda_dev), EPS, a48.LAYOUT_ALL)
         for i, (n, a, b) in enumerate((("gate", F, H), ("up", F, H), ("down", H, F)))}
    x9 = torch.zeros(9, H, device=cuda_dev)
    with pytest.raises(a48.A48Error) as e:
        a48.ffn_gate_first(w["gate"], w["up"], w["down"], x9, F // 2)
    assert e.value.code == 4  # more than 8 tokens
    with pytest.raises(a48.A48Error) as e:
        a48.ffn_gate_first(w["gate"], w["down"], w["down"], x9[:2], F // 2)
    assert e.value.code == 2  # shapes of the three matrices do not belong together
