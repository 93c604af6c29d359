"""Prefill attention on the tensor cores against the oracle's float64 definition (Section 2.1), through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

# The kernel forms every product of two fp32 numbers exactly enough (three bf16 parts each, fp32 accumulation), so what
# is left is fp32 rounding of a score s: 2^-24 |s| absolute, i.e. that much relative on its probability.  With N(0,1)
# heads of 36..128 dims |s| stays below about 8 (2e-6 would allow |s| = 30); the bound is on max|a-b| / max|b|.
ATTN_TOL = 2e-6


def _inputs(B, T, NH, hd, pos0, cap, seed, dev, amp=1.0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B * T, NH * hd, generator=g) * amp
    kc = synth.kv_cache(B, NH, cap, hd, seed=seed + 1) * amp
    vc = synth.kv_cache(B, NH, cap, hd, seed=seed + 2)
    return q, kc, vc


def _rel_to_max(a, b):
    return float(np.abs(np.asarray(a, np.float64) - b).max() / np.abs(b).max())


# one tile; two key tiles with the diagonal inside; several query tiles with a ragged last one; a cached prefix that
# is not a multiple of the tile; head dims that are padded (36 -> 64, 96 and 100 -> 128); three sequences
@pytest.mark.parametrize("B,T,NH,hd,pos0,cap", [(1, 9, 2, 64, 0, 16), (2, 70, 2, 64, 0, 128), (1, 200, 2, 128, 150, 352),
                                                (1, 260, 3, 96, 37, 300), (3, 129, 2, 36, 5, 200), (1, 300, 2, 100, 0, 300),
                                                (2, 128, 1, 128, 64, 192), (1, 64, 4, 128, 0, 64)])
def test_attention_prefill_matches_oracle(a48, oracle, cuda_dev, B, T, NH, hd, pos0, cap):
    q, kc, vc = _inputs(B, T, NH, hd, pos0, cap, seed=B * 1000 + T + hd, dev=cuda_dev)
    kc_d, vc_d = kc.to(cuda_dev), vc.to(cuda_dev)
    out = a48.attention_prefill(q.to(cuda_dev), kc_d, vc_d, B, T, pos0)
    assert a48.kernel_status() == [0, 0, 0, 0]
    ref = oracle.attention_causal(q.numpy(), kc.numpy(), vc.numpy(), B=B, T=T, n_heads=NH, pos0=pos0)
    assert _rel_to_max(out.cpu().numpy(), ref) <= ATTN_TOL
    assert torch.equal(kc_d.cpu(), kc) and torch.equal(vc_d.cpu(), vc)  # the caches are read only


def test_attention_prefill_large_scores(a48, oracle, cuda_dev):
    # heads scaled by 4: scores reach the forties, where fp32 rounding of a score alone is 3e-6 of its probability
    B, T, NH, hd = 1, 150, 2, 128
    q, kc, vc = _inputs(B, T, NH, hd, 0, T, seed=77, dev=cuda_dev, amp=4.0)
    out = a48.attention_prefill(q.to(cuda_dev), kc.to(cuda_dev), vc.to(cuda_dev), B, T)
    ref = oracle.attention_causal(q.numpy(), kc.numpy(), vc.numpy(), B=B, T=T, n_heads=NH)
    assert _rel_to_max(out.cpu().numpy(), ref) <= 2e-5


def test_attention_prefill_benchmark_shape_sampled(a48, oracle, cuda_dev):
    """32 heads of 128, 2 sequences of 4096 tokens (the launch shape the benchmark times, half its batch): a sample of
    (sequence, head) pairs against the oracle, every row of those."""
    B, T, NH, hd = 2, 4096, 32, 128
    q, kc, vc = _inputs(B, T, NH, hd, 0, T, seed=5, dev=cuda_dev)
    out = a48.attention_prefill(q.to(cuda_dev), kc.to(cuda_dev), vc.to(cuda_dev), B, T).cpu().numpy()
    assert a48.kernel_status() == [0, 0, 0, 0]
    for b, h in [(0, 0), (1, 31), (0, 17)]:
        ref = oracle.attention_causal(q[b * T:(b + 1) * T, h * hd:(h + 1) * hd].numpy(), kc[b:b + 1, h:h + 1].numpy(),
                                      vc[b:b + 1, h:h + 1].numpy(), B=1, T=T, n_heads=1)
        assert _rel_to_max(out[b * T:(b + 1) * T, h * hd:(h + 1) * hd], ref) <= ATTN_TOL


def test_attention_prefill_rejects_bad_arguments(a48, cuda_dev):
    q, kc, vc = _inputs(1, 16, 2, 160, 0, 16, seed=1, dev=cuda_dev)
    with pytest.raises(a48.A48Error) as e:
        a48.attention_prefill(q.to(cuda_dev), kc.to(cuda_dev), vc.to(cuda_dev), 1, 16,
                              workspace=torch.empty(1 << 20, dtype=torch.uint8, device=cuda_dev))
    assert e.value.code == 4  # head dims above 128 are not supported by this entry point
    q, kc, vc = _inputs(1, 16, 2, 64, 0, 16, seed=1, dev=cuda_dev)
    with pytest.raises(a48.A48Error) as e:
        a48.attention_prefill(q.to(cuda_dev), kc.to(cuda_dev), vc.to(cuda_dev), 1, 16, pos0=8)  # 8 + 16 > cap
    assert e.value.code == 2
    with pytest.raises(a48.A48Error) as e:
        a48.attention_prefill(q.to(cuda_dev), kc.to(cuda_dev), vc.to(cuda_dev), 1, 16,
                              workspace=torch.empty(64, dtype=torch.uint8, device=cuda_dev))
    assert e.value.code == 7
