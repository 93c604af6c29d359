"""The allocation-free decode entry point against the ordinary one.

bitnet_a48_linear_decode_static is for callers that must not allocate device memory once they are running
(a plugin inside a process whose memory pool is fixed at start-up, a loop that may not take allocator locks):
its scratch is an array inside the library.  The test calls it through the C ABI twice in a row on different
inputs and expects the very bits bitnet_a48_linear_ex gives with the decode kernel and a caller-provided
scratch; the second call also shows that the shared array is left usable by the first.
"""
import pytest
import torch

from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5


def test_static_scratch_decode_matches_workspace_decode(a48, cuda_dev):
    N, K = 2048, 8640  # fewer 16-row tiles than SMs: neighbouring pieces share tiles, so the scratch is really used
    w = a48.pack_ternary(synth.latent_weights(N, K, seed=5).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    for call, M in enumerate((1, 5)):
        x = synth.student_t3(M, K, seed=90 + call).to(cuda_dev)
        codes, scale, _ = a48.topk_quant_int8(x, K // 2, EPS)
        expected = a48.linear(w, codes, scale, a48.ACT_TOPK_INT8, a48.ALGO_DECODE)
        got = torch.full((M, N), float("nan"), device=cuda_dev)
        a48.linear_decode_static(w, codes, scale, got)
        torch.cuda.synchronize()
        assert torch.equal(got, expected), f"call {call}: outputs differ"
    assert a48.kernel_status() == [0, 0, 0, 0]


def test_static_scratch_decode_at_its_limit_and_after_a_smaller_call(a48, cuda_dev):
    # 16384 output features fill the built-in array exactly; the call before it used (and cleared) only a small part
    # of the array, so the large call meets a region no earlier call of this test has cleared
    small = a48.pack_ternary(synth.latent_weights(320, 2048, seed=8).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    large = a48.pack_ternary(synth.latent_weights(16384, 256, seed=9).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    for w, M in ((small, 3), (large, 8), (small, 1), (large, 2)):
        x = synth.gaussian_outlier_activations(M, w.K, seed=91 + M).to(cuda_dev)
        codes, scale = a48.quant_int4(x, EPS)
        expected = a48.linear(w, codes, scale, a48.ACT_INT4, a48.ALGO_DECODE)
        got = torch.full((M, w.N), float("nan"), device=cuda_dev)
        a48.linear_decode_static(w, codes, scale, got)
        torch.cuda.synchronize()
        assert torch.equal(got, expected)
    assert a48.kernel_status() == [0, 0, 0, 0]


def test_static_scratch_decode_rejects_what_it_cannot_hold(a48, cuda_dev):
    wide = a48.pack_ternary(synth.latent_weights(16400, 128, seed=6).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    codes = torch.zeros(1, 128, dtype=torch.int8, device=cuda_dev)
    scale = torch.ones(1, device=cuda_dev)
    with pytest.raises(a48.A48Error) as e:
        a48.linear_decode_static(wide, codes, scale, torch.empty(1, 16400, device=cuda_dev))
    assert e.value.code == 8  # BITNET_A48_ERR_LIMIT: more output features than the built-in scratch covers
    small = a48.pack_ternary(synth.latent_weights(64, 128, seed=7).to(cuda_dev), EPS, a48.LAYOUT_DECODE)
    codes9 = torch.zeros(9, 128, dtype=torch.int8, device=cuda_dev)
    with pytest.raises(a48.A48Error) as e:
        a48.linear_decode_static(small, codes9, torch.ones(9, device=cuda_dev), torch.empty(9, 64, device=cuda_dev))
    assert e.value.code == 4  # BITNET_A48_ERR_UNSUPPORTED: more than 8 tokens
