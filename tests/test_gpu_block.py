"""Block forward on the GPU against the oracle (tiny block of the first benchmark configuration)."""
import numpy as np
import pytest
import torch

from paper_2411_04965_b200 import synth

pytestmark = pytest.mark.gpu

BLOCK_TOL = 2e-3  # max |a-b| / max |b| over the block output


def make_block(a48, dev, H, NH, F, seed, ctx_cap=0, scale=1.0):
    names = (("q", H, H), ("k", H, H), ("v", H, H), ("o", H, H), ("gate", F, H), ("up", F, H), ("down", H, F))
    lat = {n: synth.latent_weights(a, b, seed=seed * 10 + i) * scale for i, (n, a, b) in enumerate(names)}
    g1, g2 = synth.norm_gains(H, seed + 100), synth.norm_gains(H, seed + 101)
    packed = {n: a48.pack_ternary(lat[n].to(dev), 1e-5, a48.LAYOUT_ALL) for n in lat}
    blk = a48.Block(packed, g1.to(dev), g2.to(dev), n_heads=NH, k_o=H // 2, k_down=F // 2, ctx_cap=ctx_cap)
    return blk, lat, g1, g2


def rel_to_max(a, b):
    return float(np.abs(np.asarray(a, np.float64) - b).max() / np.abs(b).max())


def test_block_config1(a48, oracle, cuda_dev):
    # hidden 256, 4 heads of 64, FFN 768, 32 tokens, batch 1, N(0, 0.02) latents, 3 outlier channels x20, seed 0
    H, NH, F, T = 256, 4, 768, 32
    blk, lat, g1, g2 = make_block(a48, cuda_dev, H, NH, F, seed=0)
    x = synth.gaussian_outlier_activations(T, H, seed=0, count=3)
    y = blk.forward(x.to(cuda_dev), 1, T)
    ref, _, _ = oracle.block_forward(x.numpy(), {n: v.numpy() for n, v in lat.items()}, g1.numpy(), g2.numpy(),
                                     n_heads=NH, B=1, T=T, k_o=H // 2, k_down=F // 2, nthreads=4)
    assert rel_to_max(y.cpu().numpy(), ref) <= BLOCK_TOL


@pytest.mark.parametrize("B,T,pos0", [(2, 70, 0), (2, 3, 37), (1, 1, 64), (3, 20, 5)])
def test_block_batched_cached(a48, oracle, cuda_dev, B, T, pos0):
    # latents scaled up so that the sub-layers move the residual stream visibly
    H, NH, F, cap = 128, 2, 320, 128
    blk, lat, g1, g2 = make_block(a48, cuda_dev, H, NH, F, seed=3, ctx_cap=cap, scale=25.0)
    x = synth.gaussian_outlier_activations(B * T, H, seed=5, count=2)
    kc = synth.kv_cache(B, NH, cap, H // NH, seed=6)
    vc = synth.kv_cache(B, NH, cap, H // NH, seed=7)
    kc_d, vc_d = kc.to(cuda_dev), vc.to(cuda_dev)
    y = blk.forward(x.to(cuda_dev), B, T, pos0=pos0, kcache=kc_d, vcache=vc_d)
    ref, k_new, v_new = oracle.block_forward(x.numpy(), {n: v.numpy() for n, v in lat.items()}, g1.numpy(),
                                             g2.numpy(), n_heads=NH, B=B, T=T, pos0=pos0, ctx_cap=cap,
                                             kcache=kc.numpy(), vcache=vc.numpy(), k_o=H // 2, k_down=F // 2,
                                             nthreads=4)
    assert np.abs(ref - x.numpy()).max() > 0.05 * np.abs(ref).max()
    assert rel_to_max(y.cpu().numpy(), ref) <= BLOCK_TOL
    # the cache rows of the new positions now hold the rotated keys and the values
    assert rel_to_max(kc_d[:, :, pos0:pos0 + T].cpu().numpy(), k_new) <= 1e-5
    assert rel_to_max(vc_d[:, :, pos0:pos0 + T].cpu().numpy(), v_new) <= 1e-5
    # rows outside [pos0, pos0+T) are untouched
    assert torch.equal(kc_d[:, :, :pos0].cpu(), kc[:, :, :pos0])
    assert torch.equal(kc_d[:, :, pos0 + T:].cpu(), kc[:, :, pos0 + T:])
