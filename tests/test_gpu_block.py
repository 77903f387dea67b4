"""GPU parity of the encoder-block glue (LayerNorm, attention, residual input of the linear layer) and of the whole
pre-norm block with tiled linears against the CPU oracle -- small blocks element by element, the ViT-B shaped
configuration (128 images x 197 tokens, d = 768, 12 heads, MLP 3072, k = 8) on whole sampled images."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d", [(1, 8), (5, 33), (64, 768), (300, 1000), (9, 4096)])
@pytest.mark.parametrize("bf16", [True, False])
@pytest.mark.parametrize("affine", [False, True])
def test_layernorm_matches_oracle(T, d, bf16, affine):
    x = synth.normal(80, 0, T * d, 2.0).reshape(T, d) + 0.7
    xin = synth.to_bf16_bits(x) if bf16 else x
    g = synth.normal(80, 1, d).astype(np.float32) if affine else None
    b = synth.normal(80, 2, d).astype(np.float32) if affine else None
    ref = O.layernorm(xin, g, b)
    y = B.tbn_layernorm_fwd(to_dev(xin), None if g is None else to_dev(g), None if b is None else to_dev(b))
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "layernorm")


@pytest.mark.parametrize("path", [1, 2])          # 1: the warp-level MMA kernel, 2: the tcgen05 kernel
@pytest.mark.parametrize("Nb,S,heads", [(2, 197, 12), (3, 64, 2), (1, 17, 1), (2, 128, 3), (1, 208, 1), (2, 1, 2), (2, 65, 1),
                                        (3, 129, 2), (5, 16, 1), (2, 200, 2)])
def test_attention_matches_oracle(Nb, S, heads, path):
    qkv = synth.to_bf16_bits(synth.normal(81, 0, Nb * S * 3 * heads * 64, 1.2).reshape(Nb * S, 3 * heads * 64))
    ref = O.attention(qkv, Nb, S, heads, 64)
    assert B.lib().tbn_debug_force_attention_path(path) == 0
    try:
        out = torch.full((Nb * S, heads * 64), float("nan"), dtype=torch.bfloat16, device=DEV)
        B.tbn_attention_fwd(to_dev(qkv), Nb, S, heads, 64, out=out)
        torch.cuda.synchronize()
    finally:
        B.lib().tbn_debug_force_attention_path(0)
    assert_close(to_np64(out), ref, f"attention, path {path}")
    assert B.tbn_last_device_status() == (0, 0)


def test_attention_rejects_unsupported_shapes():
    q = torch.zeros((300, 3 * 64), dtype=torch.bfloat16, device=DEV)
    for args in ((1, 300, 1, 64), (1, 100, 2, 32)):
        with pytest.raises(B.TbnError) as e:
            B.tbn_attention_fwd(q, *args)
        assert e.value.status == -3


@pytest.mark.parametrize("path", [B.PATH_GENERIC, B.PATH_SMALL, B.PATH_TENSOR])
@pytest.mark.parametrize("T,m,n,k,act,bf16", [(7, 64, 64, 4, B.ACT_NONE, True), (300, 768, 3072, 8, B.ACT_NONE, True),
                                              (130, 520, 264, 4, B.ACT_GELU, True), (40, 256, 128, 2, B.ACT_RELU, False)])
def test_linear_with_residual_on_every_path(path, T, m, n, k, act, bf16):
    x, W = synth.linear_layer(82, T, n, m, x_bf16=bf16, w_sigma=n ** -0.5)
    words, al = O.prepare(W, k, True)
    res = synth.normal(82, 400, T * m).reshape(T, m)
    res_in = synth.to_bf16_bits(res) if bf16 else res
    ref = O.linear(x, words, k, al, True, m, n, act=act) + O.widen(res_in)
    y = B.tbn_linear_res_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), 1, to_dev(res_in), act=act, path=path)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, f"linear + residual, path {path}")


def _block_params(seed, d, mlp, ks, sigma=None):
    shapes = dict(qkv=(3 * d, d), proj=(d, d), fc1=(mlp, d), fc2=(d, mlp))
    layers, tiles, alphas = {}, [], []
    for l, (name, (m, n)) in enumerate(shapes.items()):
        W = synth.normal(seed, 1 + l, m * n, sigma if sigma else n ** -0.5)
        words, al = O.prepare(W, ks[l], True)
        layers[name] = dict(words=words, p=ks[l], alphas=al, per_tile=True, m=m, n=n)
        tiles.append(to_dev(words))
        alphas.append(to_dev(al))
    return layers, tiles, alphas


@pytest.mark.parametrize("Nb,S,d,heads,mlp,ks", [(3, 50, 128, 2, 256, [4, 2, 4, 2]), (2, 197, 192, 3, 384, [8, 8, 8, 8]),
                                                 (5, 17, 64, 1, 96, [2, 1, 4, 2])])
def test_small_block_matches_oracle(Nb, S, d, heads, mlp, ks):
    x = synth.to_bf16_bits(synth.normal(83, 0, Nb * S * d).reshape(Nb * S, d))
    layers, tiles, alphas = _block_params(83, d, mlp, ks)
    ref = O.vit_block(x, Nb, S, heads, layers)
    y = B.tbn_vit_block_fwd(to_dev(x), Nb, S, heads, mlp, tiles, ks, alphas, [1, 1, 1, 1])
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "encoder block")
    assert B.tbn_last_device_status() == (0, 0)


def test_vit_b_block_config_sampled_images():
    # 128 images x 197 tokens, d = 768, 12 heads, MLP 3072; tiles with k = 8, per-tile alpha, W ~ N(0, 0.02^2), seed 3.
    # Images are independent of one another, so the oracle runs whole sampled images.
    Nb, S, d, heads, mlp, ks = 128, 197, 768, 12, 3072, [8, 8, 8, 8]
    x = synth.to_bf16_bits(synth.normal(3, 0, Nb * S * d).reshape(Nb * S, d))
    layers, tiles, alphas = _block_params(3, d, mlp, ks, sigma=0.02)
    y = B.tbn_vit_block_fwd(to_dev(x), Nb, S, heads, mlp, tiles, ks, alphas, [1, 1, 1, 1])
    torch.cuda.synchronize()
    imgs = [0, 17, 38, 59, 64, 90, 111, 127]
    rows = np.concatenate([np.arange(i * S, (i + 1) * S) for i in imgs])
    ref = O.vit_block(x[rows], len(imgs), S, heads, layers)
    assert_close(to_np64(y[torch.from_numpy(rows).to(DEV)]), ref, "ViT-B block")
    assert B.tbn_last_device_status() == (0, 0)
