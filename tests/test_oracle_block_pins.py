"""Pins for the encoder-block glue of the CPU oracle (LayerNorm, multi-head attention, the pre-norm composition):
torch's own fp64 routines and hand-checkable special cases.  Runs without a GPU."""
import numpy as np
import torch

from oracle import tbn_oracle as O


def test_layernorm_matches_torch_and_closed_forms():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((9, 48)) * 3.0 + 1.5
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (48,), eps=1e-5).numpy()
    assert np.allclose(O.layernorm(x), ref, rtol=1e-12, atol=1e-12)
    g, b = rng.standard_normal(48), rng.standard_normal(48)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (48,), torch.from_numpy(g), torch.from_numpy(b), 1e-5).numpy()
    assert np.allclose(O.layernorm(x, g, b), ref, rtol=1e-12, atol=1e-12)
    y = O.layernorm(x)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-12) and np.allclose((y ** 2).mean(axis=1), 1, atol=1e-4)
    # a constant row has zero variance: the output is exactly zero (eps keeps the division finite)
    assert np.array_equal(O.layernorm(np.full((1, 8), 7.0)), np.zeros((1, 8)))


def test_attention_matches_torch_sdpa_and_special_cases():
    rng = np.random.default_rng(1)
    Nb, S, heads, dh = 2, 7, 3, 8
    qkv = rng.standard_normal((Nb * S, 3 * heads * dh))
    t = torch.from_numpy(qkv).reshape(Nb, S, 3, heads, dh).permute(2, 0, 3, 1, 4)        # (3, Nb, heads, S, dh)
    ref = torch.nn.functional.scaled_dot_product_attention(t[0], t[1], t[2])             # scale 1/sqrt(dh)
    ref = ref.permute(0, 2, 1, 3).reshape(Nb * S, heads * dh).numpy()
    assert np.allclose(O.attention(qkv, Nb, S, heads, dh), ref, rtol=1e-11, atol=1e-12)
    # zero queries: uniform attention, every output row is the mean of the values of its image and head
    z = qkv.copy().reshape(Nb, S, 3, heads, dh)
    z[:, :, 0] = 0.0
    out = O.attention(z.reshape(Nb * S, -1), Nb, S, heads, dh).reshape(Nb, S, heads, dh)
    assert np.allclose(out, np.broadcast_to(z[:, :, 2].mean(axis=1, keepdims=True), out.shape), atol=1e-13)
    # one key far closer than the others: the output is that key's value
    q1 = np.zeros((1 * 3, 3 * 1 * 4)); q1[:, 0:4] = [50.0, 0, 0, 0]
    q1[1, 4:8] = [50.0, 0, 0, 0]; q1[:, 8:12] = rng.standard_normal((3, 4))
    out = O.attention(q1, 1, 3, 1, 4)
    assert np.allclose(out, np.broadcast_to(q1[1, 8:12], (3, 4)), atol=1e-12)


def test_block_is_the_composition_and_images_are_independent():
    rng = np.random.default_rng(2)
    Nb, S, heads, d, mlp = 3, 5, 2, 16, 32
    x = rng.standard_normal((Nb * S, d)).astype(np.float32)
    layers, dense = {}, {}
    for name, (m, n, p) in dict(qkv=(3 * d, d, 4), proj=(d, d, 2), fc1=(mlp, d, 4), fc2=(d, mlp, 2)).items():
        W = (rng.standard_normal(m * n) * n ** -0.5).astype(np.float32)
        words, al = O.prepare(W, p, True)
        layers[name] = dict(words=words, p=p, alphas=al, per_tile=True, m=m, n=n)
        dense[name] = torch.from_numpy(O.expand(words, m * n, p, al, True).astype(np.float64).reshape(m, n))
    y = O.vit_block(x, Nb, S, heads, layers)
    # the same block with torch modules in fp64
    xt = torch.from_numpy(x.astype(np.float64))
    h1 = torch.nn.functional.layer_norm(xt, (d,))
    qkv = (h1 @ dense["qkv"].T).reshape(Nb, S, 3, heads, d // heads).permute(2, 0, 3, 1, 4)
    a = torch.nn.functional.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2]).permute(0, 2, 1, 3).reshape(Nb * S, d)
    x1 = xt + a @ dense["proj"].T
    f = torch.nn.functional.gelu(torch.nn.functional.layer_norm(x1, (d,)) @ dense["fc1"].T)
    ref = (x1 + f @ dense["fc2"].T).numpy()
    assert np.allclose(y, ref, rtol=1e-10, atol=1e-10)
    # images do not see one another: the block of image 1 alone equals its rows in the batch
    y1 = O.vit_block(x[S:2 * S], 1, S, heads, layers)
    assert np.allclose(y1, y[S:2 * S], rtol=1e-12, atol=1e-12)
    # the mirrored mode differs only by storage rounding
    ym = O.vit_block(x, Nb, S, heads, layers, mirror_bf16=True)
    assert 0 < np.abs(ym - y).max() < 0.05


def test_conv_stack_is_the_composition_of_torch_layers():
    rng = np.random.default_rng(3)
    Nb, H = 2, 8
    x = rng.random((Nb, 3, H, H)).astype(np.float32)
    W0 = (rng.standard_normal((8, 3, 3, 3)) * 0.3).astype(np.float32)
    convs, dense = [], []
    cin = 8
    for cout, p, stride in ((16, 4, 2), (32, 2, 2)):
        W = (rng.standard_normal(cout * cin * 9) * (2.0 / (cin * 9)) ** 0.5).astype(np.float32)
        words, al = O.prepare(W, p, True)
        convs.append(dict(words=words, p=p, alphas=al, per_tile=True, Cout=cout, Cin=cin, stride=stride))
        dense.append((torch.from_numpy(O.expand(words, W.size, p, al, True).astype(np.float64).reshape(cout, cin, 3, 3)), stride))
        cin = cout
    Wfc = (rng.standard_normal((5, 32)) * 0.2).astype(np.float32)
    y = O.conv_stack(x, W0, convs, Wfc)
    F = torch.nn.functional
    h = F.relu(F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(W0).double(), padding=1))
    for Wd, stride in dense:
        h = F.relu(F.conv2d(h, Wd, stride=stride, padding=1))
    ref = (F.adaptive_avg_pool2d(h, 1).flatten(1) @ torch.from_numpy(Wfc).double().T).numpy()
    assert y.shape == (Nb, 5) and np.allclose(y, ref, rtol=1e-11, atol=1e-11)
