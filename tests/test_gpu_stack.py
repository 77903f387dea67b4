"""GPU parity of the ResNet-style convolution stack as a stack: full-precision first convolution, two tiled 3x3
convolutions fed with the activations the previous layer produced, global average pooling and a full-precision
classifier -- against the CPU oracle.  Also the two untiled end layers on their own."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("Nb,Cin,H,W,Cout,k,stride,pad,bf16", [(2, 3, 32, 32, 64, 3, 1, 1, True), (3, 3, 9, 11, 10, 3, 2, 1, False),
                                                              (2, 1, 7, 7, 4, 5, 1, 2, True), (1, 8, 6, 6, 16, 1, 1, 0, False),
                                                              (2, 3, 12, 12, 9, 3, 1, 0, True)])
def test_dense_conv_matches_oracle(Nb, Cin, H, W, Cout, k, stride, pad, bf16):
    x = synth.uniform(90, 0, Nb * Cin * H * W).reshape(Nb, Cin, H, W)
    xin = synth.to_bf16_bits(x) if bf16 else x
    Wt = synth.normal(90, 1, Cout * Cin * k * k, (2.0 / (Cin * k * k)) ** 0.5).reshape(Cout, Cin, k, k)
    bias = synth.normal(90, 200, Cout, 0.1)
    ref = O.conv2d_dense(xin, Wt, Cout, Cin, k, k, stride, pad, bias=bias.astype(np.float64), act=O.ACT_RELU)
    y = B.tbn_conv2d_dense_fwd(to_dev(xin), to_dev(Wt), stride, pad, bias=to_dev(bias), act=B.ACT_RELU)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "dense conv")


@pytest.mark.parametrize("Nb,C,H,W", [(3, 5, 1, 1), (2, 256, 8, 8), (1, 7, 5, 9)])
def test_global_avgpool_matches_numpy_mean(Nb, C, H, W):
    x = synth.to_bf16_bits(synth.normal(91, 0, Nb * C * H * W).reshape(Nb, C, H, W))
    y = B.tbn_global_avgpool_fwd(to_dev(x), y_dtype=B.F32)
    torch.cuda.synchronize()
    ref = O.widen(x).mean(axis=(2, 3))
    assert np.allclose(to_np64(y), ref, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("Nb,C,H,W,out_f,bf16", [(3, 5, 1, 1, 2, True), (2, 256, 8, 8, 10, True), (1, 7, 5, 9, 33, False), (4, 300, 4, 4, 10, True)])
def test_avgpool_plus_classifier_in_one_launch(Nb, C, H, W, out_f, bf16):
    x = synth.normal(93, 0, Nb * C * H * W).reshape(Nb, C, H, W)
    xin = synth.to_bf16_bits(x) if bf16 else x
    Wfc = synth.normal(93, 1, out_f * C, C ** -0.5).reshape(out_f, C)
    bias = synth.normal(93, 2, out_f, 0.1)
    ref = O.widen(xin).mean(axis=(2, 3)) @ Wfc.astype(np.float64).T + bias.astype(np.float64)
    y = B.tbn_avgpool_linear_fwd(to_dev(xin), to_dev(Wfc), to_dev(bias))
    y0 = B.tbn_avgpool_linear_fwd(to_dev(xin), to_dev(Wfc))
    torch.cuda.synchronize()
    assert np.allclose(to_np64(y), ref, rtol=1e-5, atol=1e-5)
    assert np.allclose(to_np64(y0), ref - bias.astype(np.float64), rtol=1e-5, atol=1e-5)
    # and it agrees with the two separate calls (whose classifier rounds its operands to bf16 on the tensor path)
    two = B.tbn_linear_fp_tile_fwd(B.tbn_global_avgpool_fwd(to_dev(xin), y_dtype=B.F32), out_f, to_dev(Wfc).reshape(-1), 1, y_dtype=B.F32)
    torch.cuda.synchronize()
    assert_close(to_np64(two), to_np64(y0), "separate calls against the fused one")


def run_stack(x_dev, W0_dev, convs_dev, Wfc_dev, fused_tail=False):
    h = B.tbn_conv2d_dense_fwd(x_dev, W0_dev, 1, 1, act=B.ACT_RELU)
    for (tile, alpha, Cout, k, stride) in convs_dev:
        h = B.tbn_conv2d_fwd(h, Cout, 3, 3, stride, 1, tile, k, alpha, B.ALPHA_PER_TILE, act=B.ACT_RELU)
    if fused_tail:
        return B.tbn_avgpool_linear_fwd(h, Wfc_dev)
    pooled = B.tbn_global_avgpool_fwd(h, y_dtype=B.F32)
    return B.tbn_linear_fp_tile_fwd(pooled, Wfc_dev.shape[0], Wfc_dev.reshape(-1), 1, y_dtype=B.F32)


def make_stack(seed, chans, k):
    """Weights of a stack 3 -> chans[0] (dense) -> chans[1] -> chans[2] (tiled, stride 2) -> 10 classes (dense)."""
    W0 = synth.normal(seed, 1, chans[0] * 27, (2.0 / 27) ** 0.5).reshape(chans[0], 3, 3, 3)
    convs, convs_dev = [], []
    for l in (1, 2):
        cin, cout = chans[l - 1], chans[l]
        W = synth.normal(seed, 1 + l, cout * cin * 9, (2.0 / (cin * 9)) ** 0.5)
        words, al = O.prepare(W, k, True)
        convs.append(dict(words=words, p=k, alphas=al, per_tile=True, Cout=cout, Cin=cin, stride=2))
        convs_dev.append((to_dev(words), to_dev(al), cout, k, 2))
    Wfc = synth.normal(seed, 4, 10 * chans[2], chans[2] ** -0.5).reshape(10, chans[2])
    return W0, convs, convs_dev, Wfc


@pytest.mark.parametrize("Nb,H,chans,k", [(3, 16, (16, 32, 64), 4), (2, 12, (8, 24, 40), 2)])
def test_small_stack_matches_oracle(Nb, H, chans, k):
    x = synth.to_bf16_bits(synth.uniform(92, 0, Nb * 3 * H * H).reshape(Nb, 3, H, H))
    W0, convs, convs_dev, Wfc = make_stack(92, chans, k)
    ref = O.conv_stack(x, W0, convs, Wfc)
    y = run_stack(to_dev(x), to_dev(W0), convs_dev, to_dev(Wfc))
    yf = run_stack(to_dev(x), to_dev(W0), convs_dev, to_dev(Wfc), fused_tail=True)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "conv stack")
    assert_close(to_np64(yf), ref, "conv stack, pooling and classifier in one launch")


def test_conv_stack_config_sampled_images():
    # 32x32x3 inputs ~U(0,1), batch 256, 3x3 convolutions 3 -> 64 (full precision) -> 128 -> 256 (tiled, k = 4, stride 2,
    # per-filter-block alpha), global average pooling, full-precision classifier; Kaiming-normal weights, seed 2
    Nb = 256
    x = synth.to_bf16_bits(synth.uniform(2, 0, Nb * 3 * 32 * 32).reshape(Nb, 3, 32, 32))
    W0, convs, convs_dev, Wfc = make_stack(2, (64, 128, 256), 4)
    y = run_stack(to_dev(x), to_dev(W0), convs_dev, to_dev(Wfc))
    torch.cuda.synchronize()
    imgs = np.array([0, 77, 128, 255])
    ref = O.conv_stack(x[imgs], W0, convs, Wfc)
    assert_close(to_np64(y)[imgs], ref, "conv stack config")
    assert B.tbn_last_device_status() == (0, 0)
