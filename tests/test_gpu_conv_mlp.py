"""GPU parity: tiled convolution and the MLP chain against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu

# (Nb, Cout, Cin, kh, kw, k, stride, pad, H)
CONVS = [
    (3, 2, 1, 3, 3, 2, 1, 1, 5),        # the paper's replicated-channel example
    (2, 128, 64, 3, 3, 4, 1, 1, 32),
    (2, 128, 64, 3, 3, 4, 2, 1, 32),
    (2, 256, 128, 3, 3, 4, 2, 1, 16),
    (3, 16, 8, 1, 1, 4, 1, 0, 7),
    (2, 8, 3, 3, 3, 2, 2, 1, 9),        # q = 108: four filters of 27
    (2, 4, 3, 3, 3, 3, 2, 1, 9),        # q = 36: a tile ends inside a filter
]


@pytest.mark.parametrize("Nb,Cout,Cin,kh,kw,k,stride,pad,H", CONVS)
@pytest.mark.parametrize("per_tile", [False, True])
def test_conv_matches_oracle(Nb, Cout, Cin, kh, kw, k, stride, pad, H, per_tile):
    x, W = synth.conv_layer(2, Nb, Cin, H, H, Cout, kh, kw)
    words, al = O.prepare(W, k, per_tile)
    ref = O.conv2d(x, words, k, al, per_tile, Cout, Cin, kh, kw, stride, pad, act=O.ACT_RELU)
    for path in (B.PATH_GENERIC, B.PATH_AUTO):
        y = B.tbn_conv2d_fwd(to_dev(x), Cout, kh, kw, stride, pad, to_dev(words), k, to_dev(al), int(per_tile),
                             act=B.ACT_RELU, path=path)
        torch.cuda.synchronize()
        assert_close(to_np64(y), ref, f"conv path {path}")


def test_conv_replicated_channels_are_bit_identical():
    # Sec. 4.1: single alpha, no bias -> the k copies of a filter give identical channels
    x, W = synth.conv_layer(5, 4, 8, 12, 12, 32, 3, 3)
    words, al = O.prepare(W, 4, False)
    y = B.tbn_conv2d_fwd(to_dev(x), 32, 3, 3, 1, 1, to_dev(words), 4, to_dev(al), 0)
    for j in range(1, 4):
        assert torch.equal(y[:, :8], y[:, 8 * j:8 * (j + 1)])


def test_conv_fp32_in_out_and_bias():
    x, W = synth.conv_layer(6, 2, 4, 9, 9, 8, 3, 3, x_bf16=False)
    bias = synth.normal(6, 200, 8)
    words, al = O.prepare(W, 2, True)
    ref = O.conv2d(x, words, 2, al, True, 8, 4, 3, 3, 2, 1, bias=bias.astype(np.float64))
    y = B.tbn_conv2d_fwd(to_dev(x), 8, 3, 3, 2, 1, to_dev(words), 2, to_dev(al), 1, bias=to_dev(bias))
    assert y.dtype == torch.float32
    assert_close(to_np64(y), ref, "conv fp32")


def _mlp_layers(Ws, ks):
    layers, tiles, alphas = [], [], []
    for W, k in zip(Ws, ks):
        m, n = W.shape
        words, al = O.prepare(W, k, True)
        layers.append(dict(words=words, p=k, alphas=al, per_tile=True, m=m, n=n))
        tiles.append(to_dev(words))
        alphas.append(to_dev(al))
    return layers, tiles, alphas


@pytest.mark.parametrize("T", [1, 7, 200])
def test_mlp_small_matches_oracle(T):
    dims, ks = [64, 128, 96, 10], [4, 8, 1]
    x = synth.to_bf16_bits(synth.normal(1, 0, T * dims[0]).reshape(T, dims[0]))
    Ws = [synth.normal(1, 1 + l, dims[l + 1] * dims[l], 0.1).reshape(dims[l + 1], dims[l]) for l in range(3)]
    layers, tiles, alphas = _mlp_layers(Ws, ks)
    ref = O.mlp(x, layers)
    y = B.tbn_mlp_fwd(to_dev(x), dims, tiles, ks, alphas, [1, 1, 1])
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, f"mlp T={T}")


def test_mlp_benchmark_config_sampled_rows():
    # 1024 -> 2048 -> 2048 -> 10, k = 8 on the hidden layers, batch 4096: all rows on the GPU,
    # a seeded sample of rows through the oracle
    c = synth.config_mlp(T=4096)
    layers, tiles, alphas = _mlp_layers(c["Ws"], c["ks"])
    y = B.tbn_mlp_fwd(to_dev(c["x"]), c["dims"], tiles, c["ks"], alphas, [1, 1, 1])
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(0).choice(4096, 48, replace=False))
    ref = O.mlp(c["x"][rows], layers)
    assert_close(to_np64(y)[rows], ref, "mlp config")
    # tiles built on the GPU equal the oracle's
    for W, k, t in zip(c["Ws"], c["ks"], tiles):
        t2, _ = B.tbn_aggregate_tile(to_dev(W), k, B.ALPHA_PER_TILE)
        assert torch.equal(t2, t)


# (Nb, Cout, Cin, k, stride, pad, H, W): shapes the tensor-core 3x3 kernel takes
TENSOR_CONVS = [
    (2, 128, 64, 4, 1, 1, 32, 32),     # row bands of one image
    (3, 128, 64, 4, 2, 1, 32, 32),
    (7, 256, 128, 4, 2, 1, 16, 16),    # two images per tile, odd batch (ragged last group)
    (5, 32, 16, 2, 1, 1, 4, 4),        # five whole images per tile
    (2, 200, 32, 4, 1, 1, 12, 20),     # ragged channel block, non-square image
    (3, 32, 16, 2, 1, 0, 10, 10),      # no padding
    (3, 32, 16, 2, 2, 0, 11, 13),      # stride 2 without padding
    (2, 64, 48, 1, 2, 2, 9, 9),        # padding 2, k = 1
    (1, 16, 16, 16, 1, 1, 40, 170),    # widest row that still fits, one distinct filter
    (3, 32, 16, 2, 2, 1, 13, 16),      # 8-pixel output rows stored in pairs, odd output height (7 x 8)
    (2, 32, 16, 2, 1, 1, 9, 16),       # 16-pixel rows, odd height
    (1, 32, 16, 2, 1, 1, 6, 48),       # three 16-pixel items per row
    # 32 distinct filters on 256 / 512 channels: the channel blocks share one accumulator block, written 2 / 4 times
    (2, 256, 16, 8, 1, 1, 6, 24),      # 8-pixel pieces (24-pixel rows)
    (2, 512, 16, 16, 1, 1, 12, 20),    # element-wise stores (20-pixel rows)
    (3, 384, 32, 6, 2, 1, 16, 32),     # 64 filters on three channel blocks, 16-pixel items
]


@pytest.mark.parametrize("Nb,Cout,Cin,k,stride,pad,H,W", TENSOR_CONVS)
def test_tensor_conv_matches_oracle(Nb, Cout, Cin, k, stride, pad, H, W):
    x, Wt = synth.conv_layer(3, Nb, Cin, H, W, Cout, 3, 3)
    for per_tile in (False, True):
        words, al = O.prepare(Wt, k, per_tile)
        ref = O.conv2d(x, words, k, al, per_tile, Cout, Cin, 3, 3, stride, pad, act=O.ACT_RELU)
        y = B.tbn_conv2d_fwd(to_dev(x), Cout, 3, 3, stride, pad, to_dev(words), k, to_dev(al), int(per_tile),
                             act=B.ACT_RELU, path=B.PATH_TENSOR)
        torch.cuda.synchronize()
        assert_close(to_np64(y), ref, f"tensor conv {Cout}x{Cin} s{stride} p{pad} {H}x{W}")
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("act", [B.ACT_NONE, B.ACT_GELU])
def test_tensor_conv_other_activations_and_bias(act):
    # the ReLU epilogue clamps inside the bf16 conversion; the other activations take their own branches
    x, Wt = synth.conv_layer(9, 3, 32, 16, 16, 64, 3, 3)
    words, al = O.prepare(Wt, 4, True)
    bias = synth.normal(9, 300, 64, 0.3)
    ref = O.conv2d(x, words, 4, al, True, 64, 32, 3, 3, 1, 1, bias=bias.astype(np.float64), act=act)
    y = B.tbn_conv2d_fwd(to_dev(x), 64, 3, 3, 1, 1, to_dev(words), 4, to_dev(al), 1, bias=to_dev(bias), act=act,
                         path=B.PATH_TENSOR)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, f"tensor conv act {act}")


def test_tensor_conv_fp32_bias_and_agrees_with_generic():
    x, Wt = synth.conv_layer(8, 3, 32, 14, 14, 64, 3, 3, x_bf16=False)
    bias = synth.normal(8, 200, 64)
    words, al = O.prepare(Wt, 4, True)
    ref = O.conv2d(x, words, 4, al, True, 64, 32, 3, 3, 1, 1, bias=bias.astype(np.float64), act=O.ACT_GELU)
    args = (to_dev(x), 64, 3, 3, 1, 1, to_dev(words), 4, to_dev(al), 1)
    yt = B.tbn_conv2d_fwd(*args, bias=to_dev(bias), act=B.ACT_GELU, path=B.PATH_TENSOR)
    yg = B.tbn_conv2d_fwd(*args, bias=to_dev(bias), act=B.ACT_GELU, path=B.PATH_GENERIC)
    assert yt.dtype == torch.float32
    assert_close(to_np64(yt), ref, "tensor conv fp32")
    assert_close(to_np64(yt), to_np64(yg), "tensor conv vs generic")


def test_tensor_conv_rejects_what_it_cannot_take():
    x, Wt = synth.conv_layer(2, 1, 8, 6, 6, 8, 3, 3)          # 8 input channels: not a multiple of 16
    words, al = O.prepare(Wt, 2, True)
    with pytest.raises(B.TbnError) as e:
        B.tbn_conv2d_fwd(to_dev(x), 8, 3, 3, 1, 1, to_dev(words), 2, to_dev(al), 1, path=B.PATH_TENSOR)
    assert e.value.status == -3


@pytest.mark.parametrize("T,dims,ks,act", [(200, [64, 256, 128, 24], [4, 8, 1], B.ACT_RELU),
                                           (37, [128, 512, 512, 64], [8, 4, 2], B.ACT_NONE),
                                           (1000, [256, 1024, 16], [16, 2], B.ACT_RELU),
                                           # thin last layers (1, 16 and 10 distinct rows): the CUDA-core head kernel
                                           (513, [64, 512, 1], [8, 1], B.ACT_RELU),
                                           (64, [128, 256, 16], [4, 1], B.ACT_NONE),
                                           (33, [256, 1024, 1024, 10], [8, 8, 1], B.ACT_RELU),
                                           # narrow hidden layer + thin last layer: both in one launch (16- and
                                           # 32-token blocks, ragged batch, 16 distinct rows written twice, 96 rows)
                                           (4790, [64, 512, 512, 10], [8, 2, 1], B.ACT_RELU),
                                           (70, [64, 256, 256, 32], [4, 4, 2], B.ACT_NONE),
                                           (45, [128, 256, 192, 7], [4, 2, 1], B.ACT_RELU)])
def test_mlp_compact_chain_matches_oracle_and_layerwise_chain(T, dims, ks, act):
    # shapes whose hidden tiles span whole rows with compact widths that are multiples of 8: the hidden layers'
    # k-fold broadcast stays out of HBM (compact chain); the layer-by-layer chain must give the same result
    L = len(ks)
    x = synth.to_bf16_bits(synth.normal(5, 0, T * dims[0]).reshape(T, dims[0]))
    Ws = [synth.normal(5, 1 + l, dims[l + 1] * dims[l], 0.05).reshape(dims[l + 1], dims[l]) for l in range(L)]
    layers, tiles, alphas = _mlp_layers(Ws, ks)
    ref = O.mlp(x, layers, hidden_act=O.ACT_RELU if act == B.ACT_RELU else O.ACT_NONE)
    y = B.tbn_mlp_fwd(to_dev(x), dims, tiles, ks, alphas, [1] * L, hidden_act=act)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "compact chain")
    B.tbn_debug_force_mlp_layerwise(True)
    try:
        y2 = B.tbn_mlp_fwd(to_dev(x), dims, tiles, ks, alphas, [1] * L, hidden_act=act)
        torch.cuda.synchronize()
    finally:
        B.tbn_debug_force_mlp_layerwise(False)
    assert_close(to_np64(y2), ref, "layer-by-layer chain")
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("T,dims,ks,act", [(512, [512, 4096, 2048, 10], [8, 8, 1], B.ACT_RELU),
                                           (300, [1024, 4096, 4096, 64], [4, 16, 2], B.ACT_NONE)])
def test_mlp_compact_chain_wide_layers_fan_in_scaled(T, dims, ks, act):
    # hidden widths of 4096 and folds over 512 / 1024 rows, weights ~N(0, 1/n) so that the hidden activations stay
    # of order one, as they do in a trained network: the compact chain must hold the stated tolerance here too
    L = len(ks)
    x = synth.to_bf16_bits(synth.normal(15, 0, T * dims[0]).reshape(T, dims[0]))
    Ws = [synth.normal(15, 1 + l, dims[l + 1] * dims[l], dims[l] ** -0.5).reshape(dims[l + 1], dims[l]) for l in range(L)]
    layers, tiles, alphas = _mlp_layers(Ws, ks)
    ref = O.mlp(x, layers, hidden_act=O.ACT_RELU if act == B.ACT_RELU else O.ACT_NONE)
    y = B.tbn_mlp_fwd(to_dev(x), dims, tiles, ks, alphas, [1] * L, hidden_act=act)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "wide compact chain")
    B.tbn_debug_force_mlp_layerwise(True)
    try:
        y2 = B.tbn_mlp_fwd(to_dev(x), dims, tiles, ks, alphas, [1] * L, hidden_act=act)
        torch.cuda.synchronize()
    finally:
        B.tbn_debug_force_mlp_layerwise(False)
    assert_close(to_np64(y2), ref, "wide layer-by-layer chain")
    assert B.tbn_last_device_status() == (0, 0)


def test_mlp_compact_chain_replayed_from_a_graph_and_back_to_back():
    # the compact chain runs its folds on the library's side stream (fork after the caller's queued work, join before
    # layer 1).  Calls queued back to back share one workspace, and a captured graph must carry the fork and the join:
    # both must reproduce the result of a single eager call bit for bit.
    T, dims, ks = 300, [256, 512, 512, 10], [8, 8, 1]
    x = to_dev(synth.to_bf16_bits(synth.normal(6, 0, T * dims[0]).reshape(T, dims[0])))
    Ws = [synth.normal(6, 1 + l, dims[l + 1] * dims[l], 0.05).reshape(dims[l + 1], dims[l]) for l in range(3)]
    layers, tiles, alphas = _mlp_layers(Ws, ks)
    ws = torch.empty(B.tbn_mlp_workspace_bytes(T, dims, ks, B.BF16), dtype=torch.uint8, device=DEV)
    y0 = B.tbn_mlp_fwd(x, dims, tiles, ks, alphas, [1, 1, 1], workspace=ws).clone()
    torch.cuda.synchronize()
    # other parameters through the same workspace in between: the second call's folds must not run early
    Ws2 = [synth.normal(7, 1 + l, dims[l + 1] * dims[l], 0.05).reshape(dims[l + 1], dims[l]) for l in range(3)]
    _, tiles2, alphas2 = _mlp_layers(Ws2, ks)
    ys = []
    for _ in range(3):
        B.tbn_mlp_fwd(x, dims, tiles2, ks, alphas2, [1, 1, 1], workspace=ws)
        ys.append(B.tbn_mlp_fwd(x, dims, tiles, ks, alphas, [1, 1, 1], workspace=ws).clone())
    torch.cuda.synchronize()
    for y in ys:
        assert torch.equal(y, y0)
    stream, g = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    yg = torch.empty_like(y0)
    with torch.cuda.graph(g, stream=stream):
        B.tbn_mlp_fwd(x, dims, tiles2, ks, alphas2, [1, 1, 1], workspace=ws, y=yg)
        B.tbn_mlp_fwd(x, dims, tiles, ks, alphas, [1, 1, 1], workspace=ws, y=yg)
    for _ in range(2):
        yg.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(yg, y0)
    assert B.tbn_last_device_status() == (0, 0)
