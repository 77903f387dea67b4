"""Pins for the CPU oracle: every check compares it with something other than itself --
hand-worked values, closed forms, numpy / torch library routines on special cases,
brute-force enumeration, invariants of the method, and the numbers the paper prints.
Runs without a GPU."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits_of(words, q):
    i = np.arange(q)
    return ((words[i >> 5] >> (i & 31).astype(np.uint32)) & 1).astype(np.uint8)


def kron_expand(bits, p, alphas, per_tile):
    """Eq. 4 with numpy's Kronecker product, scaled tile by tile."""
    t = np.where(bits > 0, 1.0, -1.0)
    b = np.kron(np.ones(p), t)
    a = np.repeat(np.asarray(alphas, dtype=np.float64), bits.size) if per_tile else float(alphas[0])
    return b * a


# ----------------------------------------------------------------------------- aggregate
def test_aggregate_hand_example_distinguishes_chunk_sum_from_adjacent_sum():
    # p = 2, q = 4.  Column sums of the 2 x 4 view: (-2, -1, 2, 1) -> bits 0 0 1 1.
    # Summing adjacent pairs instead would give (-1, -1, -2, 4) -> 0 0 0 1.
    W = np.array([1, -2, 3, -4, -3, 1, -1, 5], dtype=np.float32)
    bits, mism = O.aggregate(W, 2)
    assert bits.tolist() == [0, 0, 1, 1] and mism == 0


def test_aggregate_p1_is_plain_sign():
    W = synth.normal(7, 1, 1000)
    bits, _ = O.aggregate(W, 1)
    assert np.array_equal(bits, (W > 0).astype(np.uint8))


def test_aggregate_ties_and_specials_give_minus_one():
    # sums: +0, -0, nan, exactly cancelling, tiny positive
    W = np.array([0.0, -0.0, np.nan, 2.5, 1e-30,
                  0.0, -0.0, 1.0, -2.5, 0.0], dtype=np.float32)
    bits, _ = O.aggregate(W, 2)
    assert bits.tolist() == [0, 0, 0, 0, 1]


def test_aggregate_sum_is_fp32_sequential():
    # fp32: (1e8 + 1) rounds to 1e8, minus 1e8 -> 0 -> bit 0; an fp64 sum gives 1 -> bit 1.
    W = np.array([1e8, 1.0, -1e8], dtype=np.float32)
    bits, mism = O.aggregate(W, 3)
    assert bits.tolist() == [0] and mism == 1
    # reversed order would give (-1e8 + 1) + 1e8 = 0 as well, but (1 + 1e8) - 1e8 = 0, and
    # placing the small term last keeps it: (1e8 - 1e8) + 1 = 1 -> bit 1
    bits, _ = O.aggregate(np.array([1e8, -1e8, 1.0], dtype=np.float32), 3)
    assert bits.tolist() == [1]


@pytest.mark.parametrize("p,q", [(1, 37), (2, 64), (4, 96), (8, 33), (3, 50)])
def test_aggregate_inverts_expand_and_negation_complements(p, q):
    rng = np.random.default_rng(p * 100 + q)
    bits = rng.integers(0, 2, q).astype(np.uint8)
    words = O.pack_bits(bits)
    B = O.expand(words, p * q, p, np.ones(1, np.float32), False)
    back, _ = O.aggregate(B, p)           # sums are +-p
    assert np.array_equal(back, bits)
    W = rng.standard_normal(p * q).astype(np.float32)
    b1, _ = O.aggregate(W, p)
    b2, _ = O.aggregate(-W, p)
    assert np.array_equal(b1 ^ 1, b2)     # no exact zeros in a continuous draw


def test_aggregate_matches_numpy_column_sum_when_no_rounding_is_possible():
    # small integers: every partial sum is exact in fp32, so order cannot matter
    rng = np.random.default_rng(3)
    p, q = 8, 257
    W = rng.integers(-5, 6, p * q).astype(np.float32)
    bits, _ = O.aggregate(W, p)
    assert np.array_equal(bits, (W.reshape(p, q).sum(axis=0) > 0).astype(np.uint8))


def test_aggregate_rejects_indivisible():
    with pytest.raises(ValueError):
        O.aggregate(np.zeros(10, np.float32), 3)


# ----------------------------------------------------------------------------- alpha
def test_alpha_hand_and_numpy():
    W = np.array([1, -2, 3, -4, -3, 1, -1, 5], dtype=np.float32)
    assert O.alpha(W, 2, False)[0] == np.float32(20.0 / 8.0)
    assert O.alpha(W, 2, True).tolist() == [2.5, 2.5]
    W = synth.normal(5, 1, 6 * 1000, 0.02)
    a = O.alpha(W, 6, True)
    ref = np.abs(W.astype(np.float64)).reshape(6, 1000).mean(axis=1)
    assert np.allclose(a, ref, rtol=1e-6)
    assert np.isclose(O.alpha(W, 6, False)[0], np.abs(W.astype(np.float64)).mean(), rtol=1e-6)
    # half-normal mean: sigma * sqrt(2/pi)
    assert abs(O.alpha(W, 6, False)[0] / (0.02 * np.sqrt(2 / np.pi)) - 1) < 0.03


def test_alpha_uses_contiguous_segments_not_strided_ones():
    # segment 0 is all ones, segment 1 all threes: contiguous reading -> (1, 3)
    S = np.concatenate([np.ones(10), 3 * np.ones(10)]).astype(np.float32)
    assert O.alpha(S, 2, True).tolist() == [1.0, 3.0]


# ----------------------------------------------------------------------------- pack
@pytest.mark.parametrize("q", [1, 31, 32, 33, 127, 128, 129, 1000])
def test_pack_matches_numpy_packbits_little(q):
    rng = np.random.default_rng(q)
    src = rng.standard_normal(q).astype(np.float32)
    src[::7] = 0.0                                    # zero is not > 0
    words = O.pack(src)
    assert words.size % 4 == 0 and words.size * 32 >= q
    ref = np.zeros(words.size * 4, dtype=np.uint8)
    pk = np.packbits((src > 0).astype(np.uint8), bitorder="little")
    ref[:pk.size] = pk
    assert np.array_equal(words.view(np.uint8), ref)   # little-endian words == LSB-first bytes
    assert np.array_equal(O.pack_bits((src > 0).astype(np.uint8)), words)


# ----------------------------------------------------------------------------- expand
@pytest.mark.parametrize("p,q,per_tile", [(1, 40, False), (4, 25, True), (2, 64, False), (8, 9, True)])
def test_expand_is_kronecker_product(p, q, per_tile):
    rng = np.random.default_rng(p + q)
    bits = rng.integers(0, 2, q).astype(np.uint8)
    al = (rng.random(p if per_tile else 1) + 0.5).astype(np.float32)
    B = O.expand(O.pack_bits(bits), p * q, p, al, per_tile)
    assert np.array_equal(B.astype(np.float64), kron_expand(bits, p, al, per_tile))


# ----------------------------------------------------------------------------- linear
SHAPES = [  # (T, m, n, p)
    (3, 8, 8, 1), (2, 8, 8, 2), (1, 8, 8, 8), (5, 128, 784, 4), (4, 10, 128, 1),
    (3, 96, 40, 6),   # q = 640: tile spans 16 whole rows
    (2, 6, 64, 4),    # q = 96: a tile ends mid-row
    (2, 4, 64, 8),    # q = 32: several tiles per row
    (3, 7, 33, 3),    # nothing divides anything
]


@pytest.mark.parametrize("T,m,n,p", SHAPES)
@pytest.mark.parametrize("per_tile", [False, True])
def test_linear_matches_numpy_matmul_on_kron_weights_and_alg1(T, m, n, p, per_tile):
    rng = np.random.default_rng(T * 1000 + m * 10 + p)
    W = rng.standard_normal(m * n).astype(np.float32)
    x = rng.standard_normal((T, n)).astype(np.float32)
    words, al = O.prepare(W, p, per_tile)
    y = O.linear(x, words, p, al, per_tile, m, n)
    Bk = kron_expand(bits_of(words, m * n // p), p, al, per_tile).reshape(m, n)
    ref = x.astype(np.float64) @ Bk.T                       # library routine, out x in orientation
    assert np.allclose(y, ref, rtol=1e-11, atol=1e-11)
    y1 = O.linear_alg1(x, words, p, al, per_tile, m, n)     # Algorithm 1 (index walk)
    assert np.allclose(y1, y, rtol=1e-12, atol=1e-12)
    yr = O.linear(x, words, p, al, per_tile, m, n, act=O.ACT_RELU)
    assert np.array_equal(yr, np.maximum(y, 0.0))
    assert np.allclose(O.linear_alg1(x, words, p, al, per_tile, m, n, relu=True), yr, atol=1e-12)


def test_k1_is_an_ordinary_binary_weight_layer():
    # XNOR-Net style: y = mean|W| * sign(W) x
    rng = np.random.default_rng(11)
    m, n, T = 24, 50, 6
    W = rng.standard_normal((m, n)).astype(np.float32)
    x = rng.standard_normal((T, n)).astype(np.float32)
    words, al = O.prepare(W, 1, False)
    y = O.linear(x, words, 1, al, False, m, n)
    a = np.float32(np.abs(W.astype(np.float64)).mean())
    ref = float(a) * (x.astype(np.float64) @ np.where(W > 0, 1.0, -1.0).T)
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("sign", [+1.0, -1.0, 0.0])
def test_constant_sign_weights_give_alpha_times_rowsum(sign):
    # all-positive W -> all-ones tile -> y = alpha_j * rowsum(x); zero / negative W -> bits 0 -> -alpha * rowsum
    rng = np.random.default_rng(5)
    m, n, p, T = 16, 12, 4, 3               # tile spans r = 4 whole rows
    mag = rng.random(m * n).astype(np.float32) + 0.1
    W = (sign * mag).astype(np.float32)
    x = rng.standard_normal((T, n)).astype(np.float32)
    words, al = O.prepare(W, p, True, A=mag)
    y = O.linear(x, words, p, al, True, m, n)
    rs = x.astype(np.float64).sum(axis=1, keepdims=True)
    s = 1.0 if sign > 0 else -1.0
    ref = s * rs * np.repeat(al.astype(np.float64), m // p)[None, :]
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)


def test_brute_force_all_tiles_tiny_layers():
    rng = np.random.default_rng(0)
    for (m, n, p) in [(2, 2, 1), (2, 2, 2), (4, 2, 4), (2, 4, 2), (4, 4, 4), (3, 2, 2), (2, 3, 3), (4, 3, 2)]:
        q = m * n // p
        x = rng.standard_normal((2, n))
        al = rng.random(p).astype(np.float32) + 0.5
        for tile in itertools.product([0, 1], repeat=q):
            bits = np.array(tile, dtype=np.uint8)
            y = O.linear(x, O.pack_bits(bits), p, al, True, m, n)
            for b in range(2):
                for i in range(m):
                    acc = 0.0
                    for j in range(n):
                        f = i * n + j
                        acc += float(al[f // q]) * (1.0 if tile[f % q] else -1.0) * x[b, j]
                    assert abs(acc - y[b, i]) < 1e-12


def test_retiling_invariance_and_linearity():
    rng = np.random.default_rng(21)
    m, n, p, c = 16, 24, 8, 4
    q = m * n // p
    bits = rng.integers(0, 2, q).astype(np.uint8)
    x = rng.standard_normal((3, n)).astype(np.float32)
    al_small = rng.random(p // c).astype(np.float32) + 0.5
    y_fine = O.linear(x, O.pack_bits(bits), p, np.repeat(al_small, c), True, m, n)
    y_coarse = O.linear(x, O.pack_bits(np.tile(bits, c)), p // c, al_small, True, m, n)
    assert np.allclose(y_fine, y_coarse, rtol=1e-13, atol=1e-13)
    # odd in the tile, linear in alpha
    y_neg = O.linear(x, O.pack_bits(bits ^ 1), p, np.repeat(al_small, c), True, m, n)
    assert np.allclose(y_neg, -y_fine, atol=1e-13)
    y_2 = O.linear(x, O.pack_bits(bits), p, 2 * np.repeat(al_small, c), True, m, n)
    assert np.allclose(y_2, 2 * y_fine, atol=1e-13)


def test_bf16_inputs_are_widened_exactly():
    x = synth.normal(3, 0, 64).reshape(4, 16)
    xb = synth.to_bf16_bits(x)
    assert np.array_equal(O.widen(xb), synth.bf16_bits_to_f32(xb).astype(np.float64))
    # round-to-nearest-even against torch
    t = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(xb.view(np.int16), t.view(torch.int16).numpy())
    assert np.array_equal(O.round_to_bf16(x.astype(np.float64)), t.to(torch.float64).numpy())


def test_gelu_matches_torch_erf_form():
    rng = np.random.default_rng(9)
    W = rng.standard_normal(8 * 8).astype(np.float32)
    x = rng.standard_normal((5, 8)).astype(np.float32)
    words, al = O.prepare(W, 2, True)
    y = O.linear(x, words, 2, al, True, 8, 8)
    yg = O.linear(x, words, 2, al, True, 8, 8, act=O.ACT_GELU)
    ref = torch.nn.functional.gelu(torch.from_numpy(y), approximate="none").numpy()
    assert np.allclose(yg, ref, rtol=1e-12, atol=1e-14)


def test_bias_is_added_before_activation():
    rng = np.random.default_rng(2)
    W = rng.standard_normal(6 * 4).astype(np.float32)
    x = rng.standard_normal((2, 4)).astype(np.float32)
    bias = rng.standard_normal(6)
    words, al = O.prepare(W, 2, False)
    y0 = O.linear(x, words, 2, al, False, 6, 4)
    y1 = O.linear(x, words, 2, al, False, 6, 4, bias=bias, act=O.ACT_RELU)
    assert np.allclose(y1, np.maximum(y0 + bias[None, :], 0), atol=1e-14)


# ----------------------------------------------------------------------------- conv
CONVS = [  # (Nb, Cout, Cin, kh, kw, p, stride, pad, H)
    (2, 2, 1, 3, 3, 2, 1, 1, 5),
    (1, 16, 8, 1, 1, 4, 1, 0, 7),
    (2, 8, 3, 3, 3, 2, 2, 1, 9),    # q = 108 = four filters of 27
    (2, 4, 3, 3, 3, 3, 2, 1, 9),    # q = 36: a tile ends inside a filter
    (1, 6, 4, 3, 3, 1, 1, 0, 6),
]


@pytest.mark.parametrize("Nb,Cout,Cin,kh,kw,p,stride,pad,H", CONVS)
def test_conv_matches_torch_conv2d_on_kron_weights(Nb, Cout, Cin, kh, kw, p, stride, pad, H):
    rng = np.random.default_rng(Cout * 7 + p)
    W = rng.standard_normal(Cout * Cin * kh * kw).astype(np.float32)
    x = rng.random((Nb, Cin, H, H + 1)).astype(np.float32)
    words, al = O.prepare(W, p, True)
    y = O.conv2d(x, words, p, al, True, Cout, Cin, kh, kw, stride, pad)
    Bk = kron_expand(bits_of(words, W.size // p), p, al, True).reshape(Cout, Cin, kh, kw)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(Bk),
                                     stride=stride, padding=pad).numpy()
    assert y.shape == ref.shape
    assert np.allclose(y, ref, rtol=1e-11, atol=1e-11)
    # the bias branch (one value per output channel, added before the activation) against torch's bias argument;
    # distinct per-channel values, so a bias indexed by anything but the channel fails
    bias = (rng.standard_normal(Cout) * 3.0 + np.arange(Cout)).astype(np.float64)
    for act, fn in ((O.ACT_NONE, lambda v: v), (O.ACT_RELU, torch.relu)):
        yb = O.conv2d(x, words, p, al, True, Cout, Cin, kh, kw, stride, pad, bias=bias, act=act)
        refb = fn(torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(Bk), bias=torch.from_numpy(bias),
                                             stride=stride, padding=pad)).numpy()
        assert np.allclose(yb, refb, rtol=1e-11, atol=1e-11)


def test_conv_paper_example_replicated_channels():
    # Sec. 4.1: one input channel, two output channels, 3x3, p = 2, single alpha
    #           -> the two output channels are identical.
    rng = np.random.default_rng(4)
    W = rng.standard_normal(2 * 1 * 3 * 3).astype(np.float32)
    x = rng.random((3, 1, 6, 6)).astype(np.float32)
    words, al = O.prepare(W, 2, False)
    y = O.conv2d(x, words, 2, al, False, 2, 1, 3, 3, 1, 1)
    assert np.array_equal(y[:, 0], y[:, 1])
    words, al2 = O.prepare(W, 2, True)
    y2 = O.conv2d(x, words, 2, al2, True, 2, 1, 3, 3, 1, 1)
    assert np.allclose(y2[:, 1] * float(al2[0]), y2[:, 0] * float(al2[1]), rtol=1e-12, atol=1e-14)


def test_conv_1x1_is_linear_over_pixels_and_im2col_agrees():
    rng = np.random.default_rng(8)
    Nb, Cin, Cout, H = 2, 8, 16, 5
    W = rng.standard_normal(Cout * Cin).astype(np.float32)
    x = rng.random((Nb, Cin, H, H)).astype(np.float32)
    words, al = O.prepare(W, 4, True)
    y = O.conv2d(x, words, 4, al, True, Cout, Cin, 1, 1, 1, 0)
    xl = x.transpose(0, 2, 3, 1).reshape(-1, Cin)
    yl = O.linear(xl, words, 4, al, True, Cout, Cin).reshape(Nb, H, H, Cout).transpose(0, 3, 1, 2)
    assert np.allclose(y, yl, rtol=1e-13, atol=1e-13)
    # 3x3, stride 2, pad 1 through an unfold (im2col) + the linear oracle
    Cout, kh, s, pad = 8, 3, 2, 1
    W = rng.standard_normal(Cout * Cin * kh * kh).astype(np.float32)
    words, al = O.prepare(W, 2, True)
    y = O.conv2d(x, words, 2, al, True, Cout, Cin, kh, kh, s, pad)
    cols = torch.nn.functional.unfold(torch.from_numpy(x).double(), kh, padding=pad, stride=s)
    cols = cols.permute(0, 2, 1).reshape(-1, Cin * kh * kh).numpy()
    yl = O.linear(cols, words, 2, al, True, Cout, Cin * kh * kh)
    Ho = y.shape[2]
    assert np.allclose(y, yl.reshape(Nb, Ho, Ho, Cout).transpose(0, 3, 1, 2), rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------- MLP
def test_mlp_is_the_composition_of_its_layers():
    rng = np.random.default_rng(13)
    dims, ks = [12, 16, 8, 3], [2, 4, 1]
    x = rng.standard_normal((4, dims[0])).astype(np.float32)
    layers, h = [], x.astype(np.float64)
    for l in range(3):
        W = rng.standard_normal(dims[l + 1] * dims[l]).astype(np.float32)
        words, al = O.prepare(W, ks[l], True)
        layers.append(dict(words=words, p=ks[l], alphas=al, per_tile=True, m=dims[l + 1], n=dims[l]))
        Bk = kron_expand(bits_of(words, W.size // ks[l]), ks[l], al, True).reshape(dims[l + 1], dims[l])
        h = h @ Bk.T
        if l < 2:
            h = np.maximum(h, 0)
    assert np.allclose(O.mlp(x, layers), h, rtol=1e-11, atol=1e-11)


def test_mlp_mirrored_mode_rounds_hidden_tensors_like_a_bf16_cast():
    # the diagnostic mode stores every hidden tensor as bf16: composition by hand with torch's own bf16 cast
    rng = np.random.default_rng(14)
    dims, ks = [16, 24, 12, 5], [2, 4, 1]
    x = rng.standard_normal((6, dims[0])).astype(np.float32)
    layers, h = [], x.astype(np.float64)
    for l in range(3):
        W = rng.standard_normal(dims[l + 1] * dims[l]).astype(np.float32)
        words, al = O.prepare(W, ks[l], True)
        layers.append(dict(words=words, p=ks[l], alphas=al, per_tile=True, m=dims[l + 1], n=dims[l]))
        Bk = kron_expand(bits_of(words, W.size // ks[l]), ks[l], al, True).reshape(dims[l + 1], dims[l])
        h = h @ Bk.T
        if l < 2:
            h = torch.from_numpy(np.maximum(h, 0)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    got = O.mlp(x, layers, mirror_bf16=True)
    assert np.allclose(got, h, rtol=1e-11, atol=1e-11)
    assert not np.allclose(got, O.mlp(x, layers), rtol=1e-6, atol=0)      # the rounding really happens
    # round_to_bf16 itself: ties go to even, values already representable are unchanged
    v = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 3.0e-5], dtype=np.float64)
    assert np.array_equal(O.round_to_bf16(v), torch.from_numpy(v).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy())


# ----------------------------------------------------------------------------- printed numbers
def _read_table(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            rows[k] = [float(t) for t in v]
    return rows


def test_table6_storage_and_memory_reproduced():
    t6 = _read_table("table6_mcu_kb.txt")
    acc = O.mcu_mlp_accounting()
    assert abs(acc["bwnn_memory"] / 1000 - t6["BWNN"][0]) < 0.0101
    assert abs(acc["bwnn_storage"] / 1000 - t6["BWNN"][1]) < 0.0101
    assert abs(acc["tbn_memory"] / 1000 - t6["TBN4"][0]) < 0.0101
    assert abs(acc["tbn_storage"] / 1000 - t6["TBN4"][1]) < 0.0101
    # Sec. 5.1: max memory is 58 % lower
    assert round(100 * (1 - acc["tbn_memory"] / acc["bwnn_memory"])) == 58
    # the packed-tile size the library allocates covers the stored bits
    assert O.tile_words(784 * 128 // 4) * 4 >= 784 * 128 // 4 // 8


def test_table7_parameter_memory_ratios():
    t7 = _read_table("table7_param_mb.txt")
    n_params = t7["FullPrecision"][0] * 1e6 / 4          # fp32 parameters
    bwnn_mb = O.layer_storage_bytes(int(n_params), 1, 0) / 1e6
    tbn_mb = O.layer_storage_bytes(int(n_params), 4, 0) / 1e6
    assert abs(bwnn_mb - t7["BWNN"][0]) < 0.05
    assert abs(tbn_mb - t7["TBN4"][0]) < 0.05
    assert round(t7["BWNN"][0] / t7["TBN4"][0], 1) == t7["TBN4"][1]
    assert t7["FullPrecision"][0] / t7["FP_Tiled4"][0] == t7["FP_Tiled4"][1]


# ----------------------------------------------------------------------------- full-precision tiles (Sec. 5.2)
@pytest.mark.parametrize("m,n,p", [(6, 4, 3), (8, 8, 2), (7, 33, 3), (12, 16, 4), (5, 10, 1)])
def test_fp_tile_expand_is_numpy_tile_and_definition(m, n, p):
    q = m * n // p
    t = synth.normal(7, 3, q, 0.5)
    B = O.expand_fp(t, m * n, p)
    assert np.array_equal(B, np.tile(t, p))                       # 1_p (x) t with a library routine
    for f in (0, 1, q - 1, q % (m * n), m * n - 1):               # B[f] = t[f mod q], the definition
        assert B[f] == t[f % q]
    if p > 1:
        with pytest.raises(ValueError):
            O.expand_fp(t, m * n + 1, p)


@pytest.mark.parametrize("T,m,n,p", [(3, 6, 4, 3), (5, 8, 8, 2), (2, 7, 33, 3), (4, 12, 16, 4)])
def test_fp_tile_linear_matches_numpy_matmul_brute_force_and_alg1(T, m, n, p):
    q = m * n // p
    t = synth.normal(8, 3, q, 0.5)
    x = synth.normal(8, 0, T * n).reshape(T, n)
    bias = synth.normal(8, 200, m, 0.1).astype(np.float64)
    y = O.linear_fp(x, t, p, m, n, bias=bias)
    Wfull = np.tile(t.astype(np.float64), p).reshape(m, n)
    assert np.allclose(y, x.astype(np.float64) @ Wfull.T + bias, rtol=1e-12, atol=1e-12)
    brute = np.zeros((T, m))
    for b in range(T):                                             # the definition, index by index
        for i in range(m):
            brute[b, i] = sum(float(t[(i * n + j) % q]) * float(x[b, j]) for j in range(n)) + bias[i]
    assert np.allclose(y, brute, rtol=1e-12, atol=1e-12)
    walk = O.linear_fp_alg1(x, t, p, m, n)                         # second, independently written routine
    assert np.allclose(y - bias, walk, rtol=1e-12, atol=1e-12)


def test_fp_tile_p1_is_an_ordinary_dense_layer_and_rows_repeat():
    T, m, n = 4, 16, 24
    W = synth.normal(9, 1, m * n, 0.3)
    x = synth.normal(9, 0, T * n).reshape(T, n)
    ref = torch.nn.functional.linear(torch.from_numpy(x).double(), torch.from_numpy(W).double().reshape(m, n)).numpy()
    assert np.allclose(O.linear_fp(x, W, 1, m, n), ref, rtol=1e-12, atol=1e-12)
    # a tile spanning whole rows: output row i + r repeats output row i (Sec. 4.1), with no scaling in between
    p = 4
    r = m // p
    y = O.linear_fp(x, W[: m * n // p], p, m, n, act=O.ACT_RELU)
    for j in range(1, p):
        assert np.array_equal(y[:, :r], y[:, j * r:(j + 1) * r])


def test_fp_tile_with_sign_values_equals_the_binary_layer():
    # a real-valued tile holding +-alpha is the binary tile with one scaling factor
    T, m, n, p = 3, 12, 20, 3
    W = synth.normal(10, 1, m * n, 0.02)
    x = synth.normal(10, 0, T * n).reshape(T, n)
    words, al = O.prepare(W, p, False)
    q = m * n // p
    t = np.where(bits_of(words, q) > 0, al[0], -al[0]).astype(np.float32)
    assert np.allclose(O.linear_fp(x, t, p, m, n), O.linear(x, words, p, al, False, m, n), rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------- generator
def test_generator_is_counter_based_and_calibrated():
    a = synth.normal(4, 0, 10000)
    b = synth.normal(4, 0, 5000, start=5000)
    assert np.array_equal(a[5000:], b)
    assert abs(float(a.mean())) < 0.05 and abs(float(a.std()) - 1) < 0.05
    u = synth.uniform(2, 0, 10000)
    assert 0 < u.min() and u.max() < 1 and abs(float(u.mean()) - 0.5) < 0.02
    assert not np.array_equal(synth.normal(4, 1, 100), a[:100])
    assert not np.array_equal(synth.normal(5, 0, 100), a[:100])
