"""GPU parity on seeded random shapes: every kernel family that accepts the shape against the CPU oracle, with random
activation, bias, output dtype and alpha mode.  Complements the hand-picked shape lists of the other files."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu

PATHS = (B.PATH_AUTO, B.PATH_TENSOR, B.PATH_SMALL, B.PATH_GENERIC)


@pytest.mark.parametrize("seed", range(6))
def test_random_linear_layers_every_path(seed):
    rng = np.random.default_rng(1000 + seed)
    for it in range(10):
        k = int(rng.choice([1, 2, 3, 4, 8, 16]))
        r = int(rng.choice([1, 5, 8, 16, 24, 100, 128, 136, 256, 300]))
        n = int(rng.choice([8, 32, 40, 64, 96, 200, 256, 520, 1024, 2048]))
        T = int(rng.choice([1, 2, 7, 8, 9, 16, 17, 31, 33, 64, 100, 224, 225, 257, 600]))
        m = r * k
        act = int(rng.choice([B.ACT_NONE, B.ACT_RELU, B.ACT_GELU]))
        use_bias, y32, per_tile = bool(rng.integers(2)), bool(rng.integers(2)), bool(rng.integers(2))
        x32 = bool(rng.integers(4) == 0)
        x = synth.normal(seed * 100 + it, 0, T * n).reshape(T, n)
        x_in = x if x32 else synth.to_bf16_bits(x)
        x_val = x if x32 else synth.bf16_bits_to_f32(x_in)
        W = synth.normal(seed * 100 + it, 1, m * n, n ** -0.5)
        words, al = O.prepare(W, k, per_tile)
        bias = synth.normal(seed * 100 + it, 2, m, 0.2) if use_bias else None
        ref = O.linear(x_val, words, k, al, per_tile, m, n, bias=None if bias is None else bias.astype(np.float64), act=act)
        ran = 0
        for path in PATHS:
            try:
                y = B.tbn_linear_fwd(to_dev(x_in), m, to_dev(words), k, to_dev(al), int(per_tile),
                                     bias=None if bias is None else to_dev(bias), act=act,
                                     y_dtype=B.F32 if y32 else None, path=path)
            except B.TbnError as e:
                assert e.status == -3                   # this family does not take the shape
                continue
            torch.cuda.synchronize()
            ran += 1
            assert_close(to_np64(y), ref, f"T={T} m={m} n={n} k={k} act={act} bias={use_bias} y32={y32} x32={x32} path={path}")
        assert ran >= 2                                 # AUTO and the index-walk kernel take everything
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("seed", range(3))
def test_random_convolutions_every_path(seed):
    rng = np.random.default_rng(2000 + seed)
    for it in range(8):
        Cin = int(rng.choice([16, 32, 48, 64]))
        Cout = int(rng.choice([16, 32, 64, 128, 200]))
        k = int(rng.choice([1, 2, 4]))
        H, Wd = int(rng.integers(4, 24)), int(rng.choice([4, 8, 9, 15, 16, 17, 24, 32]))
        stride, pad = int(rng.choice([1, 2])), int(rng.choice([0, 1, 2]))
        Nb = int(rng.integers(1, 6))
        act = int(rng.choice([B.ACT_NONE, B.ACT_RELU, B.ACT_GELU]))
        use_bias = bool(rng.integers(2))
        x, Wt = synth.conv_layer(300 + seed * 10 + it, Nb, Cin, H, Wd, Cout, 3, 3)
        words, al = O.prepare(Wt, k, True)
        bias = synth.normal(seed * 10 + it, 3, Cout, 0.2) if use_bias else None
        ref = O.conv2d(x, words, k, al, True, Cout, Cin, 3, 3, stride, pad,
                       bias=None if bias is None else bias.astype(np.float64), act=act)
        for path in (B.PATH_AUTO, B.PATH_TENSOR, B.PATH_GENERIC):
            try:
                y = B.tbn_conv2d_fwd(to_dev(x), Cout, 3, 3, stride, pad, to_dev(words), k, to_dev(al), 1,
                                     bias=None if bias is None else to_dev(bias), act=act, path=path)
            except B.TbnError as e:
                assert e.status == -3
                continue
            torch.cuda.synchronize()
            assert_close(to_np64(y), ref, f"conv {Cin}->{Cout} k={k} {H}x{Wd} s{stride} p{pad} Nb={Nb} act={act} path={path}")
    assert B.tbn_last_device_status() == (0, 0)
