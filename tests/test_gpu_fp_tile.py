"""GPU parity, full-precision tiled weights (Sec. 5.2): the layer whose weight is a real-valued tile repeated k
times, against the CPU oracle on the same seeded inputs, within max|err| <= 1e-2 * (1 + |ref|)."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu


def case(seed, T, m, n, k, x_bf16=True, sigma=None):
    # tile values ~ N(0, 1/n): outputs of unit scale, as with the fan-in scaled initialisation the paper trains with.
    # The tensor-core kernel rounds an fp32 tile to bf16 (relative weight error 2^-9); with unit-scale outputs that
    # adds about 2^-9 / sqrt(3) = 1e-3 rms to the output error, inside the layer tolerance.
    q = m * n // k
    t = synth.normal(seed, 1, q, sigma if sigma is not None else n ** -0.5)
    x = synth.normal(seed, 0, T * n).reshape(T, n)
    if x_bf16:
        x = synth.to_bf16_bits(x)
    return x, t


def x_values(x):
    return synth.bf16_bits_to_f32(x) if x.dtype == np.uint16 else x


# (m, n, k): tiles spanning whole rows, tiles that do not, nothing aligned
SHAPES = [(512, 512, 4), (2304, 768, 8), (128, 784, 4), (96, 40, 6), (7, 33, 3), (10, 128, 1), (1024, 4096, 2)]


@pytest.mark.parametrize("m,n,k", SHAPES)
@pytest.mark.parametrize("T", [1, 17, 129])
def test_generic_path_is_exact_in_the_tile(m, n, k, T):
    x, t = case(40 + T, T, m, n, k)
    ref = O.linear_fp(x_values(x), t, k, m, n, act=O.ACT_RELU)
    got = B.tbn_linear_fp_tile_fwd(to_dev(x), m, to_dev(t), k, act=B.ACT_RELU, path=B.PATH_GENERIC, y_dtype=B.F32)
    torch.cuda.synchronize()
    assert np.allclose(to_np64(got), ref, rtol=2e-5, atol=2e-5)          # fp32 tile, fp32 accumulate: no bf16 anywhere


@pytest.mark.parametrize("m,n,k", [s for s in SHAPES if (s[0] * s[1] // s[2]) % s[1] == 0 and s[1] % 8 == 0])
@pytest.mark.parametrize("T", [1, 17, 129, 700])
@pytest.mark.parametrize("tile_bf16", [False, True])
def test_tensor_path_matches_oracle(m, n, k, T, tile_bf16):
    x, t = case(50 + T, T, m, n, k)
    if tile_bf16:
        tb = synth.to_bf16_bits(t)
        t_dev, t_ref = to_dev(tb), synth.bf16_bits_to_f32(tb)
    else:
        t_dev, t_ref = to_dev(t), t
    bias = synth.normal(50, 200, m, 0.1)
    ref = O.linear_fp(x_values(x), t_ref, k, m, n, bias=bias.astype(np.float64), act=O.ACT_GELU)
    assert B.tbn_linear_fp_tile_workspace_bytes(T, n, m, k, B.BF16, B.BF16 if tile_bf16 else B.F32) >= (0 if tile_bf16 else 2 * m * n // k)
    got = B.tbn_linear_fp_tile_fwd(to_dev(x), m, t_dev, k, bias=to_dev(bias), act=B.ACT_GELU, path=B.PATH_TENSOR)
    torch.cuda.synchronize()
    assert_close(to_np64(got), ref, f"fp tile tensor {m}x{n} k={k} T={T}")
    auto = B.tbn_linear_fp_tile_fwd(to_dev(x), m, t_dev, k, bias=to_dev(bias), act=B.ACT_GELU)
    assert torch.equal(auto, got)                                         # AUTO resolves to the tensor-core kernel here
    assert B.tbn_last_device_status() == (0, 0)


def test_rows_repeat_exactly_and_fp32_activations():
    # a tile spanning whole rows: output feature i + r is a copy of feature i (no scaling factor in between)
    T, m, n, k = 64, 512, 512, 4
    x, t = case(60, T, m, n, k, x_bf16=False)
    got = B.tbn_linear_fp_tile_fwd(to_dev(x), m, to_dev(t), k, y_dtype=B.F32)
    torch.cuda.synchronize()
    r = m // k
    for j in range(1, k):
        assert torch.equal(got[:, :r], got[:, j * r:(j + 1) * r])
    assert_close(to_np64(got), O.linear_fp(x, t, k, m, n), "fp tile fp32 x")


def test_misaligned_tile_auto_falls_back_and_errors():
    T, m, n, k = 5, 7, 33, 3
    x, t = case(61, T, m, n, k)
    got = B.tbn_linear_fp_tile_fwd(to_dev(x), m, to_dev(t), k)            # AUTO -> index-walk kernel
    assert_close(to_np64(got), O.linear_fp(x_values(x), t, k, m, n), "fp tile misaligned")
    with pytest.raises(B.TbnError):
        B.tbn_linear_fp_tile_fwd(to_dev(x), m, to_dev(t), k, path=B.PATH_TENSOR)
    with pytest.raises(B.TbnError):
        B.tbn_linear_fp_tile_fwd(to_dev(x), m, to_dev(t), k, path=B.PATH_SMALL)
    with pytest.raises(B.TbnError):
        B.tbn_linear_fp_tile_fwd(to_dev(x), 8, to_dev(t), 5)              # k does not divide the weight count
    empty = B.tbn_linear_fp_tile_fwd(torch.empty((0, n), dtype=torch.bfloat16, device=DEV), m, to_dev(t), k)
    assert empty.shape == (0, m)


def test_vit_shaped_layer_full_size_sampled_rows():
    # the paper measures this kernel on an ImageNet ViT (Table 7, "FP, Tiled_4"): fc1-shaped layer, k = 4, 128 x 197 tokens
    T, n, m, k = 128 * 197, 768, 3072, 4
    x, t = case(62, T, m, n, k, sigma=0.02)
    got = B.tbn_linear_fp_tile_fwd(to_dev(x), m, to_dev(t), k, act=B.ACT_GELU)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(5).choice(T, 16, replace=False))
    rows[-1] = T - 1
    ref = O.linear_fp(x_values(x)[rows], t, k, m, n, act=O.ACT_GELU)
    assert_close(to_np64(got)[rows], ref, "fp tile vit fc1")
    assert B.tbn_last_device_status() == (0, 0)
