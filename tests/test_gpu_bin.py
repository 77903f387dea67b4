"""GPU parity of the binary-activation layer (sign activations with a per-row scale, XNOR / popcount contraction)
against the CPU oracle: the activation bits and the integer accumulators bit for bit, the row scales to 1e-6, the
scaled outputs within the layer tolerance.  Both kernel families: the popcount kernel (any shape) and the 8-bit
integer tensor-core kernel (tiles that span whole rows)."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,n", [(1, 8), (3, 33), (5, 127), (7, 128), (9, 129), (16, 768), (37, 1000), (300, 8192)])
@pytest.mark.parametrize("bf16", [True, False])
def test_binarize_bits_exact_and_beta(T, n, bf16):
    x = synth.normal(50 + n, 0, T * n).reshape(T, n)
    x[0, : min(n, 4)] = [0.0, -0.0, 1e-30, -1.0][: min(n, 4)]
    xin = synth.to_bf16_bits(x) if bf16 else x
    bits_ref, beta_ref = O.binarize(xin)
    xb, beta = B.tbn_binarize_fwd(to_dev(xin))
    torch.cuda.synchronize()
    assert xb.shape == (T, O.row_words(n))
    assert np.array_equal(xb.cpu().numpy().view(np.uint32), O.pack_rows(bits_ref))     # padding bits are zero too
    assert np.allclose(beta.cpu().numpy(), beta_ref, rtol=1e-6, atol=0)
    xb2, none = B.tbn_binarize_fwd(to_dev(xin), with_beta=False)
    assert none is None and torch.equal(xb, xb2)


def _case(seed, T, m, n, k, per_tile, sigma=None):
    x = synth.to_bf16_bits(synth.normal(seed, 0, T * n).reshape(T, n))
    W = synth.normal(seed, 1, m * n, sigma if sigma else n ** -0.5)
    words, al = O.prepare(W, k, per_tile)
    abits, beta = O.binarize(x)
    return x, words, al, abits, beta


# (T, m, n, k): the oracle's shape zoo -- aligned tiles, several tiles per row, tiles that end inside a row, nothing divides
ZOO = [(1, 8, 8, 1), (2, 8, 8, 2), (3, 8, 8, 8), (17, 128, 784, 4), (64, 10, 128, 1), (129, 512, 512, 4),
       (5, 96, 40, 6), (3, 6, 64, 4), (2, 4, 64, 8), (3, 7, 33, 3), (9, 2304, 768, 8), (4, 16, 8, 128)]


@pytest.mark.parametrize("T,m,n,k", ZOO)
@pytest.mark.parametrize("per_tile", [False, True])
def test_popcount_kernel_integers_exact_and_outputs_close(T, m, n, k, per_tile):
    x, words, al, abits, beta = _case(60, T, m, n, k, per_tile)
    xb = to_dev(O.pack_rows(abits))
    D = B.tbn_linear_bin_fwd(xb, n, m, to_dev(words), k, to_dev(al), int(per_tile), y_dtype=B.I32, path=B.PATH_GENERIC)
    torch.cuda.synchronize()
    assert np.array_equal(D.cpu().numpy().astype(np.int64), O.linear_bin_int(abits, words, k, m, n))
    bias = synth.normal(60, 200, m, 0.1)
    ref = O.linear_bin(abits, beta, words, k, al, per_tile, m, n, bias=bias.astype(np.float64), act=O.ACT_RELU)
    y = B.tbn_linear_bin_fwd(xb, n, m, to_dev(words), k, to_dev(al), int(per_tile), beta=to_dev(beta), bias=to_dev(bias),
                             act=B.ACT_RELU, y_dtype=B.F32, path=B.PATH_GENERIC)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "popcount kernel")


# shapes the tensor-core kernel takes: ragged token tails, ragged row blocks, rows shorter / longer than a stage
TENSOR = [(1, 128, 32, 1), (33, 256, 256, 2), (129, 512, 512, 4), (300, 2304, 768, 8), (777, 1200, 992, 4),
          (260, 64, 4096, 2), (50, 8, 64, 1), (513, 3072, 768, 16)]


@pytest.mark.parametrize("T,m,n,k", TENSOR)
def test_tensor_kernel_integers_exact_every_tile_shape(T, m, n, k):
    x, words, al, abits, beta = _case(61, T, m, n, k, True)
    xb, td, ad = to_dev(O.pack_rows(abits)), to_dev(words), to_dev(al)
    want = O.linear_bin_int(abits, words, k, m, n)
    cand = 0
    try:
        while B.lib().tbn_debug_force_bin_config(cand) == 0:
            D = B.tbn_linear_bin_fwd(xb, n, m, td, k, ad, 1, y_dtype=B.I32, path=B.PATH_TENSOR)
            torch.cuda.synchronize()
            assert np.array_equal(D.cpu().numpy().astype(np.int64), want), f"tile shape {cand}"
            cand += 1
    finally:
        B.lib().tbn_debug_force_bin_config(-1)
    assert cand >= 2
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("T,m,n,k", [(300, 2304, 768, 8), (777, 1200, 992, 4), (64, 512, 512, 4)])
@pytest.mark.parametrize("act,y_dtype,with_bias", [(B.ACT_NONE, B.BF16, False), (B.ACT_RELU, B.BF16, False),
                                                   (B.ACT_GELU, B.BF16, True), (B.ACT_RELU, B.F32, True),
                                                   (B.ACT_NONE, B.F32, False)])
def test_tensor_kernel_scaled_outputs_and_agreement_with_popcount_kernel(T, m, n, k, act, y_dtype, with_bias):
    x, words, al, abits, beta = _case(62, T, m, n, k, True)
    xb, td, ad = to_dev(O.pack_rows(abits)), to_dev(words), to_dev(al)
    bias = synth.normal(62, 200, m, 0.2) if with_bias else None
    ref = O.linear_bin(abits, beta, words, k, al, True, m, n, bias=None if bias is None else bias.astype(np.float64),
                       act=act)
    kw = dict(beta=to_dev(beta), bias=None if bias is None else to_dev(bias), act=act, y_dtype=y_dtype)
    yt = B.tbn_linear_bin_fwd(xb, n, m, td, k, ad, 1, path=B.PATH_TENSOR, **kw)
    yg = B.tbn_linear_bin_fwd(xb, n, m, td, k, ad, 1, path=B.PATH_GENERIC, **kw)
    torch.cuda.synchronize()
    assert_close(to_np64(yt), ref, "tensor kernel")
    assert_close(to_np64(yg), ref, "popcount kernel")
    assert B.tbn_last_device_status() == (0, 0)


def test_binarize_then_layer_end_to_end_and_single_alpha_no_beta():
    # the two calls chained on the device; per-layer alpha, no beta: y = alpha * D
    T, m, n, k = 200, 768, 768, 8
    x, words, al, abits, beta = _case(63, T, m, n, k, False)
    xb, bt = B.tbn_binarize_fwd(to_dev(x))
    y = B.tbn_linear_bin_fwd(xb, n, m, to_dev(words), k, to_dev(al), 0, y_dtype=B.F32)
    torch.cuda.synchronize()
    ref = O.linear_bin(abits, None, words, k, al, False, m, n)
    assert_close(to_np64(y), ref, "no beta")
    assert np.array_equal(to_np64(y), (float(al[0]) * O.linear_bin_int(abits, words, k, m, n)).astype(np.float32).astype(np.float64))


def test_large_sweep_shape_sampled_rows_integers_exact():
    # the large linear sweep's shape with binary activations: 8192 x 8192, T = 4096, k in {2, 16}; sampled rows
    T, m, n = 4096, 8192, 8192
    x = synth.to_bf16_bits(synth.normal(4, 0, T * n).reshape(T, n))
    W = synth.normal(4, 1, m * n, 0.02)
    xb, bt = B.tbn_binarize_fwd(to_dev(x))
    rows = np.unique(np.concatenate([np.arange(0, T, 128) + np.arange(T // 128) % 128, [0, T - 1]]))
    abits, beta = O.binarize(x[rows])
    assert np.array_equal(xb[torch.from_numpy(rows).to(DEV)].cpu().numpy().view(np.uint32), O.pack_rows(abits))
    for k in (2, 16):
        words, al = O.prepare(W, k, True)
        D = B.tbn_linear_bin_fwd(xb, n, m, to_dev(words), k, to_dev(al), 1, y_dtype=B.I32)
        torch.cuda.synchronize()
        assert np.array_equal(D[torch.from_numpy(rows).to(DEV)].cpu().numpy().astype(np.int64),
                              O.linear_bin_int(abits, words, k, m, n))
        y = B.tbn_linear_bin_fwd(xb, n, m, to_dev(words), k, to_dev(al), 1, beta=bt, act=B.ACT_RELU, y_dtype=B.BF16)
        torch.cuda.synchronize()
        ref = O.linear_bin(abits, beta, words, k, al, True, m, n, act=O.ACT_RELU)
        assert_close(to_np64(y[torch.from_numpy(rows).to(DEV)]), ref, f"sweep shape k={k}")
    assert B.tbn_last_device_status() == (0, 0)


def expand_reference(bits_rows: np.ndarray, n: int) -> np.ndarray:
    """The documented byte form written out element by element: byte 4 s + j of each group of 32 elements is 0xFF when
    element 8 j + 7 - s of the group is +1, else 0x00."""
    T = bits_rows.shape[0]
    out = np.zeros((T, n), dtype=np.uint8)
    for g in range(n // 32):
        for sft in range(8):
            for j in range(4):
                out[:, 32 * g + 4 * sft + j] = np.where(bits_rows[:, 32 * g + 8 * j + 7 - sft] != 0, 0xFF, 0x00)
    return out


@pytest.mark.parametrize("T,n", [(1, 32), (5, 96), (130, 768), (33, 4096)])
def test_expand_to_bytes_matches_the_documented_order(T, n):
    x = synth.to_bf16_bits(synth.normal(70 + n, 0, T * n).reshape(T, n))
    abits, _ = O.binarize(x)
    xb = to_dev(O.pack_rows(abits))
    got, pop = B.tbn_bin_expand_fwd(xb, n)
    torch.cuda.synchronize()
    assert got.shape == (T, n) and got.dtype == torch.uint8
    assert np.array_equal(got.cpu().numpy(), expand_reference(np.asarray(abits), n))
    assert np.array_equal(pop.cpu().numpy(), np.asarray(abits, dtype=np.int64).sum(axis=1))
    with pytest.raises(B.TbnError) as e:
        B.tbn_bin_expand_fwd(torch.zeros((2, 4), dtype=torch.int32, device=DEV), 40)      # not a multiple of 32
    assert e.value.status == -3


@pytest.mark.parametrize("T,n,bf16", [(3, 32, True), (70, 992, True), (130, 768, False), (33, 8192, True)])
def test_one_pass_binarize_with_bytes_equals_the_two_passes(T, n, bf16):
    x = synth.normal(80 + n, 0, T * n).reshape(T, n)
    x[0, :4] = [0.0, -0.0, 1e-30, -1.0]
    xin = to_dev(synth.to_bf16_bits(x) if bf16 else x)
    xb, beta = B.tbn_binarize_fwd(xin)
    xbytes, xpop = B.tbn_bin_expand_fwd(xb, n)
    xb1, beta1, xbytes1, xpop1 = B.tbn_binarize_bytes_fwd(xin)
    torch.cuda.synchronize()
    assert torch.equal(xb, xb1) and torch.equal(beta, beta1) and torch.equal(xbytes, xbytes1) and torch.equal(xpop, xpop1)


@pytest.mark.parametrize("T,m,n,k", TENSOR)
def test_byte_form_integers_exact_every_tile_shape(T, m, n, k):
    x, words, al, abits, beta = _case(64, T, m, n, k, True)
    xb, td, ad = to_dev(O.pack_rows(abits)), to_dev(words), to_dev(al)
    xbytes, xpop = B.tbn_bin_expand_fwd(xb, n)
    want = O.linear_bin_int(abits, words, k, m, n)
    cand = 0
    try:
        while B.lib().tbn_debug_force_bin_config(cand) == 0:
            D = B.tbn_linear_bin_bytes_fwd(xbytes, xpop, n, m, td, k, ad, 1, y_dtype=B.I32)
            torch.cuda.synchronize()
            assert np.array_equal(D.cpu().numpy().astype(np.int64), want), f"tile shape {cand}"
            cand += 1
    finally:
        B.lib().tbn_debug_force_bin_config(-1)
    assert cand >= 2
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("act,y_dtype,with_bias", [(B.ACT_RELU, B.BF16, False), (B.ACT_GELU, B.BF16, True), (B.ACT_NONE, B.F32, True)])
def test_byte_form_scaled_outputs(act, y_dtype, with_bias):
    T, m, n, k = 777, 1200, 992, 4
    x, words, al, abits, beta = _case(65, T, m, n, k, True)
    xb, td, ad = to_dev(O.pack_rows(abits)), to_dev(words), to_dev(al)
    bias = synth.normal(65, 200, m, 0.2) if with_bias else None
    ref = O.linear_bin(abits, beta, words, k, al, True, m, n, bias=None if bias is None else bias.astype(np.float64), act=act)
    y = B.tbn_linear_bin_bytes_fwd(*B.tbn_bin_expand_fwd(xb, n), n, m, td, k, ad, 1, beta=to_dev(beta),
                                   bias=None if bias is None else to_dev(bias), act=act, y_dtype=y_dtype)
    torch.cuda.synchronize()
    assert_close(to_np64(y), ref, "byte form")
    assert B.tbn_last_device_status() == (0, 0)


def test_byte_form_large_sweep_shape_sampled_rows_integers_exact():
    T, m, n = 4096, 8192, 8192
    x = synth.to_bf16_bits(synth.normal(4, 0, T * n).reshape(T, n))
    W = synth.normal(4, 1, m * n, 0.02)
    xb, bt = B.tbn_binarize_fwd(to_dev(x))
    xbytes, xpop = B.tbn_bin_expand_fwd(xb, n)
    rows = np.unique(np.concatenate([np.arange(0, T, 128) + np.arange(T // 128) % 128, [0, T - 1]]))
    abits, beta = O.binarize(x[rows])
    for k in (2, 16):
        words, al = O.prepare(W, k, True)
        D = B.tbn_linear_bin_bytes_fwd(xbytes, xpop, n, m, to_dev(words), k, to_dev(al), 1, y_dtype=B.I32)
        torch.cuda.synchronize()
        assert np.array_equal(D[torch.from_numpy(rows).to(DEV)].cpu().numpy().astype(np.int64),
                              O.linear_bin_int(abits, words, k, m, n))
    assert B.tbn_last_device_status() == (0, 0)


def test_argument_errors():
    xb = torch.zeros((4, 4), dtype=torch.int32, device=DEV)
    t = torch.zeros(8, dtype=torch.int32, device=DEV)
    a = torch.ones(4, device=DEV)
    with pytest.raises(B.TbnError) as e:
        B.tbn_linear_bin_fwd(xb, 64, 64, t, 3, a, 1)                       # 3 does not divide 4096
    assert e.value.status == -2
    with pytest.raises(B.TbnError) as e:
        B.tbn_linear_bin_fwd(xb, 40, 96, t, 6, a, 1, path=B.PATH_TENSOR)   # rows of 40 bits: not word aligned
    assert e.value.status == -3
    with pytest.raises(B.TbnError) as e:
        B.tbn_linear_bin_fwd(xb, 64, 64, t, 4, a, 1, path=B.PATH_SMALL)
    assert e.value.status == -3
