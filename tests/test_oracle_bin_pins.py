"""Pins for the binary-activation part of the CPU oracle (Sec. 7: binary weights and binary activations; the
reading of the activation rule is listed in the design notes).  Each check compares the oracle with something
other than itself: numpy on +-1 matrices, the XNOR / popcount identity evaluated with Python integers, closed
forms and brute force.  Runs without a GPU."""
import itertools

import numpy as np
import pytest

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import synth


def bits_of(words, q):
    i = np.arange(q)
    return ((words[i >> 5] >> (i & 31).astype(np.uint32)) & 1).astype(np.uint8)


def expanded_pm1(words, m, n, p):
    """Eq. 4-5 with numpy: the unscaled +-1 weight matrix."""
    t = np.where(bits_of(words, m * n // p) > 0, 1, -1).astype(np.int64)
    return np.tile(t, p).reshape(m, n)


def test_binarize_is_the_threshold_rule_and_row_mean():
    x = synth.normal(3, 0, 7 * 45).reshape(7, 45)
    x[0, :5] = [0.0, -0.0, np.nan, 1e-30, -1e-30]
    bits, beta = O.binarize(x)
    assert bits[0, :5].tolist() == [0, 0, 0, 1, 0]                    # zero, negative zero and NaN are -1
    assert np.array_equal(bits[1:], (x[1:] > 0).astype(np.uint8))
    assert np.allclose(beta[1:], np.abs(x[1:].astype(np.float64)).mean(axis=1), rtol=1e-7)
    # bf16 inputs are taken at their exact values
    xb = synth.to_bf16_bits(x[1:])
    bits_b, beta_b = O.binarize(xb)
    xf = synth.bf16_bits_to_f32(xb)
    assert np.array_equal(bits_b, (xf > 0).astype(np.uint8))
    assert np.allclose(beta_b, np.abs(xf.astype(np.float64)).mean(axis=1), rtol=1e-7)


@pytest.mark.parametrize("n", [1, 31, 32, 33, 127, 128, 129, 300])
def test_pack_rows_matches_numpy_packbits_little(n):
    bits = (np.random.default_rng(n).random((5, n)) > 0.5).astype(np.uint8)
    rows = O.pack_rows(bits)
    assert rows.shape == (5, O.row_words(n)) and rows.shape[1] % 4 == 0
    for t in range(5):
        ref = np.packbits(bits[t], bitorder="little")
        got = rows[t].view(np.uint8)
        assert np.array_equal(got[:ref.size], ref)
        assert not got[ref.size:].any()                               # padding bits are zero


SHAPES = [  # (T, m, n, p)
    (3, 8, 8, 1), (3, 8, 8, 2), (2, 8, 8, 8), (5, 128, 784, 4), (4, 10, 128, 1), (2, 96, 40, 6),
    (3, 6, 64, 4), (3, 4, 64, 8), (4, 7, 33, 3),
]


@pytest.mark.parametrize("T,m,n,p", SHAPES)
def test_integer_accumulator_is_the_pm1_matrix_product_and_the_xnor_popcount_identity(T, m, n, p):
    rng = np.random.default_rng(m * 31 + n)
    W = rng.standard_normal(m * n).astype(np.float32)
    words, _ = O.prepare(W, p, True)
    x = rng.standard_normal((T, n)).astype(np.float32)
    abits, _ = O.binarize(x)
    D = O.linear_bin_int(abits, words, p, m, n)
    Bpm = expanded_pm1(words, m, n, p)
    a_pm = np.where(abits > 0, 1, -1).astype(np.int64)
    assert np.array_equal(D, a_pm @ Bpm.T)                            # numpy integer product on +-1 matrices
    # XNOR / popcount: a dot product of n +-1 values is 2 * popcount(xnor) - n = n - 2 * popcount(xor),
    # evaluated on rows packed into Python integers
    for t in range(T):
        xa = int.from_bytes(np.packbits(abits[t], bitorder="little").tobytes(), "little")
        for i in range(m):
            wb = int.from_bytes(np.packbits((Bpm[i] > 0).astype(np.uint8), bitorder="little").tobytes(), "little")
            assert D[t, i] == n - 2 * bin(xa ^ wb).count("1")


def test_p1_is_a_plain_xnor_layer():
    # p = 1: sign(W) against sign(x), scaled by mean|W| and mean|x_t| (the binary layer the paper's related work describes)
    rng = np.random.default_rng(5)
    m, n, T = 12, 40, 6
    W = rng.standard_normal((m, n)).astype(np.float32)
    x = rng.standard_normal((T, n)).astype(np.float32)
    words, al = O.prepare(W, 1, False)
    abits, beta = O.binarize(x)
    y = O.linear_bin(abits, beta, words, 1, al, False, m, n)
    ref = (np.sign(x).astype(np.float64) @ np.sign(W).astype(np.float64).T)
    ref = ref * np.abs(W.astype(np.float64)).mean() * np.abs(x.astype(np.float64)).mean(axis=1)[:, None]
    assert np.allclose(y, ref, rtol=1e-6, atol=1e-9)                  # alpha and beta are rounded to fp32


@pytest.mark.parametrize("T,m,n,p,per_tile", [(3, 16, 24, 4, True), (2, 12, 20, 2, False), (3, 6, 64, 4, True),
                                              (2, 7, 33, 3, True)])
def test_scaled_output_is_beta_times_alpha_weighted_segment_sums(T, m, n, p, per_tile):
    rng = np.random.default_rng(n)
    W = rng.standard_normal(m * n).astype(np.float32)
    words, al = O.prepare(W, p, per_tile)
    x = rng.standard_normal((T, n)).astype(np.float32)
    abits, beta = O.binarize(x)
    bias = rng.standard_normal(m)
    y = O.linear_bin(abits, beta, words, p, al, per_tile, m, n, bias=bias, act=O.ACT_RELU)
    # by hand: walk the flat weight index, alpha changes every q entries (Algorithm 1's walk) on +-1 activations
    q = m * n // p
    Bpm = expanded_pm1(words, m, n, p).reshape(-1).astype(np.float64)
    a_idx = (np.arange(m * n) // q) if per_tile else np.zeros(m * n, dtype=np.int64)
    Bhat = (Bpm * al.astype(np.float64)[a_idx]).reshape(m, n)
    a_pm = np.where(abits > 0, 1.0, -1.0)
    ref = np.maximum(beta.astype(np.float64)[:, None] * (a_pm @ Bhat.T) + bias[None, :], 0.0)
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    if q % n == 0:                                                    # whole rows per tile: y = beta_t alpha_j D
        D = O.linear_bin_int(abits, words, p, m, n)
        r = q // n
        aj = al.astype(np.float64)[(np.arange(m) // r) if per_tile else np.zeros(m, dtype=np.int64)]
        ref2 = np.maximum(beta.astype(np.float64)[:, None] * aj[None, :] * D + bias[None, :], 0.0)
        assert np.allclose(y, ref2, rtol=1e-12, atol=1e-12)


def test_brute_force_all_tiles_and_inputs_tiny():
    # m = 2, n = 3, p in {1, 2, 3, 6}: every tile and every sign pattern of one input row
    m, n = 2, 3
    for p in (1, 2, 3, 6):
        q = m * n // p
        for tile in itertools.product([0, 1], repeat=q):
            words = O.pack_bits(np.array(tile, dtype=np.uint8))
            for a in itertools.product([0, 1], repeat=n):
                D = O.linear_bin_int(np.array([a], dtype=np.uint8), words, p, m, n)
                for i in range(m):
                    want = sum((1 if tile[(i * n + j) % q] else -1) * (1 if a[j] else -1) for j in range(n))
                    assert D[0, i] == want


def test_all_ones_and_flips():
    # all-ones tile and all-positive input: D = n; flipping the input negates D; flipping one input bit changes D by 2
    m, n, p = 8, 64, 4
    words = O.pack_bits(np.ones(m * n // p, dtype=np.uint8))
    a = np.ones((1, n), dtype=np.uint8)
    assert np.array_equal(O.linear_bin_int(a, words, p, m, n), np.full((1, m), n))
    assert np.array_equal(O.linear_bin_int(1 - a, words, p, m, n), np.full((1, m), -n))
    a[0, 17] = 0
    assert np.array_equal(O.linear_bin_int(a, words, p, m, n), np.full((1, m), n - 2))
