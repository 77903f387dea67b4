"""CPU pins of the identity behind compact chaining (Sec. 4.1): with a tile that spans whole rows, output channel
j * r + c of a tiled layer is alpha_j times the pre-activation of distinct row c, so a layer's k-fold output is a function of
its r distinct pre-activations alone.  The GPU entry point that consumes the compact form is tested against the two-layer
oracle; these tests pin, on the oracle itself, that the compact form carries the same information."""
import numpy as np
import pytest

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import synth


@pytest.mark.parametrize("T,n,m,k,per_tile", [(5, 32, 64, 4, True), (3, 48, 96, 8, True), (4, 16, 40, 5, False), (2, 64, 64, 1, True)])
@pytest.mark.parametrize("act", [O.ACT_NONE, O.ACT_RELU, O.ACT_GELU])
def test_full_output_is_act_of_alpha_times_the_distinct_pre_activations(T, n, m, k, per_tile, act):
    x = synth.normal(120, 0, T * n).reshape(T, n)
    W = synth.normal(120, 1, m * n, n ** -0.5)
    words, al = O.prepare(W, k, per_tile)
    r = m // k
    full = O.linear(x, words, k, al, per_tile, m, n, act=act)
    # the same tile read as a k = 1 layer of r outputs with a scaling factor of one: the distinct pre-activations
    z = O.linear(x, words, 1, np.ones(1, dtype=np.float32), False, r, n)
    assert z.shape == (T, r)
    alphas = np.asarray(al, dtype=np.float64) if per_tile else np.full(k, float(al[0]))
    rebuilt = np.concatenate([alphas[j] * z for j in range(k)], axis=1)
    if act == O.ACT_RELU:
        rebuilt = np.maximum(rebuilt, 0.0)
    elif act == O.ACT_GELU:
        from math import erf, sqrt
        rebuilt = np.vectorize(lambda v: 0.5 * v * (1.0 + erf(v / sqrt(2.0))))(rebuilt)
    assert np.allclose(full, rebuilt, rtol=1e-12, atol=1e-12)


def test_identity_fails_when_the_tile_does_not_span_whole_rows():
    # q = 24 bits against rows of 16 inputs: output channels are no longer scaled copies of r distinct rows
    T, n, m, k = 3, 16, 6, 4
    x = synth.normal(121, 0, T * n).reshape(T, n)
    W = synth.normal(121, 1, m * n, 0.25)
    words, al = O.prepare(W, k, True)
    full = O.linear(x, words, k, al, True, m, n)
    ratios = full[:, 1:] / full[:, :1]
    assert not np.allclose(ratios, ratios[0:1, :])        # columns are not multiples of one another token by token
