"""GPU parity of compact chaining through an activation (first layer writes only its distinct pre-activations, the
second rebuilds act(alpha_j z) on chip) against the CPU oracle's plain two-layer composition."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu


def chain(T, d_in, hidden, kz, out_f, k, act_z, act=B.ACT_NONE, with_bias=False, y_dtype=B.BF16, seed=110, per_tile_z=True):
    x = synth.to_bf16_bits(synth.normal(seed, 0, T * d_in).reshape(T, d_in))
    W1 = synth.normal(seed, 1, hidden * d_in, d_in ** -0.5)
    W2 = synth.normal(seed, 2, out_f * hidden, hidden ** -0.5)
    w1, a1 = O.prepare(W1, kz, per_tile_z)
    w2, a2 = O.prepare(W2, k, True)
    bias = synth.normal(seed, 200, out_f, 0.2) if with_bias else None
    h = O.linear(x, w1, kz, a1, per_tile_z, hidden, d_in, act=act_z)
    ref = O.linear(h, w2, k, a2, True, out_f, hidden, bias=None if bias is None else bias.astype(np.float64), act=act)
    # first layer in compact form: the same tile as a k = 1 layer of r_z outputs with alpha 1
    rz = hidden // kz
    one = torch.ones(1, device=DEV)
    z = B.tbn_linear_fwd(to_dev(x), rz, to_dev(w1), 1, one, B.ALPHA_PER_LAYER)
    y = B.tbn_linear_compact_fwd(z, kz, to_dev(a1), int(per_tile_z), act_z, out_f, to_dev(w2), k, to_dev(a2), 1,
                                 bias=None if bias is None else to_dev(bias), act=act, y_dtype=y_dtype)
    torch.cuda.synchronize()
    return to_np64(y), ref


@pytest.mark.parametrize("T,d_in,hidden,kz,out_f,k", [(300, 128, 512, 8, 96, 4), (129, 64, 256, 2, 200, 8), (1, 64, 128, 2, 8, 1),
                                                      (777, 256, 1536, 4, 768, 8), (64, 96, 320, 5, 40, 2)])
@pytest.mark.parametrize("act_z", [B.ACT_GELU, B.ACT_RELU, B.ACT_NONE])
def test_compact_chain_matches_two_layer_oracle(T, d_in, hidden, kz, out_f, k, act_z):
    got, ref = chain(T, d_in, hidden, kz, out_f, k, act_z)
    assert_close(got, ref, f"compact chain act {act_z}")
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("act,with_bias,y_dtype,per_tile_z", [(B.ACT_RELU, False, B.BF16, False), (B.ACT_GELU, True, B.BF16, True),
                                                               (B.ACT_NONE, True, B.F32, True), (B.ACT_RELU, True, B.F32, False)])
def test_compact_chain_epilogue_variants(act, with_bias, y_dtype, per_tile_z):
    got, ref = chain(260, 128, 768, 4, 264, 4, B.ACT_GELU, act=act, with_bias=with_bias, y_dtype=y_dtype, per_tile_z=per_tile_z)
    assert_close(got, ref, "compact chain epilogue")


def test_vit_mlp_shape_sampled_rows_and_rejections():
    # ViT-B MLP: 768 -> 3072 (k = 8, GELU) -> 768 (k = 8), T = 25,216; sampled rows through the oracle
    T, d, mlp, k = 128 * 197, 768, 3072, 8
    x = synth.to_bf16_bits(synth.normal(3, 0, T * d).reshape(T, d))
    w1, a1 = O.prepare(synth.normal(3, 3, mlp * d, 0.02), k, True)
    w2, a2 = O.prepare(synth.normal(3, 4, d * mlp, 0.02), k, True)
    z = B.tbn_linear_fwd(to_dev(x), mlp // k, to_dev(w1), 1, torch.ones(1, device=DEV), B.ALPHA_PER_LAYER)
    y = B.tbn_linear_compact_fwd(z, k, to_dev(a1), 1, B.ACT_GELU, d, to_dev(w2), k, to_dev(a2), 1)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(5).choice(T, 24, replace=False)); rows[-1] = T - 1
    h = O.linear(x[rows], w1, k, a1, True, mlp, d, act=O.ACT_GELU)
    ref = O.linear(h, w2, k, a2, True, d, mlp)
    assert_close(to_np64(y)[rows], ref, "ViT MLP compact")
    zz = torch.zeros((4, 96), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(B.TbnError) as e:                                  # r_z = 96 is not a multiple of 64
        B.tbn_linear_compact_fwd(zz, 2, to_dev(a1), 1, B.ACT_GELU, 8, to_dev(w2), 1, to_dev(a2), 1)
    assert e.value.status == -3
