"""GPU parity of the training-side tiling module: forward (tile bits and B_hat bit-exact, alpha to 1e-6) and the
straight-through backward (the pure pass-through part bit-exact, the alpha path to 1e-6) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, to_dev

pytestmark = pytest.mark.gpu

CASES = [(8, 1), (8, 2), (8, 8), (7 * 33, 3), (512 * 512, 4), (2304 * 768, 8), (1000 * 37, 5), (4097 * 6, 6), (300, 300),
         (2048 * 2048, 16)]


@pytest.mark.parametrize("N,k", CASES)
@pytest.mark.parametrize("per_tile", [False, True])
@pytest.mark.parametrize("with_A", [False, True])
def test_tile_fwd_and_bwd_match_oracle(N, k, per_tile, with_A):
    W = synth.normal(70, 1, N, 0.02)
    A = synth.normal(70, 101, N, 0.05) if with_A else None
    W[:3] = [0.0, -0.0, 1e-30][: min(3, N)]
    G = synth.normal(70, 300, N, 1.0)
    mode = B.ALPHA_PER_TILE if per_tile else B.ALPHA_PER_LAYER
    Bh_ref, words, al = O.tile_fwd(W, k, per_tile, A)
    Wd, Ad = to_dev(W), (to_dev(A) if with_A else None)
    Bh, tile, alpha = B.tbn_tile_fwd(Wd, k, mode, A=Ad)
    torch.cuda.synchronize()
    assert np.array_equal(tile.cpu().numpy().view(np.uint32), words)
    assert np.allclose(alpha.cpu().numpy(), al, rtol=1e-6, atol=0)
    # B_hat is +-alpha_j: exact given the kernel's own alpha
    t = np.where(O.aggregate(W, k)[0] > 0, 1.0, -1.0).astype(np.float32)
    a_dev = alpha.cpu().numpy()
    want = (np.repeat(a_dev, N // k) if per_tile else a_dev[0]) * np.tile(t, k)
    assert np.array_equal(Bh.cpu().numpy(), want.astype(np.float32))
    assert np.allclose(Bh.cpu().numpy(), Bh_ref, rtol=1e-6, atol=0)
    Bh16, _, _ = B.tbn_tile_fwd(Wd, k, mode, A=Ad, b_dtype=B.BF16)
    assert torch.equal(Bh16, Bh.to(torch.bfloat16))

    # backward with the oracle's tile and alpha as inputs (so the comparison isolates the backward)
    dW_ref, dA_ref, dal_ref = O.tile_bwd(G, words, al, per_tile, W, k, A)
    dW, dA, dalpha = B.tbn_tile_bwd(to_dev(G), to_dev(words), to_dev(al), Wd, k, mode, A=Ad)
    torch.cuda.synchronize()
    scale = max(1.0, float(np.abs(dal_ref).max()))
    assert np.allclose(dalpha.cpu().numpy(), dal_ref, rtol=1e-6, atol=1e-6 * scale)
    if with_A:
        # the straight-through part is one fp32 multiply: bit-exact
        assert np.array_equal(dW.cpu().numpy(), dW_ref.astype(np.float32))
        assert np.allclose(dA.cpu().numpy(), dA_ref, rtol=2e-6, atol=1e-6 * scale / (N // k if per_tile else N))
    else:
        assert dA is None
        assert np.allclose(dW.cpu().numpy(), dW_ref, rtol=2e-6, atol=1e-6 * (float(np.abs(dW_ref).max()) + 1e-30))


def test_backward_is_reproducible_and_checks_arguments():
    N, k = 768 * 768, 8
    W, G = to_dev(synth.normal(71, 1, N, 0.02)), to_dev(synth.normal(71, 300, N))
    _, tile, alpha = B.tbn_tile_fwd(W, k)
    r1 = B.tbn_tile_bwd(G, tile, alpha, W, k)
    r2 = B.tbn_tile_bwd(G, tile, alpha, W, k)
    torch.cuda.synchronize()
    assert torch.equal(r1[0], r2[0]) and torch.equal(r1[2], r2[2])
    lib = B.lib()
    p = W.data_ptr()
    assert lib.tbn_tile_bwd(p, p, p, p, None, N, 7, 1, p, None, None, p, 1 << 30, None) == -2      # 7 does not divide N
    assert lib.tbn_tile_bwd(p, p, p, p, p, N, 8, 1, p, None, None, p, 1 << 30, None) == -1         # A without dA
    assert lib.tbn_tile_bwd(p, p, p, p, None, N, 8, 1, p, None, None, p, 16, None) == -4           # workspace too small
