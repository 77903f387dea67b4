"""Pins for the training-side tiling module of the CPU oracle (Sec. 3: Eq. 1-5 forward, straight-through backward,
scaling factors of Eq. 6-8 differentiated as ordinary functions).  Compared with torch autograd on an independently
written module, with finite differences where the function is differentiable, and with hand values."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O


def torch_module(W, A, p, per_tile):
    """The module written with torch ops: hard tile with a straight-through gradient, alpha by autograd."""
    N = W.numel()
    q = N // p
    s = W.reshape(p, q).sum(dim=0)
    t = torch.where(s > 0, 1.0, -1.0).to(W.dtype)
    B_hard = t.repeat(p)
    B = W + (B_hard - W).detach()                       # forward: B_hard; backward: identity to W
    S = W if A is None else A
    if per_tile:
        alpha = S.abs().reshape(p, q).mean(dim=1)
        return (alpha[:, None] * B.reshape(p, q)).reshape(-1)
    return S.abs().mean() * B


@pytest.mark.parametrize("N,p,per_tile,with_A", [(24, 4, True, True), (24, 4, True, False), (30, 3, False, True),
                                                 (30, 3, False, False), (64, 1, True, True), (16, 16, True, False)])
def test_forward_and_backward_match_torch_autograd(N, p, per_tile, with_A):
    rng = np.random.default_rng(N + p)
    W = rng.standard_normal(N).astype(np.float32)
    A = rng.standard_normal(N).astype(np.float32) if with_A else None
    G = rng.standard_normal(N)
    Bh, words, al = O.tile_fwd(W, p, per_tile, A)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    At = torch.tensor(A, dtype=torch.float64, requires_grad=True) if with_A else None
    out = torch_module(Wt, At, p, per_tile)
    assert np.allclose(Bh, out.detach().numpy(), rtol=1e-6, atol=0)           # alpha is rounded to fp32 in the oracle
    (out * torch.tensor(G)).sum().backward()
    dW, dA, dalpha = O.tile_bwd(G, words, al, per_tile, W, p, A)
    assert np.allclose(dW, Wt.grad.numpy(), rtol=1e-6, atol=1e-9)
    if with_A:
        assert np.allclose(dA, At.grad.numpy(), rtol=1e-6, atol=1e-9)
    else:
        assert dA is None


def test_alpha_path_matches_finite_differences():
    # L(A) = sum G * (alpha(A) (.) B) is differentiable in A (away from zeros): central differences in fp64
    rng = np.random.default_rng(9)
    N, p = 20, 4
    W = rng.standard_normal(N).astype(np.float32)
    A = (rng.standard_normal(N) + np.sign(rng.standard_normal(N)) * 0.5).astype(np.float32)
    G = rng.standard_normal(N)
    _, words, al = O.tile_fwd(W, p, True, A)
    _, dA, dalpha = O.tile_bwd(G, words, al, True, W, p, A)
    q = N // p
    t = np.where(O.aggregate(W, p)[0] > 0, 1.0, -1.0)
    B = np.tile(t, p)

    def loss(Av):
        a = np.abs(Av).reshape(p, q).mean(axis=1)
        return float(np.sum(G * np.repeat(a, q) * B))

    A64 = A.astype(np.float64)
    for f in range(N):
        e = np.zeros(N); e[f] = 1e-6
        fd = (loss(A64 + e) - loss(A64 - e)) / 2e-6
        assert abs(fd - dA[f]) <= 1e-6 * max(1.0, abs(fd))
    assert np.allclose(dalpha, (G * B).reshape(p, q).sum(axis=1), rtol=1e-12)


def test_hand_example_straight_through():
    # p = 2, q = 2, W = (1, -2, 3, -1): column sums (4, -3) -> tile (+1, -1); alpha_0 = 1.5, alpha_1 = 2 (from W)
    W = np.array([1, -2, 3, -1], dtype=np.float32)
    G = np.array([1.0, 10.0, 100.0, 1000.0])
    Bh, words, al = O.tile_fwd(W, 2, True)
    assert Bh.tolist() == [1.5, -1.5, 2.0, -2.0] and al.tolist() == [1.5, 2.0]
    dW, dA, dalpha = O.tile_bwd(G, words, al, True, W, 2)
    # dalpha = (1*1 + 10*(-1), 100*1 + 1000*(-1)) = (-9, -900); dL/dW = alpha*G + dalpha*sign(W)/2
    assert dalpha.tolist() == [-9.0, -900.0]
    assert dW.tolist() == [1.5 - 4.5, 15.0 + 4.5, 200.0 - 450.0, 2000.0 + 450.0]
    # with a separate A the straight-through part alone reaches W
    A = np.array([2, 2, -4, 0], dtype=np.float32)
    Bh, words, al = O.tile_fwd(W, 2, True, A)
    dW, dA, dalpha = O.tile_bwd(G, words, al, True, W, 2, A)
    assert al.tolist() == [2.0, 2.0] and dW.tolist() == [2.0, 20.0, 200.0, 2000.0]
    assert dA.tolist() == [-4.5, -4.5, 450.0, 0.0]                         # sign(0) = 0
