"""Shared helpers of the GPU parity tests: tolerance rule, host<->device shuttling."""
import numpy as np
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth

DEV = "cuda:0"


def to_dev(a: np.ndarray, bf16: bool = False) -> torch.Tensor:
    """numpy -> device tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(DEV)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32).copy()).to(DEV)
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def words_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def assert_close(y_gpu: np.ndarray, y_ref: np.ndarray, what: str = ""):
    """The contract: max |err| <= 1e-2 * (1 + |ref|) elementwise.  Because that bound is loose for
    outputs much smaller than 1, a second, self-imposed bound catches wrong-alpha / wrong-tile bugs:
    |err| <= 2e-2 * rms(ref) + 2^-8 * |ref| (the second term is half a bf16 ulp of the stored output)."""
    assert y_gpu.shape == y_ref.shape, (what, y_gpu.shape, y_ref.shape)
    err = np.abs(y_gpu - y_ref)
    bound = 1e-2 * (1.0 + np.abs(y_ref))
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, f"{what}: max err/bound = {worst:.3g}"
    rms = float(np.sqrt(np.mean(y_ref ** 2))) if err.size else 0.0
    if rms > 0:
        tight = 2e-2 * rms + np.abs(y_ref) / 256.0
        w2 = float((err / tight).max())
        assert w2 <= 1.0, f"{what}: max err / (2e-2 rms + half bf16 ulp) = {w2:.3g}"


def make_linear_case(seed, T, m, n, k, per_tile=True, x_bf16=True, w_sigma=0.02):
    """Seeded inputs + the oracle's tile/alpha for one fully-connected layer."""
    x, W = synth.linear_layer(seed, T, n, m, x_bf16=x_bf16, w_sigma=w_sigma)
    words, al = O.prepare(W, k, per_tile)
    return x, W, words, al
