"""GPU parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(AUTO path, caller-sized workspace): all outputs on the GPU, a seeded sample of rows / images through the
CPU oracle.  The small configurations are covered element by element in the other test files."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, to_dev, to_np64

pytestmark = pytest.mark.gpu


def sweep_sample_rows(T: int, count: int = 512) -> np.ndarray:
    """Token rows for the oracle at the sweep's largest batch: at least one row inside every token tile of both tile
    widths the kernel uses there (224 and 256 tokens), the first and the last row, and seeded random rows up to
    `count` in all."""
    rows = {0, T - 1}
    for width in (224, 256):
        for i in range((T + width - 1) // width):
            rows.add(min(i * width + (i * 37 + 11) % width, T - 1))
    rng = np.random.default_rng(4)
    while len(rows) < count:
        rows.add(int(rng.integers(0, T)))
    return np.array(sorted(rows), dtype=np.int64)


def test_large_linear_sweep_full_size_sampled_rows():
    # in = out = 8192, T = 16384 bf16 tokens, W ~ N(0, 0.02^2) aggregated on the GPU, per-tile alpha, seed 4
    c = synth.config_large_linear(16384)
    xd, Wd = to_dev(c["x"]), to_dev(c["W"])
    rows = sweep_sample_rows(c["T"])
    assert len(rows) >= 512
    y = torch.empty((c["T"], c["m"]), dtype=torch.bfloat16, device=DEV)
    ws = torch.empty(max(max(B.tbn_linear_workspace_bytes(c["T"], c["n"], c["m"], k, B.BF16) for k in (2, 4, 8, 16)), 16),
                     dtype=torch.uint8, device=DEV)
    for k in (2, 4, 8, 16):
        tile, alpha = B.tbn_aggregate_tile(Wd, k, B.ALPHA_PER_TILE)
        words, al = O.prepare(c["W"], k, True)
        assert np.array_equal(tile.cpu().numpy().view(np.uint32), words)
        assert np.allclose(alpha.cpu().numpy(), al, rtol=1e-6)
        assert B.tbn_linear_select_path(c["T"], c["n"], c["m"], k, B.BF16) == B.PATH_TENSOR
        y.fill_(float("nan"))
        B.tbn_linear_fwd(xd, c["m"], tile, k, alpha, B.ALPHA_PER_TILE, y=y, workspace=ws)
        torch.cuda.synchronize()
        assert not bool(torch.isnan(y).any()), "an output element was never written"
        ref = O.linear(c["x"][rows], words, k, al, True, c["m"], c["n"])
        assert_close(to_np64(y[torch.from_numpy(rows).to(DEV)]), ref, f"large linear k={k}")
        # the k repetitions of a distinct row differ only by alpha_j (Sec. 4.1): a property of the whole output that
        # holds at any size (the sampled rows above are what is compared with the oracle)
        r = c["m"] // k
        z0 = y[:, :r].float() / alpha[0]
        zj = y[:, (k - 1) * r:].float() / alpha[k - 1]
        assert torch.allclose(z0, zj, rtol=2e-2, atol=2e-2 * float(z0.abs().mean()))
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("T", [1, 16, 256, 4096])
def test_large_linear_sweep_smaller_batches(T):
    c = synth.config_large_linear(T)
    xd = to_dev(c["x"])
    for k in (2, 16):
        words, al = O.prepare(c["W"], k, True)
        ws = torch.empty(max(B.tbn_linear_workspace_bytes(T, c["n"], c["m"], k, B.BF16), 16), dtype=torch.uint8, device=DEV)
        y = B.tbn_linear_fwd(xd, c["m"], to_dev(words), k, to_dev(al), B.ALPHA_PER_TILE, workspace=ws)
        torch.cuda.synchronize()
        rows = np.unique(np.linspace(0, T - 1, min(T, 4)).astype(np.int64))
        ref = O.linear(c["x"][rows], words, k, al, True, c["m"], c["n"])
        assert_close(to_np64(y)[rows], ref, f"large linear T={T} k={k}")


@pytest.mark.parametrize("n,m", [(768, 2304), (768, 768), (768, 3072), (3072, 768)])
def test_vit_block_linears_full_size_sampled_rows(n, m):
    # ViT-B shaped encoder block: 128 images x 197 tokens, d = 768, MLP 3072; tiles with k = 8, seed 3
    T, k = 128 * 197, 8
    x, W = synth.linear_layer(3, T, n, m, x_bf16=True)
    words, al = O.prepare(W, k, True)
    y = B.tbn_linear_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), B.ALPHA_PER_TILE, act=B.ACT_GELU if m == 3072 else B.ACT_NONE)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(3).choice(T, 24, replace=False))
    rows[-1] = T - 1
    ref = O.linear(x[rows], words, k, al, True, m, n, act=O.ACT_GELU if m == 3072 else O.ACT_NONE)
    assert_close(to_np64(y)[rows], ref, f"vit linear {n}->{m}")


@pytest.mark.parametrize("Cin,H,Cout,stride", [(64, 32, 128, 2), (128, 16, 256, 2), (64, 32, 128, 1)])
def test_conv_stack_layers_full_batch_sampled_images(Cin, H, Cout, stride):
    # ResNet-style 3x3 convolutions, batch 256, NCHW bf16 ~U(0,1), Kaiming-normal weights, k = 4, seed 2
    x, W = synth.conv_layer(2, 256, Cin, H, H, Cout, 3, 3)
    words, al = O.prepare(W, 4, True)
    y = B.tbn_conv2d_fwd(to_dev(x), Cout, 3, 3, stride, 1, to_dev(words), 4, to_dev(al), B.ALPHA_PER_TILE, act=B.ACT_RELU)
    torch.cuda.synchronize()
    imgs = np.array([0, 101, 255])
    ref = O.conv2d(x[imgs], words, 4, al, True, Cout, Cin, 3, 3, stride, 1, act=O.ACT_RELU)
    assert_close(to_np64(y)[imgs], ref, f"conv {Cin}->{Cout} s{stride}")
    assert B.tbn_last_device_status() == (0, 0)
