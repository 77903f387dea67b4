"""GPU parity, fully-connected forward: every kernel family against the CPU oracle on the same
seeded inputs, element by element, within max|err| <= 1e-2 * (1 + |ref|)."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, make_linear_case, to_dev, to_np64

pytestmark = pytest.mark.gpu

# (m, n, k): a shape zoo -- aligned, misaligned, several tiles per row, nothing divides
ZOO = [(8, 8, 1), (8, 8, 2), (8, 8, 8), (128, 784, 4), (10, 128, 1), (512, 512, 4), (2304, 768, 8),
       (96, 40, 6), (6, 64, 4), (4, 64, 8), (7, 33, 3)]
TOKENS = [1, 2, 3, 17, 64, 129]


def run(path, x, words, al, per_tile, m, k, act=B.ACT_NONE, bias=None, y_dtype=None):
    y = B.tbn_linear_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), int(per_tile),
                         bias=None if bias is None else to_dev(bias), act=act, y_dtype=y_dtype, path=path)
    torch.cuda.synchronize()
    return to_np64(y)


@pytest.mark.parametrize("m,n,k", ZOO)
@pytest.mark.parametrize("T", TOKENS)
def test_generic_path_matches_oracle(m, n, k, T):
    for per_tile in (False, True):
        for x_bf16 in (False, True):
            x, W, words, al = make_linear_case(100 + T, T, m, n, k, per_tile, x_bf16, w_sigma=1.0)
            ref = O.linear(x, words, k, al, per_tile, m, n)
            got = run(B.PATH_GENERIC, x, words, al, per_tile, m, k, y_dtype=B.F32)
            assert_close(got, ref, f"generic {m}x{n} k={k} T={T}")


ALIGNED = [(m, n, k) for (m, n, k) in ZOO if (m * n // k) % n == 0 and n % 8 == 0]


@pytest.mark.parametrize("m,n,k", ALIGNED + [(2048, 1024, 8), (64, 8200, 2)])
@pytest.mark.parametrize("T", [1, 2, 3, 5, 12, 17, 40, 70])
def test_small_batch_path_matches_oracle(m, n, k, T):
    for per_tile in (False, True):
        for x_bf16 in (False, True):
            x, W, words, al = make_linear_case(200 + T, T, m, n, k, per_tile, x_bf16)
            ref = O.linear(x, words, k, al, per_tile, m, n, act=O.ACT_RELU)
            got = run(B.PATH_SMALL, x, words, al, per_tile, m, k, act=B.ACT_RELU)
            assert_close(got, ref, f"small {m}x{n} k={k} T={T}")


def test_small_batch_rejects_misaligned_tiles():
    x, W, words, al = make_linear_case(1, 2, 6, 64, 4)
    with pytest.raises(B.TbnError) as e:
        run(B.PATH_SMALL, x, words, al, True, 6, 4)
    assert e.value.status == -3


@pytest.mark.parametrize("act", [B.ACT_NONE, B.ACT_RELU, B.ACT_GELU])
@pytest.mark.parametrize("path", [B.PATH_GENERIC, B.PATH_SMALL, B.PATH_AUTO])
def test_bias_activation_and_output_dtypes(act, path):
    m, n, k, T = 64, 128, 4, 5
    x, W, words, al = make_linear_case(7, T, m, n, k, True, True, w_sigma=1.0)
    bias = synth.normal(7, 200, m)
    ref = O.linear(x, words, k, al, True, m, n, bias=bias.astype(np.float64), act=act)
    for yd in (B.F32, B.BF16):
        got = run(path, x, words, al, True, m, k, act=act, bias=bias, y_dtype=yd)
        assert_close(got, ref, f"act={act} path={path} yd={yd}")


def test_single_fc_config_all_paths_agree():
    # single layer 512 -> 512, k = 4, batch 64, fp32 activations, W ~ N(0, 0.02), seed 0
    c = synth.config_single_fc()
    words, al = O.prepare(c["W"], c["k"], True)
    tile, alpha = B.tbn_aggregate_tile(to_dev(c["W"]), c["k"], B.ALPHA_PER_TILE)
    assert np.array_equal(tile.cpu().numpy().view(np.uint32), words)
    ref = O.linear(c["x"], words, c["k"], al, True, c["m"], c["n"])
    xd = to_dev(c["x"])
    outs = {}
    for path in (B.PATH_GENERIC, B.PATH_SMALL, B.PATH_AUTO):
        y = B.tbn_linear_fwd(xd, c["m"], tile, c["k"], alpha, B.ALPHA_PER_TILE, path=path)
        outs[path] = to_np64(y)
        assert_close(outs[path], ref, f"config 1 path {path}")
    # shortcut kernels vs the generic kernel (which never uses the shortcut): fp32 reassociation only
    assert np.allclose(outs[B.PATH_SMALL], outs[B.PATH_GENERIC], rtol=1e-4, atol=1e-5)


def test_zero_tokens_is_a_noop_and_zero_alpha_gives_zeros():
    m, n, k = 16, 32, 2
    x, W, words, al = make_linear_case(3, 4, m, n, k)
    y = B.tbn_linear_fwd(torch.empty((0, n), dtype=torch.bfloat16, device=DEV), m, to_dev(words), k,
                         to_dev(al), B.ALPHA_PER_TILE)
    assert y.shape == (0, m)
    got = run(B.PATH_AUTO, x, words, np.zeros(k, np.float32), True, m, k)
    assert np.all(got == 0)


def test_host_buffer_entry_point_matches_device_entry_point():
    m, n, k, T = 256, 512, 4, 33
    x, W, words, al = make_linear_case(9, T, m, n, k)
    xh = torch.from_numpy(x.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    yh = torch.empty((T, m), dtype=torch.bfloat16).pin_memory()
    ws = torch.empty(B.tbn_linear_host_workspace_bytes(T, n, m, k, B.BF16, B.BF16), dtype=torch.uint8, device=DEV)
    tile, alpha = to_dev(words), to_dev(al)
    B.tbn_linear_fwd_host(xh, yh, tile, k, alpha, B.ALPHA_PER_TILE, ws)
    yd = B.tbn_linear_fwd(xh.to(DEV), m, tile, k, alpha, B.ALPHA_PER_TILE)
    assert torch.equal(yh, yd.cpu())
    assert_close(to_np64(yh), O.linear(x, words, k, al, True, m, n), "host entry point")


def test_host_buffer_entry_point_chunked_pipeline():
    # rows of 16 KB: the batch is large enough to go through in several chunks with a ragged last one (copies in,
    # compute and copies out overlap); every token row must still come back, in its place
    m, n, k, T = 1024, 8192, 4, 4708
    x, W, words, al = make_linear_case(12, T, m, n, k)
    xh = torch.from_numpy(x.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    tile, alpha = to_dev(words), to_dev(al)
    ws = torch.empty(B.tbn_linear_host_workspace_bytes(T, n, m, k, B.BF16, B.BF16), dtype=torch.uint8, device=DEV)
    yd = B.tbn_linear_fwd(xh.to(DEV), m, tile, k, alpha, B.ALPHA_PER_TILE).cpu()
    for _ in range(2):                                        # the second call reuses the copy streams and events
        yh = torch.full((T, m), float("nan"), dtype=torch.bfloat16).pin_memory()
        B.tbn_linear_fwd_host(xh, yh, tile, k, alpha, B.ALPHA_PER_TILE, ws)
        assert not torch.isnan(yh).any()
        assert_close(to_np64(yh), to_np64(yd), "chunked host entry point vs device entry point")
    rows = np.r_[0:8, 2040:2056, 4090:4104, T - 8:T]          # chunk seams and the tail
    assert_close(to_np64(yh)[rows], O.linear(x[rows], words, k, al, True, m, n), "chunked host entry point")
    assert B.tbn_last_device_status() == (0, 0)


# ------------------------------------------------------------------------------------------------
# tensor-core (tcgen05) path
TENSOR_SHAPES = ALIGNED + [(2048, 1024, 8), (64, 8200, 2), (256, 72, 1), (1024, 4096, 2)]


@pytest.mark.parametrize("m,n,k", TENSOR_SHAPES)
@pytest.mark.parametrize("T", [1, 3, 17, 64, 129, 200, 500])
def test_tensor_path_matches_oracle(m, n, k, T):
    for per_tile in (False, True):
        x, W, words, al = make_linear_case(300 + T, T, m, n, k, per_tile, True)
        ref = O.linear(x, words, k, al, per_tile, m, n, act=O.ACT_RELU)
        got = run(B.PATH_TENSOR, x, words, al, per_tile, m, k, act=B.ACT_RELU)
        assert_close(got, ref, f"tensor {m}x{n} k={k} T={T}")
    assert B.tbn_last_device_status() == (0, 0)


def test_tensor_path_fp32_activations_bias_fp32_out():
    m, n, k, T = 512, 512, 4, 64
    x, W, words, al = make_linear_case(0, T, m, n, k, True, False)
    bias = synth.normal(0, 200, m, 0.1)
    ref = O.linear(x, words, k, al, True, m, n, bias=bias.astype(np.float64), act=O.ACT_GELU)
    got = run(B.PATH_TENSOR, x, words, al, True, m, k, act=B.ACT_GELU, bias=bias, y_dtype=B.F32)
    assert_close(got, ref, "tensor fp32 in/out")


def test_tensor_path_gelu_bf16_out_wide_range():
    # bf16 outputs take the tanh-form GELU (fitted to the erf form, special-function tanh).  Pre-activations here
    # spread over about [-9, 9], so the fit's whole range, both tails and the cap on v^2 are exercised; beside the
    # contract bound the error must stay within the form's own budget, 2.5e-5 + 2.5e-4 |v|, plus the bf16 rounding
    # of the stored value.
    m, n, k, T = 512, 256, 4, 300
    x, W, words, al = make_linear_case(31, T, m, n, k, True, True, w_sigma=0.2)
    bias = synth.normal(31, 200, m, 0.5)
    pre = O.linear(x, words, k, al, True, m, n, bias=bias.astype(np.float64))
    assert pre.min() < -6.0 and pre.max() > 6.0
    ref = O.linear(x, words, k, al, True, m, n, bias=bias.astype(np.float64), act=O.ACT_GELU)
    got = run(B.PATH_TENSOR, x, words, al, True, m, k, act=B.ACT_GELU, bias=bias, y_dtype=B.BF16)
    assert_close(got, ref, "tensor gelu bf16")
    # fp32 accumulation of 256 bf16 products moves v by ~1e-5 |v|; the stored value is rounded to bf16 (half an ulp: up to 2^-8 relative)
    budget = 2.5e-5 + 3.0e-4 * np.abs(pre) + np.abs(ref) / 256.0 + 1e-6
    assert float((np.abs(got - ref) / budget).max()) <= 1.0


@pytest.fixture
def forced_config():
    """Pins the tensor-core linear kernel's tile shape / split factor for one test and always restores the
    automatic choice."""
    yield B.tbn_debug_force_linear_config
    B.tbn_debug_force_linear_config(-1)


def tile_shape_count() -> int:
    n = 0
    while B.lib().tbn_debug_force_linear_config(n, 1) == 0:
        n += 1
    B.tbn_debug_force_linear_config(-1)
    return n


@pytest.mark.parametrize("splits", [1, 2, 4])
def test_tensor_path_every_tile_shape(splits, forced_config):
    # the planner picks one token-tile shape per call; the tuning hook pins each of them in turn on a case with
    # several token tiles, a ragged token tail and a ragged row block, unsplit and with the contraction split
    m, n, k, T = 1200, 1000, 4, 777
    x, W, words, al = make_linear_case(21, T, m, n, k, True, True)
    ref = O.linear(x, words, k, al, True, m, n)
    count = tile_shape_count()
    assert count >= 7
    ws = torch.empty(64 << 20, dtype=torch.uint8, device=DEV)
    for cand in range(count):
        forced_config(cand, splits)
        y = B.tbn_linear_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), 1, path=B.PATH_TENSOR, workspace=ws)
        torch.cuda.synchronize()
        assert_close(to_np64(y), ref, f"tensor tile shape {cand} splits {splits}")
    assert B.tbn_last_device_status() == (0, 0)


def test_forced_config_rejects_invalid_split_factors():
    for bad in (0, 3, 5, 6, 32, -1):
        assert B.lib().tbn_debug_force_linear_config(0, bad) == -1
    assert B.lib().tbn_debug_force_linear_config(10 ** 6, 1) == -1
    B.tbn_debug_force_linear_config(-1)


@pytest.mark.parametrize("k", [2, 16])
def test_tensor_path_many_tiles_sampled_rows(k):
    # several waves of CTA tiles, ragged token tail; a seeded sample of rows through the oracle
    m, n, T = 4096, 2048, 3000
    x, W, words, al = make_linear_case(11, T, m, n, k, True, True)
    got = run(B.PATH_TENSOR, x, words, al, True, m, k)
    rows = np.sort(np.random.default_rng(1).choice(T, 40, replace=False))
    rows[-1] = T - 1
    ref = O.linear(x[rows], words, k, al, True, m, n)
    assert_close(got[rows], ref, f"tensor many tiles k={k}")
    # and the whole output against the generic kernel (no shortcut, CUDA cores)
    gen = run(B.PATH_GENERIC, x, words, al, True, m, k)
    assert_close(got, gen, "tensor vs generic")
    assert B.tbn_last_device_status() == (0, 0)


@pytest.mark.parametrize("T,m,n,k", [(1, 8192, 8192, 2), (16, 8192, 8192, 16), (40, 4096, 4096, 4), (256, 2048, 8192, 8),
                                     (3, 512, 2056, 2)])
def test_tensor_path_split_k_matches_oracle_and_is_deterministic(T, m, n, k):
    # few output tiles, long contraction: the kernel splits K over several CTAs and adds the partial tiles in a
    # fixed order; sampled output columns through the oracle, and run-to-run bit equality
    x, W, words, al = make_linear_case(21, T, m, n, k, True, True)
    assert B.tbn_linear_workspace_bytes(T, n, m, k, B.BF16) > 0          # split-K scratch is requested
    xd, td, ad = to_dev(x), to_dev(words), to_dev(al)
    y1 = B.tbn_linear_fwd(xd, m, td, k, ad, 1, act=B.ACT_RELU, path=B.PATH_TENSOR)
    y2 = B.tbn_linear_fwd(xd, m, td, k, ad, 1, act=B.ACT_RELU, path=B.PATH_TENSOR)
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)
    ref = O.linear(x, words, k, al, True, m, n, act=O.ACT_RELU)
    assert_close(to_np64(y1), ref, f"split-K T={T} {m}x{n} k={k}")
    # without scratch the kernel runs unsplit and must agree to fp32 reassociation
    y3 = B.tbn_linear_fwd(xd, m, td, k, ad, 1, act=B.ACT_RELU, path=B.PATH_TENSOR,
                          workspace=torch.empty(16, dtype=torch.uint8, device=DEV))
    assert_close(to_np64(y3), ref, "unsplit")
    assert B.tbn_last_device_status() == (0, 0)
