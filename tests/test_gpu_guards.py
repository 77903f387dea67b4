"""Two safety nets that need a GPU.  (1) The bounded waits of the tensor-core kernels really give up: a probe kernel
waits, through the same routines, on a barrier nothing arrives at, with the limit shortened to a fraction of a
millisecond; it must return, leave TBN_ERR_TIMEOUT and its detail in the status word, and the next ordinary launch must
work.  Nothing is starved and nothing waits unbounded.  (2) Guard bands: outputs of every kernel family are written
into the middle of a larger buffer whose margins hold a known pattern, with ragged shapes; the margins must be
untouched afterwards (a substitute for a memory checker on ragged-edge stores)."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import DEV, assert_close, make_linear_case, to_dev, to_np64

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    assert B.tbn_last_device_status() == (0, 0)
    B.tbn_debug_set_wait_limit_us(200)
    try:
        detail = (12 << 24) | 345
        B.tbn_debug_wait_timeout_probe(detail)
        code, got = B.tbn_last_device_status()
        assert code == -6 and got in (detail, detail + 1), (code, got)     # whichever waiter ran out first
        assert B.tbn_last_device_status() == (0, 0)                         # reading cleared the record, not the limit
        B.tbn_debug_wait_timeout_probe(7)
        assert B.tbn_last_device_status()[0] == -6
    finally:
        B.tbn_debug_set_wait_limit_us(0)
    # an ordinary tensor-core launch afterwards: correct result, clean status
    m, n, k, T = 256, 256, 4, 300
    x, W, words, al = make_linear_case(95, T, m, n, k)
    y = B.tbn_linear_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), 1, path=B.PATH_TENSOR)
    torch.cuda.synchronize()
    assert_close(to_np64(y), O.linear(x, words, k, al, True, m, n), "after the probe")
    assert B.tbn_last_device_status() == (0, 0)


class Guarded:
    """An output tensor in the middle of a buffer with 8 KiB margins of a known byte pattern."""
    MARGIN = 8192

    def __init__(self, shape, dtype):
        self.nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-self.nbytes) % 256
        self.buf = torch.full((2 * self.MARGIN + self.nbytes + pad,), 0xA5, dtype=torch.uint8, device=DEV)
        self.out = self.buf[self.MARGIN:self.MARGIN + self.nbytes].view(dtype).view(*shape)

    def check(self, what):
        torch.cuda.synchronize()
        head, tail = self.buf[:self.MARGIN], self.buf[self.MARGIN + self.nbytes:]
        assert bool((head == 0xA5).all()) and bool((tail == 0xA5).all()), f"{what}: wrote outside its output"


@pytest.mark.parametrize("path", [B.PATH_GENERIC, B.PATH_SMALL, B.PATH_TENSOR])
@pytest.mark.parametrize("T,m,n,k,dtype", [(777, 1200, 1000, 4, torch.bfloat16), (3, 40, 72, 5, torch.float32),
                                           (129, 136, 264, 1, torch.bfloat16), (65, 2304, 768, 8, torch.float32)])
def test_linear_outputs_stay_inside_their_buffer(path, T, m, n, k, dtype):
    x, W, words, al = make_linear_case(96, T, m, n, k)
    g = Guarded((T, m), dtype)
    yd = B.BF16 if dtype == torch.bfloat16 else B.F32
    try:
        B.tbn_linear_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), 1, act=B.ACT_RELU, y_dtype=yd, path=path, y=g.out)
    except B.TbnError as e:
        assert e.status == -3
        return
    g.check(f"linear path {path}")
    assert_close(to_np64(g.out), O.linear(x, words, k, al, True, m, n, act=O.ACT_RELU), "guarded linear")


@pytest.mark.parametrize("T,m,n,k,splits", [(40, 520, 2056, 4, 4), (200, 264, 4096, 2, 8)])
def test_split_k_outputs_stay_inside_their_buffer(T, m, n, k, splits):
    x, W, words, al = make_linear_case(97, T, m, n, k)
    g = Guarded((T, m), torch.bfloat16)
    ws = torch.empty(64 << 20, dtype=torch.uint8, device=DEV)
    B.tbn_debug_force_linear_config(3, splits)
    try:
        B.tbn_linear_fwd(to_dev(x), m, to_dev(words), k, to_dev(al), 1, path=B.PATH_TENSOR, y=g.out, workspace=ws)
    finally:
        B.tbn_debug_force_linear_config(-1)
    g.check("split-K linear")
    assert_close(to_np64(g.out), O.linear(x, words, k, al, True, m, n), "guarded split-K")


@pytest.mark.parametrize("Nb,Cout,Cin,k,stride,pad,H,W", [(3, 200, 32, 4, 1, 1, 12, 20), (3, 32, 16, 2, 2, 1, 13, 16),
                                                          (2, 8, 3, 2, 2, 1, 9, 9), (5, 32, 16, 2, 1, 1, 4, 4)])
def test_conv_outputs_stay_inside_their_buffer(Nb, Cout, Cin, k, stride, pad, H, W):
    x, Wt = synth.conv_layer(98, Nb, Cin, H, W, Cout, 3, 3)
    words, al = O.prepare(Wt, k, True)
    Ho, Wo = O.conv_out_hw(H, W, 3, 3, stride, pad)
    g = Guarded((Nb, Cout, Ho, Wo), torch.bfloat16)
    B.tbn_conv2d_fwd(to_dev(x), Cout, 3, 3, stride, pad, to_dev(words), k, to_dev(al), 1, act=B.ACT_RELU, y=g.out)
    g.check("conv")
    assert_close(to_np64(g.out), O.conv2d(x, words, k, al, True, Cout, Cin, 3, 3, stride, pad, act=O.ACT_RELU), "guarded conv")


@pytest.mark.parametrize("path", [B.PATH_GENERIC, B.PATH_TENSOR])
@pytest.mark.parametrize("T,m,n,k,yd", [(777, 1200, 992, 4, B.BF16), (33, 40, 64, 5, B.F32), (130, 136, 256, 1, B.I32)])
def test_binary_layer_outputs_stay_inside_their_buffer(path, T, m, n, k, yd):
    x = synth.to_bf16_bits(synth.normal(99, 0, T * n).reshape(T, n))
    words, al = O.prepare(synth.normal(99, 1, m * n, n ** -0.5), k, True)
    abits, beta = O.binarize(x)
    g = Guarded((T, m), {B.BF16: torch.bfloat16, B.F32: torch.float32, B.I32: torch.int32}[yd])
    gb = Guarded((T, O.row_words(n)), torch.int32)
    B.tbn_binarize_fwd(to_dev(x), x_bits=gb.out, beta=torch.empty(T, device=DEV))
    gb.check("binarize")
    try:
        B.tbn_linear_bin_fwd(gb.out, n, m, to_dev(words), k, to_dev(al), 1, beta=to_dev(beta), y_dtype=yd, path=path, y=g.out)
    except B.TbnError as e:
        assert e.status == -3
        return
    g.check(f"binary layer path {path}")
    if yd == B.I32:
        assert np.array_equal(g.out.cpu().numpy().astype(np.int64), O.linear_bin_int(abits, words, k, m, n))
    else:
        assert_close(to_np64(g.out), O.linear_bin(abits, beta, words, k, al, True, m, n), "guarded binary layer")


def test_mlp_and_block_outputs_stay_inside_their_buffer():
    T, dims, ks = 333, [64, 512, 512, 10], [8, 2, 1]
    x = synth.to_bf16_bits(synth.normal(100, 0, T * dims[0]).reshape(T, dims[0]))
    layers, tiles, alphas = [], [], []
    for l in range(3):
        words, al = O.prepare(synth.normal(100, 1 + l, dims[l + 1] * dims[l], dims[l] ** -0.5), ks[l], True)
        layers.append(dict(words=words, p=ks[l], alphas=al, per_tile=True, m=dims[l + 1], n=dims[l]))
        tiles.append(to_dev(words)); alphas.append(to_dev(al))
    g = Guarded((T, dims[-1]), torch.bfloat16)
    B.tbn_mlp_fwd(to_dev(x), dims, tiles, ks, alphas, [1, 1, 1], y=g.out)
    g.check("mlp")
    assert_close(to_np64(g.out), O.mlp(x, layers), "guarded mlp")
    Nb, S, d, heads, mlp = 3, 37, 128, 2, 200
    xb = synth.to_bf16_bits(synth.normal(101, 0, Nb * S * d).reshape(Nb * S, d))
    shapes = dict(qkv=(3 * d, d), proj=(d, d), fc1=(mlp, d), fc2=(d, mlp))
    blayers, btiles, balphas = {}, [], []
    for l, (name, (m_, n_)) in enumerate(shapes.items()):
        words, al = O.prepare(synth.normal(101, 1 + l, m_ * n_, n_ ** -0.5), 4, True)
        blayers[name] = dict(words=words, p=4, alphas=al, per_tile=True, m=m_, n=n_)
        btiles.append(to_dev(words)); balphas.append(to_dev(al))
    g = Guarded((Nb * S, d), torch.bfloat16)
    B.tbn_vit_block_fwd(to_dev(xb), Nb, S, heads, mlp, btiles, [4] * 4, balphas, [1] * 4, y=g.out)
    g.check("encoder block")
    assert_close(to_np64(g.out), O.vit_block(xb, Nb, S, heads, blayers), "guarded block")
