"""ctypes binding of libtbn.so: the same entry points as include/tbn.h, argument marshalling only.

Tensors are torch tensors (device memory and streams come from torch; every step of the
computation runs inside the library's kernels).  There is no fallback: if the shared library is
missing or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtbn.so")

OK = 0
F32, BF16, I32 = 0, 1, 2
ALPHA_PER_LAYER, ALPHA_PER_TILE = 0, 1
ACT_NONE, ACT_RELU, ACT_GELU = 0, 1, 2
PATH_AUTO, PATH_GENERIC, PATH_SMALL, PATH_TENSOR = 0, 1, 2, 3

c_i32, c_i64, c_int, c_vp, c_sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t

_LINEAR_ARGS = [c_vp, c_int, c_i64, c_i32, c_i32, c_vp, c_i32, c_vp, c_int, c_vp, c_int, c_vp, c_int,
                c_vp, c_sz, c_vp]
_CONV_ARGS = [c_vp, c_int] + [c_i32] * 9 + [c_vp, c_i32, c_vp, c_int, c_vp, c_int, c_vp, c_int, c_vp, c_sz, c_vp]

SIGNATURES = {
    "tbn_tile_words": (c_i64, [c_i64]),
    "tbn_status_string": (ctypes.c_char_p, [c_int]),
    "tbn_aggregate_workspace_bytes": (c_sz, [c_i64, c_i32]),
    "tbn_aggregate_tile": (c_int, [c_vp, c_vp, c_i64, c_i32, c_int, c_vp, c_vp, c_vp, c_sz, c_vp]),
    "tbn_aggregate_tile_static": (c_int, [c_vp, c_vp, c_i64, c_i32, c_int, c_vp, c_vp, c_vp]),
    "tbn_pack_tile": (c_int, [c_vp, c_i64, c_vp, c_vp]),
    "tbn_expand_tile": (c_int, [c_vp, c_i64, c_i32, c_vp, c_int, c_vp, c_vp]),
    "tbn_linear_workspace_bytes": (c_sz, [c_i64, c_i32, c_i32, c_i32, c_int]),
    "tbn_linear_fwd": (c_int, _LINEAR_ARGS),
    "tbn_linear_fwd_path": (c_int, _LINEAR_ARGS + [c_int]),
    "tbn_linear_select_path": (c_int, [c_i64, c_i32, c_i32, c_i32, c_int]),
    "tbn_linear_res_fwd": (c_int, [c_vp, c_int, c_i64, c_i32, c_i32, c_vp, c_i32, c_vp, c_int, c_vp, c_int, c_vp, c_vp, c_int,
                                   c_vp, c_sz, c_vp, c_int]),
    "tbn_linear_compact_fwd": (c_int, [c_vp, c_i64, c_i32, c_i32, c_vp, c_int, c_int, c_i32, c_vp, c_i32, c_vp, c_int, c_vp, c_int,
                                       c_vp, c_int, c_vp]),
    "tbn_layernorm_fwd": (c_int, [c_vp, c_int, c_i64, c_i32, c_vp, c_vp, ctypes.c_float, c_vp, c_int, c_vp]),
    "tbn_attention_fwd": (c_int, [c_vp, c_i32, c_i32, c_i32, c_i32, c_vp, c_vp]),
    "tbn_vit_block_workspace_bytes": (c_sz, [c_i32, c_i32, c_i32, c_i32, c_vp]),
    "tbn_vit_block_fwd": (c_int, [c_vp, c_i32, c_i32, c_i32, c_i32, c_i32, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_sz, c_vp]),
    "tbn_linear_fp_tile_workspace_bytes": (c_sz, [c_i64, c_i32, c_i32, c_i32, c_int, c_int]),
    "tbn_linear_fp_tile_fwd": (c_int, [c_vp, c_int, c_i64, c_i32, c_i32, c_vp, c_int, c_i32, c_vp, c_int, c_vp, c_int,
                                       c_vp, c_sz, c_vp, c_int]),
    "tbn_linear_host_workspace_bytes": (c_sz, [c_i64, c_i32, c_i32, c_i32, c_int, c_int]),
    "tbn_linear_fwd_host": (c_int, _LINEAR_ARGS),
    "tbn_conv2d_workspace_bytes": (c_sz, [c_i32] * 10 + [c_int]),
    "tbn_conv2d_fwd": (c_int, _CONV_ARGS),
    "tbn_conv2d_fwd_path": (c_int, _CONV_ARGS + [c_int]),
    "tbn_conv2d_dense_fwd": (c_int, [c_vp, c_int] + [c_i32] * 9 + [c_vp, c_vp, c_int, c_vp, c_int, c_vp]),
    "tbn_global_avgpool_fwd": (c_int, [c_vp, c_int, c_i32, c_i32, c_i32, c_i32, c_vp, c_int, c_vp]),
    "tbn_mlp_workspace_bytes": (c_sz, [c_i64, c_i32, c_vp, c_vp, c_int]),
    "tbn_mlp_fwd": (c_int, [c_vp, c_int, c_i64, c_i32, c_vp, c_vp, c_vp, c_vp, c_vp, c_int, c_vp, c_int,
                            c_vp, c_sz, c_vp]),
    "tbn_last_device_status": (c_int, [c_vp, c_vp, c_vp]),
    "tbn_debug_record_status": (c_int, [c_int, c_int, c_vp]),
    "tbn_debug_set_wait_limit_us": (c_int, [c_int]),
    "tbn_debug_wait_timeout_probe": (c_int, [c_int, c_vp]),
    "tbn_debug_force_linear_config": (c_int, [c_int, c_int]),
    "tbn_debug_force_mlp_layerwise": (c_int, [c_int]),
    "tbn_debug_force_bin_config": (c_int, [c_int]),
    "tbn_tile_fwd": (c_int, [c_vp, c_vp, c_i64, c_i32, c_int, c_vp, c_int, c_vp, c_vp, c_vp, c_sz, c_vp]),
    "tbn_tile_bwd_workspace_bytes": (c_sz, [c_i64, c_i32]),
    "tbn_tile_bwd": (c_int, [c_vp, c_vp, c_vp, c_vp, c_vp, c_i64, c_i32, c_int, c_vp, c_vp, c_vp, c_vp, c_sz, c_vp]),
    "tbn_row_words": (c_i64, [c_i32]),
    "tbn_binarize_fwd": (c_int, [c_vp, c_int, c_i64, c_i32, c_vp, c_vp, c_vp]),
    "tbn_linear_bin_fwd": (c_int, [c_vp, c_i64, c_i32, c_i32, c_vp, c_i32, c_vp, c_int, c_vp, c_vp, c_int, c_vp, c_int,
                                   c_vp, c_int]),
    "tbn_debug_force_attention_path": (c_int, [c_int]),
    "tbn_avgpool_linear_fwd": (c_int, [c_vp, c_int, c_i32, c_i32, c_i32, c_i32, c_vp, c_vp, c_i32, c_vp, c_vp]),
    "tbn_bin_expand_fwd": (c_int, [c_vp, c_i64, c_i32, c_vp, c_vp, c_vp]),
    "tbn_binarize_bytes_fwd": (c_int, [c_vp, c_int, c_i64, c_i32, c_vp, c_vp, c_vp, c_vp, c_vp]),
    "tbn_linear_bin_bytes_fwd": (c_int, [c_vp, c_vp, c_i64, c_i32, c_i32, c_vp, c_i32, c_vp, c_int, c_vp, c_vp, c_int, c_vp,
                                         c_int, c_vp]),
}

_lib = None


class TbnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().tbn_status_string(status).decode() if _lib is not None else "?"
        super().__init__(f"{where}: status {status} ({msg})")


def lib() -> ctypes.CDLL:
    """Load libtbn.so (built in-tree by paper_2407_12075_b200.build); raise if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2407_12075_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise TbnError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _torch_dtype(code: int):
    return {BF16: torch.bfloat16, F32: torch.float32, I32: torch.int32}[code]


def _ws(nbytes: int, device):
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------------------------
def tbn_tile_words(q: int) -> int:
    return int(lib().tbn_tile_words(q))


def tbn_aggregate_tile(W: torch.Tensor, k: int, alpha_mode: int = ALPHA_PER_TILE, A: torch.Tensor | None = None,
                       workspace: torch.Tensor | None = None):
    """Eq. 1-3 and Eq. 6-8 on the device.  Returns (tile_bits int32[words], alpha float32[1 or k])."""
    N = W.numel()
    if k <= 0 or N % k:
        raise TbnError(-2, "tbn_aggregate_tile")
    tile = torch.empty(tbn_tile_words(N // k), dtype=torch.int32, device=W.device)
    alpha = torch.empty(k if alpha_mode == ALPHA_PER_TILE else 1, dtype=torch.float32, device=W.device)
    need = lib().tbn_aggregate_workspace_bytes(N, k)
    ws = workspace if workspace is not None else _ws(need, W.device)
    _check(lib().tbn_aggregate_tile(_ptr(W), _ptr(A), N, k, alpha_mode, _ptr(tile), _ptr(alpha), _ptr(ws),
                                    ws.numel(), _stream()), "tbn_aggregate_tile")
    return tile, alpha


def tbn_aggregate_tile_static(W: torch.Tensor, k: int, tile: torch.Tensor, alpha: torch.Tensor,
                              alpha_mode: int = ALPHA_PER_TILE, A: torch.Tensor | None = None):
    """Same result as tbn_aggregate_tile, for callers that cannot allocate: the scratch is an array built
    into the library (1 MiB per GPU), so this wrapper allocates nothing either -- the caller passes the
    output tensors.  Layers whose scratch need exceeds 1 MiB raise TbnError(-4).  Calls that could overlap
    on the GPU share the array and must be ordered by the caller; make the first call on a device before
    any stream capture."""
    _check(lib().tbn_aggregate_tile_static(_ptr(W), _ptr(A), W.numel(), k, alpha_mode, _ptr(tile), _ptr(alpha),
                                           _stream()), "tbn_aggregate_tile_static")
    return tile, alpha


def tbn_pack_tile(src: torch.Tensor) -> torch.Tensor:
    q = src.numel()
    tile = torch.empty(tbn_tile_words(q), dtype=torch.int32, device=src.device)
    _check(lib().tbn_pack_tile(_ptr(src), q, _ptr(tile), _stream()), "tbn_pack_tile")
    return tile


def tbn_expand_tile(tile: torch.Tensor, N: int, k: int, alpha: torch.Tensor, alpha_mode: int) -> torch.Tensor:
    out = torch.empty(N, dtype=torch.float32, device=tile.device)
    _check(lib().tbn_expand_tile(_ptr(tile), N, k, _ptr(alpha), alpha_mode, _ptr(out), _stream()),
           "tbn_expand_tile")
    return out


def tbn_linear_workspace_bytes(T, in_f, out_f, k, x_dtype) -> int:
    return int(lib().tbn_linear_workspace_bytes(T, in_f, out_f, k, x_dtype))


def tbn_linear_select_path(T, in_f, out_f, k, x_dtype) -> int:
    return int(lib().tbn_linear_select_path(T, in_f, out_f, k, x_dtype))


def tbn_linear_fwd(x: torch.Tensor, out_f: int, tile: torch.Tensor, k: int, alpha: torch.Tensor,
                   alpha_mode: int, bias: torch.Tensor | None = None, act: int = ACT_NONE,
                   y_dtype: int | None = None, path: int = PATH_AUTO, y: torch.Tensor | None = None,
                   workspace: torch.Tensor | None = None) -> torch.Tensor:
    T, in_f = x.shape
    xd = _dtype_code(x)
    yd = xd if y_dtype is None else y_dtype
    if y is None:
        y = torch.empty((T, out_f), dtype=_torch_dtype(yd), device=x.device)
    ws = workspace if workspace is not None else _ws(tbn_linear_workspace_bytes(T, in_f, out_f, k, xd), x.device)
    _check(lib().tbn_linear_fwd_path(_ptr(x), xd, T, in_f, out_f, _ptr(tile), k, _ptr(alpha), alpha_mode,
                                     _ptr(bias), act, _ptr(y), yd, _ptr(ws), ws.numel(), _stream(), path),
           "tbn_linear_fwd")
    return y


def tbn_linear_fp_tile_workspace_bytes(T, in_f, out_f, k, x_dtype, tile_dtype) -> int:
    return int(lib().tbn_linear_fp_tile_workspace_bytes(T, in_f, out_f, k, x_dtype, tile_dtype))


def tbn_linear_fp_tile_fwd(x: torch.Tensor, out_f: int, tile_values: torch.Tensor, k: int,
                           bias: torch.Tensor | None = None, act: int = ACT_NONE, y_dtype: int | None = None,
                           path: int = PATH_AUTO, y: torch.Tensor | None = None,
                           workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Layer whose weight is a real-valued tile (fp32 or bf16, q values) repeated k times."""
    T, in_f = x.shape
    xd, td = _dtype_code(x), _dtype_code(tile_values)
    yd = xd if y_dtype is None else y_dtype
    if y is None:
        y = torch.empty((T, out_f), dtype=_torch_dtype(yd), device=x.device)
    ws = workspace if workspace is not None else _ws(tbn_linear_fp_tile_workspace_bytes(T, in_f, out_f, k, xd, td),
                                                     x.device)
    _check(lib().tbn_linear_fp_tile_fwd(_ptr(x), xd, T, in_f, out_f, _ptr(tile_values), td, k, _ptr(bias), act,
                                        _ptr(y), yd, _ptr(ws), ws.numel(), _stream(), path),
           "tbn_linear_fp_tile_fwd")
    return y


def tbn_linear_host_workspace_bytes(T, in_f, out_f, k, x_dtype, y_dtype) -> int:
    return int(lib().tbn_linear_host_workspace_bytes(T, in_f, out_f, k, x_dtype, y_dtype))


def tbn_linear_fwd_host(x_host: torch.Tensor, y_host: torch.Tensor, tile, k, alpha, alpha_mode,
                        workspace: torch.Tensor, bias=None, act=ACT_NONE):
    """x_host / y_host are HOST tensors (pinned); workspace, tile, alpha live on the device."""
    T, in_f = x_host.shape
    out_f = y_host.shape[1]
    _check(lib().tbn_linear_fwd_host(_ptr(x_host), _dtype_code(x_host), T, in_f, out_f, _ptr(tile), k,
                                     _ptr(alpha), alpha_mode, _ptr(bias), act, _ptr(y_host),
                                     _dtype_code(y_host), _ptr(workspace), workspace.numel(), _stream()),
           "tbn_linear_fwd_host")
    return y_host


def tbn_conv2d_fwd(x: torch.Tensor, Cout: int, kh: int, kw: int, stride: int, pad: int, tile, k, alpha,
                   alpha_mode, bias=None, act=ACT_NONE, y_dtype=None, path=PATH_AUTO, y=None) -> torch.Tensor:
    Nb, Cin, H, Wd = x.shape
    xd = _dtype_code(x)
    yd = xd if y_dtype is None else y_dtype
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (Wd + 2 * pad - kw) // stride + 1
    if y is None:
        y = torch.empty((Nb, Cout, max(Ho, 0), max(Wo, 0)), dtype=_torch_dtype(yd), device=x.device)
    need = lib().tbn_conv2d_workspace_bytes(Nb, Cin, H, Wd, Cout, kh, kw, stride, pad, k, xd)
    ws = _ws(need, x.device)
    _check(lib().tbn_conv2d_fwd_path(_ptr(x), xd, Nb, Cin, H, Wd, Cout, kh, kw, stride, pad, _ptr(tile), k,
                                     _ptr(alpha), alpha_mode, _ptr(bias), act, _ptr(y), yd, _ptr(ws),
                                     ws.numel(), _stream(), path), "tbn_conv2d_fwd")
    return y


def _i32_array(vals):
    return (c_i32 * len(vals))(*[int(v) for v in vals])


def tbn_mlp_workspace_bytes(T, dims, ks, x_dtype) -> int:
    L = len(ks)
    return int(lib().tbn_mlp_workspace_bytes(T, L, ctypes.cast(_i32_array(dims), c_vp),
                                             ctypes.cast(_i32_array(ks), c_vp), x_dtype))


def tbn_mlp_fwd(x: torch.Tensor, dims, tiles, ks, alphas, alpha_modes, hidden_act=ACT_RELU, y_dtype=None,
                workspace: torch.Tensor | None = None, y: torch.Tensor | None = None) -> torch.Tensor:
    T = x.shape[0]
    L = len(ks)
    xd = _dtype_code(x)
    yd = xd if y_dtype is None else y_dtype
    if y is None:
        y = torch.empty((T, dims[-1]), dtype=_torch_dtype(yd), device=x.device)
    ws = workspace if workspace is not None else _ws(tbn_mlp_workspace_bytes(T, dims, ks, xd), x.device)
    d_arr, k_arr = _i32_array(dims), _i32_array(ks)
    m_arr = (c_int * L)(*[int(v) for v in alpha_modes])
    t_arr = (c_vp * L)(*[_ptr(t) for t in tiles])
    a_arr = (c_vp * L)(*[_ptr(a) for a in alphas])
    _check(lib().tbn_mlp_fwd(_ptr(x), xd, T, L, ctypes.cast(d_arr, c_vp), ctypes.cast(t_arr, c_vp),
                             ctypes.cast(k_arr, c_vp), ctypes.cast(a_arr, c_vp), ctypes.cast(m_arr, c_vp),
                             hidden_act, _ptr(y), yd, _ptr(ws), ws.numel(), _stream()), "tbn_mlp_fwd")
    return y


def tbn_last_device_status():
    code, detail = c_int(0), c_int(0)
    _check(lib().tbn_last_device_status(_stream(), ctypes.byref(code), ctypes.byref(detail)),
           "tbn_last_device_status")
    return int(code.value), int(detail.value)


def tbn_debug_record_status(code: int, detail: int):
    _check(lib().tbn_debug_record_status(code, detail, _stream()), "tbn_debug_record_status")


def tbn_debug_force_linear_config(candidate: int, splits: int = 1):
    _check(lib().tbn_debug_force_linear_config(candidate, splits), "tbn_debug_force_linear_config")


def tbn_debug_force_mlp_layerwise(on: bool):
    _check(lib().tbn_debug_force_mlp_layerwise(int(bool(on))), "tbn_debug_force_mlp_layerwise")


def tbn_row_words(n: int) -> int:
    return int(lib().tbn_row_words(n))


def tbn_binarize_fwd(x: torch.Tensor, with_beta: bool = True, x_bits: torch.Tensor | None = None,
                     beta: torch.Tensor | None = None):
    """Sign bits of the activations, packed row by row, and the per-row scale mean|x|.  Returns (x_bits, beta)."""
    T, n = x.shape
    if x_bits is None:
        x_bits = torch.empty((T, tbn_row_words(n)), dtype=torch.int32, device=x.device)
    if with_beta and beta is None:
        beta = torch.empty(T, dtype=torch.float32, device=x.device)
    _check(lib().tbn_binarize_fwd(_ptr(x), _dtype_code(x), T, n, _ptr(x_bits), _ptr(beta) if with_beta else None,
                                  _stream()), "tbn_binarize_fwd")
    return x_bits, (beta if with_beta else None)


def tbn_linear_bin_fwd(x_bits: torch.Tensor, in_f: int, out_f: int, tile: torch.Tensor, k: int, alpha: torch.Tensor,
                       alpha_mode: int, beta: torch.Tensor | None = None, bias: torch.Tensor | None = None,
                       act: int = ACT_NONE, y_dtype: int = BF16, path: int = PATH_AUTO,
                       y: torch.Tensor | None = None) -> torch.Tensor:
    T = x_bits.shape[0]
    if y is None:
        y = torch.empty((T, out_f), dtype=_torch_dtype(y_dtype), device=x_bits.device)
    _check(lib().tbn_linear_bin_fwd(_ptr(x_bits), T, in_f, out_f, _ptr(tile), k, _ptr(alpha), alpha_mode, _ptr(beta),
                                    _ptr(bias), act, _ptr(y), y_dtype, _stream(), path), "tbn_linear_bin_fwd")
    return y


def tbn_bin_expand_fwd(x_bits: torch.Tensor, in_f: int, x_bytes: torch.Tensor | None = None, x_pop: torch.Tensor | None = None):
    """Packed activation signs -> (one byte per element, 0x00 / 0xFF, in the tensor kernel's element order; row popcounts)."""
    T = x_bits.shape[0]
    if x_bytes is None:
        x_bytes = torch.empty((T, in_f), dtype=torch.uint8, device=x_bits.device)
    if x_pop is None:
        x_pop = torch.empty(T, dtype=torch.int32, device=x_bits.device)
    _check(lib().tbn_bin_expand_fwd(_ptr(x_bits), T, in_f, _ptr(x_bytes), _ptr(x_pop), _stream()), "tbn_bin_expand_fwd")
    return x_bytes, x_pop


def tbn_binarize_bytes_fwd(x: torch.Tensor):
    """Threshold, packing, row scale, sign bytes and row popcounts in one pass.  Returns (x_bits, beta, x_bytes, x_pop)."""
    T, n = x.shape
    x_bits = torch.empty((T, tbn_row_words(n)), dtype=torch.int32, device=x.device)
    beta = torch.empty(T, dtype=torch.float32, device=x.device)
    x_bytes = torch.empty((T, n), dtype=torch.uint8, device=x.device)
    x_pop = torch.empty(T, dtype=torch.int32, device=x.device)
    _check(lib().tbn_binarize_bytes_fwd(_ptr(x), _dtype_code(x), T, n, _ptr(x_bits), _ptr(beta), _ptr(x_bytes), _ptr(x_pop),
                                        _stream()), "tbn_binarize_bytes_fwd")
    return x_bits, beta, x_bytes, x_pop


def tbn_linear_bin_bytes_fwd(x_bytes: torch.Tensor, x_pop: torch.Tensor, in_f: int, out_f: int, tile: torch.Tensor, k: int,
                             alpha: torch.Tensor, alpha_mode: int, beta: torch.Tensor | None = None,
                             bias: torch.Tensor | None = None, act: int = ACT_NONE, y_dtype: int = BF16,
                             y: torch.Tensor | None = None) -> torch.Tensor:
    T = x_bytes.shape[0]
    if y is None:
        y = torch.empty((T, out_f), dtype=_torch_dtype(y_dtype), device=x_bytes.device)
    _check(lib().tbn_linear_bin_bytes_fwd(_ptr(x_bytes), _ptr(x_pop), T, in_f, out_f, _ptr(tile), k, _ptr(alpha), alpha_mode,
                                          _ptr(beta), _ptr(bias), act, _ptr(y), y_dtype, _stream()), "tbn_linear_bin_bytes_fwd")
    return y


def tbn_tile_fwd(W: torch.Tensor, k: int, alpha_mode: int = ALPHA_PER_TILE, A: torch.Tensor | None = None,
                 b_dtype: int = F32):
    """Training forward of the tiling module.  Returns (B_hat [N], tile_bits, alpha)."""
    N = W.numel()
    if k <= 0 or N % k:
        raise TbnError(-2, "tbn_tile_fwd")
    B_hat = torch.empty(N, dtype=_torch_dtype(b_dtype), device=W.device)
    tile = torch.empty(tbn_tile_words(N // k), dtype=torch.int32, device=W.device)
    alpha = torch.empty(k if alpha_mode == ALPHA_PER_TILE else 1, dtype=torch.float32, device=W.device)
    ws = _ws(lib().tbn_aggregate_workspace_bytes(N, k), W.device)
    _check(lib().tbn_tile_fwd(_ptr(W), _ptr(A), N, k, alpha_mode, _ptr(B_hat), b_dtype, _ptr(tile), _ptr(alpha), _ptr(ws),
                              ws.numel(), _stream()), "tbn_tile_fwd")
    return B_hat, tile, alpha


def tbn_tile_bwd(G: torch.Tensor, tile: torch.Tensor, alpha: torch.Tensor, W: torch.Tensor, k: int,
                 alpha_mode: int = ALPHA_PER_TILE, A: torch.Tensor | None = None):
    """Straight-through backward of the tiling module.  Returns (dW, dA or None, dalpha)."""
    N = W.numel()
    dW = torch.empty(N, dtype=torch.float32, device=W.device)
    dA = torch.empty(N, dtype=torch.float32, device=W.device) if A is not None else None
    dalpha = torch.empty(k if alpha_mode == ALPHA_PER_TILE else 1, dtype=torch.float32, device=W.device)
    ws = _ws(lib().tbn_tile_bwd_workspace_bytes(N, k), W.device)
    _check(lib().tbn_tile_bwd(_ptr(G), _ptr(tile), _ptr(alpha), _ptr(W), _ptr(A), N, k, alpha_mode, _ptr(dW), _ptr(dA),
                              _ptr(dalpha), _ptr(ws), ws.numel(), _stream()), "tbn_tile_bwd")
    return dW, dA, dalpha


def tbn_linear_res_fwd(x: torch.Tensor, out_f: int, tile: torch.Tensor, k: int, alpha: torch.Tensor, alpha_mode: int,
                       residual: torch.Tensor, bias: torch.Tensor | None = None, act: int = ACT_NONE,
                       path: int = PATH_AUTO, y: torch.Tensor | None = None, workspace: torch.Tensor | None = None):
    """y = act(layer(x)) + residual; residual has y's shape and dtype."""
    T, in_f = x.shape
    xd, yd = _dtype_code(x), _dtype_code(residual)
    if y is None:
        y = torch.empty((T, out_f), dtype=residual.dtype, device=x.device)
    ws = workspace if workspace is not None else _ws(tbn_linear_workspace_bytes(T, in_f, out_f, k, xd), x.device)
    _check(lib().tbn_linear_res_fwd(_ptr(x), xd, T, in_f, out_f, _ptr(tile), k, _ptr(alpha), alpha_mode, _ptr(bias), act,
                                    _ptr(residual), _ptr(y), yd, _ptr(ws), ws.numel(), _stream(), path), "tbn_linear_res_fwd")
    return y


def tbn_layernorm_fwd(x: torch.Tensor, gamma: torch.Tensor | None = None, beta: torch.Tensor | None = None,
                      eps: float = 1e-5, y_dtype: int | None = None) -> torch.Tensor:
    T, d = x.shape
    yd = _dtype_code(x) if y_dtype is None else y_dtype
    y = torch.empty((T, d), dtype=_torch_dtype(yd), device=x.device)
    _check(lib().tbn_layernorm_fwd(_ptr(x), _dtype_code(x), T, d, _ptr(gamma), _ptr(beta), eps, _ptr(y), yd, _stream()),
           "tbn_layernorm_fwd")
    return y


def tbn_attention_fwd(qkv: torch.Tensor, Nb: int, S: int, heads: int, d_head: int, out: torch.Tensor | None = None) -> torch.Tensor:
    if out is None:
        out = torch.empty((Nb * S, heads * d_head), dtype=torch.bfloat16, device=qkv.device)
    _check(lib().tbn_attention_fwd(_ptr(qkv), Nb, S, heads, d_head, _ptr(out), _stream()), "tbn_attention_fwd")
    return out


def tbn_vit_block_workspace_bytes(Nb, S, d, mlp_dim, ks) -> int:
    return int(lib().tbn_vit_block_workspace_bytes(Nb, S, d, mlp_dim, ctypes.cast(_i32_array(ks), c_vp)))


def tbn_vit_block_fwd(x: torch.Tensor, Nb: int, S: int, heads: int, mlp_dim: int, tiles, ks, alphas, alpha_modes,
                      workspace: torch.Tensor | None = None, y: torch.Tensor | None = None) -> torch.Tensor:
    """Pre-norm encoder block; tiles / ks / alphas / alpha_modes in the order qkv, proj, fc1, fc2."""
    T, d = x.shape
    if y is None:
        y = torch.empty_like(x)
    ws = workspace if workspace is not None else _ws(tbn_vit_block_workspace_bytes(Nb, S, d, mlp_dim, ks), x.device)
    k_arr = _i32_array(ks)
    m_arr = (c_int * 4)(*[int(v) for v in alpha_modes])
    t_arr = (c_vp * 4)(*[_ptr(t) for t in tiles])
    a_arr = (c_vp * 4)(*[_ptr(a) for a in alphas])
    _check(lib().tbn_vit_block_fwd(_ptr(x), Nb, S, d, heads, mlp_dim, ctypes.cast(t_arr, c_vp), ctypes.cast(k_arr, c_vp),
                                   ctypes.cast(a_arr, c_vp), ctypes.cast(m_arr, c_vp), _ptr(y), _ptr(ws), ws.numel(),
                                   _stream()), "tbn_vit_block_fwd")
    return y


def tbn_conv2d_dense_fwd(x: torch.Tensor, weight: torch.Tensor, stride: int, pad: int, bias=None, act=ACT_NONE,
                         y_dtype=None) -> torch.Tensor:
    """Convolution with an explicit fp32 weight (Cout, Cin, kh, kw): the untiled first layer of a stack."""
    Nb, Cin, H, Wd = x.shape
    Cout, _, kh, kw = weight.shape
    xd = _dtype_code(x)
    yd = xd if y_dtype is None else y_dtype
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (Wd + 2 * pad - kw) // stride + 1
    y = torch.empty((Nb, Cout, Ho, Wo), dtype=_torch_dtype(yd), device=x.device)
    _check(lib().tbn_conv2d_dense_fwd(_ptr(x), xd, Nb, Cin, H, Wd, Cout, kh, kw, stride, pad, _ptr(weight), _ptr(bias), act,
                                      _ptr(y), yd, _stream()), "tbn_conv2d_dense_fwd")
    return y


def tbn_global_avgpool_fwd(x: torch.Tensor, y_dtype=None) -> torch.Tensor:
    Nb, C, H, Wd = x.shape
    xd = _dtype_code(x)
    yd = xd if y_dtype is None else y_dtype
    y = torch.empty((Nb, C), dtype=_torch_dtype(yd), device=x.device)
    _check(lib().tbn_global_avgpool_fwd(_ptr(x), xd, Nb, C, H, Wd, _ptr(y), yd, _stream()), "tbn_global_avgpool_fwd")
    return y


def tbn_avgpool_linear_fwd(x: torch.Tensor, weight: torch.Tensor, bias: torch.Tensor | None = None) -> torch.Tensor:
    """Global average pooling followed by a dense fp32 classifier (weight: out_f x C) in one launch; y: Nb x out_f fp32."""
    Nb, C, H, Wd = x.shape
    out_f = weight.shape[0]
    y = torch.empty((Nb, out_f), dtype=torch.float32, device=x.device)
    _check(lib().tbn_avgpool_linear_fwd(_ptr(x), _dtype_code(x), Nb, C, H, Wd, _ptr(weight), _ptr(bias), out_f, _ptr(y),
                                        _stream()), "tbn_avgpool_linear_fwd")
    return y


def tbn_debug_set_wait_limit_us(limit_us: int):
    _check(lib().tbn_debug_set_wait_limit_us(limit_us), "tbn_debug_set_wait_limit_us")


def tbn_debug_wait_timeout_probe(detail: int):
    _check(lib().tbn_debug_wait_timeout_probe(detail, _stream()), "tbn_debug_wait_timeout_probe")


def tbn_linear_compact_fwd(z: torch.Tensor, kz: int, alpha_z: torch.Tensor, alpha_mode_z: int, act_z: int, out_f: int,
                           tile: torch.Tensor, k: int, alpha: torch.Tensor, alpha_mode: int, bias=None, act=ACT_NONE,
                           y_dtype: int = BF16, y: torch.Tensor | None = None) -> torch.Tensor:
    """Second of two tiled layers chained in compact form: z holds the first layer's distinct pre-activations
    (T x r_z, bf16); its k_z-fold output act_z(alpha_z[j] * z) is rebuilt on chip."""
    T, rz = z.shape
    if y is None:
        y = torch.empty((T, out_f), dtype=_torch_dtype(y_dtype), device=z.device)
    _check(lib().tbn_linear_compact_fwd(_ptr(z), T, rz, kz, _ptr(alpha_z), alpha_mode_z, act_z, out_f, _ptr(tile), k,
                                        _ptr(alpha), alpha_mode, _ptr(bias), act, _ptr(y), y_dtype, _stream()),
           "tbn_linear_compact_fwd")
    return y
