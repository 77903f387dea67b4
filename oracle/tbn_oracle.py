"""CPU oracle for the Tiled Bit Networks forward -- TEST INFRASTRUCTURE, not the product.

Thin numpy front-end over ``tbn_oracle.c`` (plain C, fp64) plus the compositions
(MLP chain, storage accounting) that are easier to state in Python.  It shares no
code with the CUDA library and must only be used by the test-suite, the smoke
check and the benchmark's CPU-baseline leg.

Every function names the passage of the paper it restates.  Parity pins live in
``tests/test_oracle_*.py``; no function here is unpinned.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tbn_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libtbn_oracle.so")

ACT_NONE, ACT_RELU, ACT_GELU = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA, no fast-math, no FMA contraction)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    cmd = ["gcc", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
           "-o", _LIB_PATH, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.tbn_oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().tbn_oracle_num_threads())


# --------------------------------------------------------------------------- #
# exact widening of the stored activation formats                              #
# --------------------------------------------------------------------------- #
def widen(x: np.ndarray) -> np.ndarray:
    """fp32 array, or uint16 array holding bf16 bit patterns -> fp64, exactly."""
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return np.ascontiguousarray(x, dtype=np.float64)


def round_to_bf16(v: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bf16 (ties to even), returned as fp64.  Used only by the
    'mirrored' MLP mode that imitates a pipeline storing bf16 between layers."""
    f = np.ascontiguousarray(v, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)) << np.uint64(16)
    return r.astype(np.uint32).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- #
# Sec. 3: tile construction                                                    #
# --------------------------------------------------------------------------- #
def tile_words(q: int) -> int:
    """Words of the packed tile: ceil(q/32) rounded up to a multiple of 4 (128 bits)."""
    return ((int(q) + 31) // 32 + 3) // 4 * 4


def aggregate(W: np.ndarray, p: int):
    """Eq. 1-3.  Returns (bits uint8[q] in {0,1}, count of fp64 sign disagreements)."""
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(-1)
    N = W.size
    if p <= 0 or N % p:
        raise ValueError("p must divide N (Sec. 3: p*q = N)")
    bits = np.empty(N // p, dtype=np.uint8)
    mism = ctypes.c_int64(0)
    rc = _load().tbn_oracle_aggregate(_p(W), ctypes.c_int64(N), ctypes.c_int32(p), _p(bits),
                                      ctypes.byref(mism))
    assert rc == 0
    return bits, int(mism.value)


def alpha(S: np.ndarray, p: int, per_tile: bool) -> np.ndarray:
    """Eq. 6 (per layer) / Eq. 7-8 (per tile); S is W or the separate tensor A."""
    S = np.ascontiguousarray(S, dtype=np.float32).reshape(-1)
    out = np.empty(p if per_tile else 1, dtype=np.float32)
    rc = _load().tbn_oracle_alpha(_p(S), ctypes.c_int64(S.size), ctypes.c_int32(p),
                                  ctypes.c_int(1 if per_tile else 0), _p(out))
    if rc != 0:
        raise ValueError("p must divide N")
    return out


def pack(src: np.ndarray) -> np.ndarray:
    """Sec. 5.1 bit packing of a real vector: src > 0 -> 1.  LSB-first 32-bit words."""
    src = np.ascontiguousarray(src, dtype=np.float32).reshape(-1)
    words = np.empty(tile_words(src.size), dtype=np.uint32)
    _load().tbn_oracle_pack(_p(src), ctypes.c_int64(src.size), _p(words), ctypes.c_int64(words.size))
    return words


def pack_bits(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint8).reshape(-1)
    words = np.empty(tile_words(bits.size), dtype=np.uint32)
    _load().tbn_oracle_pack_bits(_p(bits), ctypes.c_int64(bits.size), _p(words),
                                 ctypes.c_int64(words.size))
    return words


def expand(words: np.ndarray, N: int, p: int, alphas: np.ndarray, per_tile: bool) -> np.ndarray:
    """Eq. 4-5 + scaling: flat B_hat (fp32, N elements)."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    alphas = np.ascontiguousarray(alphas, dtype=np.float32)
    out = np.empty(N, dtype=np.float32)
    rc = _load().tbn_oracle_expand(_p(words), ctypes.c_int64(N), ctypes.c_int32(p), _p(alphas),
                                   ctypes.c_int(1 if per_tile else 0), _p(out))
    if rc != 0:
        raise ValueError("p must divide N")
    return out


def prepare(W: np.ndarray, p: int, per_tile: bool, A: np.ndarray | None = None):
    """Whole prepare step of one layer: (packed words, alphas)."""
    bits, _ = aggregate(W, p)
    return pack_bits(bits), alpha(W if A is None else A, p, per_tile)


# --------------------------------------------------------------------------- #
# Layer forward                                                                #
# --------------------------------------------------------------------------- #
def linear_dense(x: np.ndarray, B_hat: np.ndarray, m: int, n: int, bias=None, act=ACT_NONE):
    """y = act(B_hat x + bias) with an explicit m x n weight, naive fp64."""
    xd = widen(x).reshape(-1, n)
    T = xd.shape[0]
    B_hat = np.ascontiguousarray(B_hat, dtype=np.float32).reshape(m, n)
    bd = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    y = np.empty((T, m), dtype=np.float64)
    _load().tbn_oracle_linear(_p(xd), ctypes.c_int64(T), ctypes.c_int32(n), ctypes.c_int32(m),
                              _p(B_hat), _p(bd), ctypes.c_int(act), _p(y))
    return y


def linear(x, words, p, alphas, per_tile, m, n, bias=None, act=ACT_NONE):
    """Tiled fully-connected layer: expand the tile (Eq. 4-5), then the dense product."""
    B_hat = expand(words, m * n, p, alphas, per_tile)
    return linear_dense(x, B_hat, m, n, bias, act)


def expand_fp(tile: np.ndarray, N: int, p: int) -> np.ndarray:
    """Full-precision tiled weights (Sec. 5.2, Table 7 "FP, Tiled"): B[f] = t[f mod q], flat fp32."""
    tile = np.ascontiguousarray(tile, dtype=np.float32)
    out = np.empty(N, dtype=np.float32)
    rc = _load().tbn_oracle_expand_fp(_p(tile), ctypes.c_int64(N), ctypes.c_int32(p), _p(out))
    if rc != 0:
        raise ValueError("p must divide N")
    return out


def linear_fp(x, tile, p, m, n, bias=None, act=ACT_NONE):
    """Fully-connected layer whose weight is a real-valued tile repeated p times: expand, then the dense product."""
    return linear_dense(x, expand_fp(tile, m * n, p), m, n, bias, act)


def linear_fp_alg1(x, tile, p, m, n, relu=False):
    """The index-walk form (Algorithm 1) applied to a real-valued tile, all scaling factors 1."""
    q = m * n // p
    xd = widen(x).reshape(-1, n)
    T = xd.shape[0]
    t = np.ascontiguousarray(tile, dtype=np.float32)
    ones = np.ones(p, dtype=np.float32)
    y = np.empty((T, m), dtype=np.float64)
    _load().tbn_oracle_linear_alg1(_p(xd), ctypes.c_int64(T), ctypes.c_int32(n), ctypes.c_int32(m), _p(t),
                                   ctypes.c_int64(q), _p(ones), ctypes.c_int(1 if relu else 0), _p(y))
    return y


def linear_alg1(x, words, p, alphas, per_tile, m, n, relu=False):
    """Algorithm 1: the index-walk form of the same layer."""
    q = m * n // p
    w = np.ascontiguousarray(words, dtype=np.uint32)
    idx = np.arange(q)
    tile = np.where((w[idx >> 5] >> (idx & 31).astype(np.uint32)) & 1, 1.0, -1.0).astype(np.float32)
    al = np.ascontiguousarray(alphas, dtype=np.float32)
    if not per_tile:
        al = np.full(p, al[0], dtype=np.float32)
    xd = widen(x).reshape(-1, n)
    T = xd.shape[0]
    y = np.empty((T, m), dtype=np.float64)
    _load().tbn_oracle_linear_alg1(_p(xd), ctypes.c_int64(T), ctypes.c_int32(n), ctypes.c_int32(m),
                                   _p(tile), ctypes.c_int64(q), _p(al), ctypes.c_int(int(relu)), _p(y))
    return y


# --------------------------------------------------------------------------- #
# Binary activations (Sec. 7: binary weights AND binary activations)           #
# --------------------------------------------------------------------------- #
def row_words(n: int) -> int:
    """Words of one packed activation row: ceil(n/32) rounded up to a multiple of 4 (16-byte rows)."""
    return ((int(n) + 31) // 32 + 3) // 4 * 4


def binarize(x: np.ndarray):
    """Threshold rule of Eq. 3 applied to the activations, and the per-row scale beta_t = ||x_t||_1 / n
    (Eq. 6 applied to one input row).  Returns (bits uint8 [T, n] in {0,1}, beta float32 [T])."""
    xd = widen(x)
    T, n = xd.shape
    bits = np.empty((T, n), dtype=np.uint8)
    beta = np.empty(T, dtype=np.float32)
    _load().tbn_oracle_binarize(_p(np.ascontiguousarray(xd)), ctypes.c_int64(T), ctypes.c_int32(n), _p(bits), _p(beta))
    return bits, beta


def pack_rows(bits: np.ndarray) -> np.ndarray:
    """[T, n] bits -> [T, row_words(n)] uint32, each row packed like a tile (LSB first, zero padding)."""
    T, n = bits.shape
    out = np.zeros((T, row_words(n)), dtype=np.uint32)
    for t in range(T):
        out[t, :tile_words(n)][: (n + 31) // 32] = pack_bits(bits[t])[: (n + 31) // 32]
    return out


def linear_bin_int(abits: np.ndarray, words: np.ndarray, p: int, m: int, n: int) -> np.ndarray:
    """D[t][i] = sum_j b[i][j] a[t][j] over +-1 values: the integer accumulator of the binary-activation layer."""
    abits = np.ascontiguousarray(abits, dtype=np.uint8)
    T = abits.shape[0]
    words = np.ascontiguousarray(words, dtype=np.uint32)
    D = np.empty((T, m), dtype=np.int64)
    _load().tbn_oracle_linear_bin_int(_p(abits), ctypes.c_int64(T), ctypes.c_int32(n), ctypes.c_int32(m), _p(words),
                                      ctypes.c_int64(m * n // p), _p(D))
    return D


def linear_bin(abits, beta, words, p, alphas, per_tile, m, n, bias=None, act=ACT_NONE):
    """y[t][i] = act(beta_t * sum_j B_hat[i][j] a[t][j] + bias[i]): the tiled layer of Eq. 4-8 applied to the
    sign vector of the activations, each row scaled by its beta -- i.e. the dense layer on the inputs beta_t * (+-1)."""
    a_pm = np.where(np.asarray(abits) > 0, 1.0, -1.0)
    if beta is not None:
        a_pm = a_pm * np.asarray(beta, dtype=np.float64)[:, None]      # exact: beta_t * (+-1)
    return linear(a_pm, words, p, alphas, per_tile, m, n, bias=bias, act=act)


def conv_out_hw(H, Wd, kh, kw, stride, pad):
    return (H + 2 * pad - kh) // stride + 1, (Wd + 2 * pad - kw) // stride + 1


def conv2d_dense(x, B_hat, Cout, Cin, kh, kw, stride, pad, bias=None, act=ACT_NONE):
    xd = widen(x)
    Nb, C, H, Wd = xd.shape
    assert C == Cin
    xd = np.ascontiguousarray(xd)
    B_hat = np.ascontiguousarray(B_hat, dtype=np.float32).reshape(-1)
    bd = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    Ho, Wo = conv_out_hw(H, Wd, kh, kw, stride, pad)
    y = np.empty((Nb, Cout, Ho, Wo), dtype=np.float64)
    _load().tbn_oracle_conv2d(_p(xd), ctypes.c_int32(Nb), ctypes.c_int32(Cin), ctypes.c_int32(H),
                              ctypes.c_int32(Wd), ctypes.c_int32(Cout), ctypes.c_int32(kh),
                              ctypes.c_int32(kw), ctypes.c_int32(stride), ctypes.c_int32(pad),
                              _p(B_hat), _p(bd), ctypes.c_int(act), _p(y))
    return y


def conv2d(x, words, p, alphas, per_tile, Cout, Cin, kh, kw, stride, pad, bias=None, act=ACT_NONE):
    """Tiled convolution: the tile fills the (Cout,Cin,kh,kw) tensor in row-major order."""
    B_hat = expand(words, Cout * Cin * kh * kw, p, alphas, per_tile)
    return conv2d_dense(x, B_hat, Cout, Cin, kh, kw, stride, pad, bias, act)


def conv_stack(x, W0, convs, Wfc):
    """ResNet-style stack with full-precision ends (Sec. 3: layers below the size threshold are not tiled):
    dense 3x3 convolution W0 (stride 1, padding 1) -> ReLU -> tiled 3x3 convolutions (each a dict words, p, alphas, per_tile,
    Cout, Cin, stride; padding 1) with ReLU -> global average pooling -> dense classifier Wfc [classes, C].  fp64."""
    W0 = np.asarray(W0, dtype=np.float32)
    h = conv2d_dense(x, W0, W0.shape[0], W0.shape[1], W0.shape[2], W0.shape[3], 1, 1, act=ACT_RELU)
    for c in convs:
        h = conv2d(h, c["words"], c["p"], c["alphas"], c["per_tile"], c["Cout"], c["Cin"], 3, 3, c["stride"], 1, act=ACT_RELU)
    pooled = h.mean(axis=(2, 3))
    Wfc = np.asarray(Wfc, dtype=np.float32)
    return linear_dense(pooled, Wfc, Wfc.shape[0], Wfc.shape[1])


def mlp(x, layers, hidden_act=ACT_RELU, mirror_bf16=False):
    """Chain of tiled fully-connected layers (Sec. 5.1's MLP with fused ReLU).

    layers: list of dicts(words, p, alphas, per_tile, m, n).  The hidden activation
    follows every layer but the last.  Strict mode keeps fp64 between layers;
    mirror_bf16 rounds each hidden tensor to bf16 (diagnostic only).
    """
    h = widen(x)
    for li, L in enumerate(layers):
        last = li == len(layers) - 1
        h = linear(h, L["words"], L["p"], L["alphas"], L["per_tile"], L["m"], L["n"],
                   act=ACT_NONE if last else hidden_act)
        if mirror_bf16 and not last:
            h = round_to_bf16(h)
    return h


# --------------------------------------------------------------------------- #
# Transformer encoder block with tiled linears (Sec. 4.3 trains Vision            #
# Transformers whose Q, K, V, projection and feed-forward layers are tiled;    #
# Sec. 5.2 profiles the kernel inside one).  The glue is the standard pre-norm  #
# block; none of it is specific to the paper.                                   #
# --------------------------------------------------------------------------- #
def layernorm(x: np.ndarray, gamma=None, beta=None, eps: float = 1e-5) -> np.ndarray:
    """Row-wise (v - mean) / sqrt(var + eps) with the biased variance, optional affine; fp64."""
    v = widen(x)
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    y = (v - mu) / np.sqrt(var + eps)
    if gamma is not None:
        y = y * np.asarray(gamma, dtype=np.float64)
    if beta is not None:
        y = y + np.asarray(beta, dtype=np.float64)
    return y


def attention(qkv: np.ndarray, Nb: int, S: int, heads: int, d_head: int) -> np.ndarray:
    """Multi-head softmax attention.  qkv: [Nb*S, 3*heads*d_head] with columns (q | k | v), head h at
    h*d_head inside each third.  out[b, s, h*d_head + e] = sum_t softmax_t(q_s . k_t / sqrt(d_head)) v_t[e]; fp64."""
    v = widen(qkv).reshape(Nb, S, 3, heads, d_head)
    out = np.empty((Nb, S, heads, d_head))
    for b in range(Nb):
        for h in range(heads):
            q, k, val = v[b, :, 0, h, :], v[b, :, 1, h, :], v[b, :, 2, h, :]
            sc = (q @ k.T) / np.sqrt(float(d_head))
            sc = sc - sc.max(axis=1, keepdims=True)
            pr = np.exp(sc)
            pr = pr / pr.sum(axis=1, keepdims=True)
            out[b, :, h, :] = pr @ val
    return out.reshape(Nb * S, heads * d_head)


def vit_block(x: np.ndarray, Nb: int, S: int, heads: int, layers: dict, mirror_bf16: bool = False) -> np.ndarray:
    """Pre-norm encoder block: x1 = x + proj(attn(qkv(LN(x)))); y = x1 + fc2(gelu(fc1(LN(x1)))).
    layers: dict with keys qkv, proj, fc1, fc2, each dict(words, p, alphas, per_tile, m, n).  LayerNorm without affine
    parameters, eps 1e-5; GELU in its erf form.  Strict mode keeps fp64 throughout; mirror_bf16 rounds every tensor a
    bf16 pipeline would store (diagnostic)."""
    rnd = round_to_bf16 if mirror_bf16 else (lambda v: v)

    def lin(h, name, act=ACT_NONE):
        L = layers[name]
        return linear(h, L["words"], L["p"], L["alphas"], L["per_tile"], L["m"], L["n"], act=act)

    x0 = widen(x)
    d = x0.shape[1]
    h1 = rnd(layernorm(x0))
    qkv = rnd(lin(h1, "qkv"))
    a = rnd(attention(qkv, Nb, S, heads, d // heads))
    x1 = rnd(x0 + lin(a, "proj"))
    h2 = rnd(layernorm(x1))
    f = rnd(lin(h2, "fc1", ACT_GELU))
    return x1 + lin(f, "fc2")


# --------------------------------------------------------------------------- #
# Training-side tiling module (Sec. 3: Eq. 1-5 in the forward of a custom       #
# differentiation module, gradients passed straight through on the way back)   #
# --------------------------------------------------------------------------- #
def tile_fwd(W: np.ndarray, p: int, per_tile: bool, A: np.ndarray | None = None):
    """Training forward of the tiling module: W (and A) -> the scaled tiled weight B_hat the layer then uses
    (Eq. 1-5, then Eq. 6 / Eq. 7-8 and the scaling paragraph).  Returns (B_hat fp32 [N], packed tile, alphas)."""
    words, al = prepare(W, p, per_tile, A)
    return expand(words, np.asarray(W).size, p, al, per_tile), words, al


def tile_bwd(G: np.ndarray, words: np.ndarray, alphas: np.ndarray, per_tile: bool, W: np.ndarray, p: int,
             A: np.ndarray | None = None):
    """Backward of the tiling module for G = dL/dB_hat (fp64 arithmetic).

    Eq. 1-5 are not differentiable; the paper passes the gradient with respect to B straight through to W
    (the straight-through paragraph of Sec. 3):  dL/dW := dL/dB.  B_hat = alpha_j * B, so dL/dB = alpha_j * G.
    The scaling factors are ordinary differentiable functions of S (= A, or W when no separate tensor is used):
    alpha_j = sum_{f in segment j} |S[f]| / q (Eq. 8; one segment of N values for Eq. 6), hence
        dL/dalpha_j = sum_{f in segment j} G[f] * B[f],      dL/dS[f] = dL/dalpha_{j(f)} * sign(S[f]) / q
    with sign(0) = 0.  Without a separate A both contributions land on W.
    Returns (dW [N], dA [N] or None, dalpha [1 or p])."""
    G = np.asarray(G, dtype=np.float64).reshape(-1)
    N = G.size
    q = N // p
    i = np.arange(q)
    t = np.where((np.asarray(words, dtype=np.uint32)[i >> 5] >> (i & 31).astype(np.uint32)) & 1, 1.0, -1.0)
    al = np.asarray(alphas, dtype=np.float64)
    dW = np.empty(N)
    dalpha = np.zeros(p if per_tile else 1)
    for j in range(p):
        seg = slice(j * q, (j + 1) * q)
        dW[seg] = (al[j] if per_tile else al[0]) * G[seg]
        dalpha[j if per_tile else 0] += float(np.sum(G[seg] * t))
    S = np.asarray(W if A is None else A, dtype=np.float64).reshape(-1)
    dS = np.empty(N)
    for j in range(p):
        seg = slice(j * q, (j + 1) * q)
        dS[seg] = (dalpha[j] / q if per_tile else dalpha[0] / N) * np.sign(S[seg])
    if A is None:
        return dW + dS, None, dalpha
    return dW, dS, dalpha


# --------------------------------------------------------------------------- #
# Storage accounting (Sec. 5.1 Table 6, Sec. 5.2 Table 7)                      #
# --------------------------------------------------------------------------- #
def layer_storage_bytes(N: int, p: int, n_alpha: int) -> float:
    """Bytes saved for one layer: q = N/p bits plus fp32 scalars (end of Sec. 3)."""
    return (N // p) / 8.0 + 4.0 * n_alpha


def mcu_mlp_accounting(n_in=784, hidden=128, n_out=10, p=4):
    """Table 6's storage and max-memory figures for the MNIST MLP, in bytes.

    The untiled classifier (below the size threshold lambda) is a 1-bit layer;
    the binary-weight model's figures count weight bits only, the tiled model's
    add its fp32 scalars; activations are fp32; max memory is reached in layer 1.
    """
    n1, n2 = n_in * hidden, hidden * n_out
    act_bytes = 4 * n_in + 4 * hidden
    bwnn_storage = (n1 + n2) / 8.0
    bwnn_memory = n1 / 8.0 + act_bytes
    tbn_storage = layer_storage_bytes(n1, p, p) + layer_storage_bytes(n2, 1, 1)
    tbn_memory = n1 / p / 8.0 + 4 * p + act_bytes
    return dict(bwnn_storage=bwnn_storage, bwnn_memory=bwnn_memory,
                tbn_storage=tbn_storage, tbn_memory=tbn_memory)
