"""Small, self-contained runs of single kernels, sized for a profiler capture (a few hundred MB on the device, a handful
of launches):

    python -m paper_2407_12075_b200.profile_cases <case> [--reps N]

Cases: linear_k2, linear_k16 (8192 x 8192, T = 8192), bin_k2, bin_k16 (binary activations, 8192 x 8192, T = 4096),
binbytes_k2, binbytes_k16 (the same with the activation signs as bytes),
conv_s2 (64 -> 128, 32 x 32, batch 64), attention (64 images x 12 heads x 197 tokens), binarize, tile_bwd,
first_conv (dense 3 -> 64, 32 x 32, batch 256), compact_gelu (second MLP layer of a ViT-B block fed the first layer's 384 distinct pre-activations, T = 25,216).
Inputs are seeded device-side random values of the benchmark's shapes; every run checks the device status word.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case")
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)

    def rand_tile(q):
        return torch.randint(-2 ** 31, 2 ** 31 - 1, (B.tbn_tile_words(q),), device=dev, dtype=torch.int32, generator=gen)

    n = m = 8192
    if args.case in ("linear_k2", "linear_k16"):
        k, T = int(args.case.split("_k")[1]), 8192
        x = torch.randn(T, n, device=dev, generator=gen).to(torch.bfloat16)
        y = torch.empty(T, m, device=dev, dtype=torch.bfloat16)
        tile, alpha = rand_tile(n * m // k), torch.rand(k, device=dev, generator=gen) * 0.02
        ws = torch.empty(max(B.tbn_linear_workspace_bytes(T, n, m, k, B.BF16), 16), dtype=torch.uint8, device=dev)
        run = lambda: B.tbn_linear_fwd(x, m, tile, k, alpha, B.ALPHA_PER_TILE, y=y, workspace=ws)
    elif args.case in ("bin_k2", "bin_k16", "binarize", "binbytes_k2", "binbytes_k16"):
        T = 4096
        x = torch.randn(T, n, device=dev, generator=gen).to(torch.bfloat16)
        xb, beta = B.tbn_binarize_fwd(x)
        if args.case == "binarize":
            run = lambda: B.tbn_binarize_fwd(x, x_bits=xb, beta=beta)
        else:
            k = int(args.case.split("_k")[1])
            y = torch.empty(T, m, device=dev, dtype=torch.bfloat16)
            tile, alpha = rand_tile(n * m // k), torch.rand(k, device=dev, generator=gen) * 0.02
            if args.case.startswith("binbytes"):
                xbytes, xpop = B.tbn_bin_expand_fwd(xb, n)
                run = lambda: B.tbn_linear_bin_bytes_fwd(xbytes, xpop, n, m, tile, k, alpha, B.ALPHA_PER_TILE, beta=beta, y=y)
            else:
                run = lambda: B.tbn_linear_bin_fwd(xb, n, m, tile, k, alpha, B.ALPHA_PER_TILE, beta=beta, y=y)
    elif args.case == "conv_s2":
        xc = torch.rand(64, 64, 32, 32, device=dev, generator=gen).to(torch.bfloat16)
        tile, alpha = rand_tile(128 * 64 * 9 // 4), torch.rand(4, device=dev, generator=gen) * 0.05
        run = lambda: B.tbn_conv2d_fwd(xc, 128, 3, 3, 2, 1, tile, 4, alpha, B.ALPHA_PER_TILE, act=B.ACT_RELU)
    elif args.case == "attention":
        qkv = torch.randn(64 * 197, 3 * 768, device=dev, generator=gen).to(torch.bfloat16)
        run = lambda: B.tbn_attention_fwd(qkv, 64, 197, 12, 64)
    elif args.case == "compact_gelu":
        T, d, mlp, k = 128 * 197, 768, 3072, 8
        z = torch.randn(T, mlp // k, device=dev, generator=gen).to(torch.bfloat16)
        y = torch.empty(T, d, device=dev, dtype=torch.bfloat16)
        tile = rand_tile(d * mlp // k)
        a1, a2 = torch.rand(k, device=dev, generator=gen) * 0.05, torch.rand(k, device=dev, generator=gen) * 0.02
        run = lambda: B.tbn_linear_compact_fwd(z, k, a1, B.ALPHA_PER_TILE, B.ACT_GELU, d, tile, k, a2, B.ALPHA_PER_TILE, y=y)
    elif args.case == "first_conv":
        xc = torch.rand(256, 3, 32, 32, device=dev, generator=gen).to(torch.bfloat16)
        W0 = torch.randn(64, 3, 3, 3, device=dev, generator=gen) * 0.27
        run = lambda: B.tbn_conv2d_dense_fwd(xc, W0, 1, 1, act=B.ACT_RELU)
    elif args.case == "tile_bwd":
        N, k = 4096 * 4096, 4
        W = torch.randn(N, device=dev, generator=gen) * 0.02
        G = torch.randn(N, device=dev, generator=gen)
        _, tile, alpha = B.tbn_tile_fwd(W, k)
        run = lambda: B.tbn_tile_bwd(G, tile, alpha, W, k)
    else:
        raise SystemExit(f"unknown case {args.case}")
    for _ in range(args.reps):
        run()
    torch.cuda.synchronize()
    code, detail = B.tbn_last_device_status()
    if code != 0:
        raise SystemExit(f"device status {code} / {detail}")
    print("ok", args.case)


if __name__ == "__main__":
    main()
