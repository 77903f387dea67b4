#!/usr/bin/env python
"""Benchmark of the tiled-layer forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--tokens T]

Workload (default): the large fully-connected sweep at its largest batch -- in = out = 8192,
T = 16384 bf16 tokens ~N(0,1), W ~N(0, 0.02^2) aggregated to a tile, per-tile alpha, seed 4.
One step = one forward for each k in {2, 4, 8, 16} on the same activations (4 kernel launches).
The activation and output tensors (268 MB each) are larger than L2, so nothing is cache-resident
from one launch to the next.  Metric: algorithmic TFLOP/s = sum_k 2*T*(8192/k)*8192 / time, i.e. the
flops of the distinct rows only (the k-fold replication is a store, not a contraction).

With --gpus N > 1 (under torchrun) every rank runs the same workload on its own GPU: the path has
no exchange step, so ranks are independent replicas and the value is the sum over ranks.

--impl reference times the CPU oracle (plain C, fp64, never tuned) on a bounded sample of the same
workload, on the host cores of the machine.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N_FEAT = 8192
KS = (2, 4, 8, 16)
SEED = 4
METRIC = "tbn_layer_fwd_algorithmic_tflops"
UNIT = "TFLOP/s"


def algorithmic_flops(T: int, k: int) -> float:
    """2*T*r*n with r = out/k distinct rows (tile spans whole rows for every k here)."""
    return 2.0 * T * (N_FEAT // k) * N_FEAT


def algorithmic_bytes(T: int, k: int) -> float:
    """activations in + outputs out (bf16) + packed tile + alphas."""
    return 2.0 * T * N_FEAT * 2 + (N_FEAT * N_FEAT // k) / 8 + 4 * k


# DRAM traffic of the dominant launch (k = 2) from an ncu capture of that kernel at T = 8192 (dram bytes read +
# written: 235.9 MB); traffic is proportional to T.  The figure is only valid for the kernel source it was taken
# from: the hash below covers the code (comments stripped) of tc_linear.cu and tc_common.cuh.
TRAFFIC_BYTES_AT_T8192 = 138.699520e6 + 97.207040e6
TRAFFIC_SOURCE_HASH = "142aa7ff97fc3d03"


def kernel_source_hash() -> str:
    """Hash of the linear kernel's code with comments and blank space removed (a reworded comment is not a new kernel)."""
    import hashlib
    import re
    h = hashlib.sha256()
    for f in ("tc_linear.cu", "tc_common.cuh"):
        with open(os.path.join(ROOT, "paper_2407_12075_b200", "csrc", f), "r") as fh:
            code = re.sub(r"/\*.*?\*/", "", fh.read(), flags=re.S)
        code = re.sub(r"//[^\n]*", "", code)
        h.update(re.sub(r"\s+", " ", code).encode())
    return h.hexdigest()[:16]


def measured_traffic(T: int):
    if kernel_source_hash() != TRAFFIC_SOURCE_HASH:
        return None                      # the kernel changed since the counters were taken
    return TRAFFIC_BYTES_AT_T8192 * T / 8192.0


def max_over_ranks(value: float, device=None) -> float:
    """Multi-rank timing rule: every rank times its own replica on its own device, the job's time is the
    maximum over ranks.  A no-op without an initialised process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


BURST_LIMIT_MS = 100.0


def tensor_peak_for(region_ms: float, peaks: dict, sm_mhz=None, sm_max_mhz=None):
    """The bf16 GEMM peak that applies to a timed region.  The burst figure was taken over a few milliseconds at
    boost clocks, the sustained one over seconds under the power cap; the cap pulls the clocks down within some
    tens of milliseconds.  So: a region shorter than 100 ms is a burst; a longer one is sustained unless the clocks
    sampled during it stayed within 5 % of the maximum (the part never throttled).  Returns (peak, label)."""
    if region_ms < BURST_LIMIT_MS:
        return peaks["bf16_tflops"], "burst"
    if sm_mhz and sm_max_mhz and sm_mhz >= 0.95 * sm_max_mhz:
        return peaks["bf16_tflops"], "burst"
    return peaks["bf16_tflops_sustained"], "sustained"


def whole_job_value(flops_per_rank_step: float, world: int, ms_per_step: float) -> float:
    """Aggregate algorithmic TFLOP/s of `world` independent replicas (weak scaling)."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def wait_first(self, limit_s: float = 8.0):
        """nvidia-smi can take seconds to produce its first line on a fresh box: wait for it before timing."""
        t0 = time.time()
        while self.proc is not None and not self.rows and time.time() - t0 < limit_s:
            time.sleep(0.05)

    def mark(self):
        """Rows from here on belong to the timed region."""
        self.first = len(self.rows)

    def count(self) -> int:
        return len(self.rows) - getattr(self, "first", 0)

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[getattr(self, "first", 0):]:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def workload_config(T: int) -> dict:
    """The `config` object of the JSON line; both arms print the same one."""
    return dict(workload=f"large linear sweep 8192x8192, T={T}, k in {list(KS)}, per-tile alpha, seed {SEED}",
                step=f"one forward per k ({len(KS)} launches)", l2="inputs larger than L2 (x and y 268 MB each)",
                multi_gpu="replicas only (no exchange step in the path)")


def oracle_sample(x_bits: np.ndarray, W: np.ndarray, k: int, rows: int, seed: int = 0):
    """Time the CPU oracle (expand the tile, naive fp64 product) on `rows` seeded token rows."""
    from oracle import tbn_oracle as O
    T = x_bits.shape[0]
    pick = np.sort(np.random.default_rng(seed).choice(T, size=min(rows, T), replace=False))
    words, al = O.prepare(W, k, True)
    xs = np.ascontiguousarray(x_bits[pick])
    t0 = time.perf_counter()
    ref = O.linear(xs, words, k, al, True, N_FEAT, N_FEAT)
    dt = time.perf_counter() - t0
    return dt, len(pick), O.num_threads(), pick, ref


def run_reference(args, T: int):
    """--impl reference: the oracle as it stands, on the host cores, on a bounded sample per step."""
    from paper_2407_12075_b200 import synth
    W = synth.normal(SEED, 1, N_FEAT * N_FEAT, 0.02).reshape(N_FEAT, N_FEAT)
    # Tiles are prepared once (not part of a step).  The oracle's layer call has a large fixed cost (it expands the tile to
    # the dense weight matrix), so the sample of a step is bounded in two ways: at most 64 token rows, and -- when all steps
    # with all four k would take more than about two minutes -- one k per step, taken in turn.
    from oracle import tbn_oracle as O
    prepared = {k: O.prepare(W, k, True) for k in KS}
    rows = 64
    x = synth.to_bf16_bits(synth.normal(SEED, 0, rows * N_FEAT).reshape(rows, N_FEAT))

    def layer_seconds(k):
        words, al = prepared[k]
        t0 = time.perf_counter()
        O.linear(x, words, k, al, True, N_FEAT, N_FEAT)
        return time.perf_counter() - t0

    probe = sum(layer_seconds(k) for k in KS)                 # untimed: decides the sampling
    n_steps = args.warmup + args.steps
    rotate = n_steps * probe > 120.0
    cores = O.num_threads()
    t_sum, f_sum = 0.0, 0.0
    for step in range(n_steps):
        ks = (KS[step % len(KS)],) if rotate else KS
        t = sum(layer_seconds(k) for k in ks)
        if step >= args.warmup:
            t_sum += t
            f_sum += sum(algorithmic_flops(rows, k) for k in ks)
    ms = 1e3 * t_sum / max(args.steps, 1)
    value = f_sum / max(t_sum, 1e-12) / 1e12
    sample = (f"{rows} of {T} token rows x all 8192 outputs, " + (f"one k of {list(KS)} per step in turn" if rotate else f"each k in {list(KS)}") +
              "; dense fp64 product (the oracle never uses the replicated-row shortcut); value counts algorithmic flops")
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic", impl="reference",
                config=workload_config(T),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tokens", type=int, default=16384, help="development override of the batch size")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true")
    ap.add_argument("--ks", default="", help="development override: comma-separated subset of k values")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.ks:
        global KS
        KS = tuple(int(v) for v in args.ks.split(","))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, args.tokens)
        return

    run_ours(args, rank, world, local_rank)



def measure_other_configs(B, torch, dev, peaks):
    """Device-time measurements of the other benchmark configurations (context for the headline line):
    the small single layer, the 3-layer MLP, the tiled 3x3 convolutions, the ViT-B block's four tiled
    linears and the small-batch end of the large linear sweep.  Inputs are seeded device-side normals /
    uniforms of the configured shapes (timing does not depend on the values; parity on the seeded inputs
    of each configuration is covered by the test-suite).  Each entry is the mean over CUDA-graph replays, so
    the host's launch latency is excluded; 'l2' says whether the operands stay L2-resident between replays."""
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234)
    hbm = peaks["hbm_gbs"] * 1e9
    tens = peaks["bf16_tflops"] * 1e12          # every entry is a burst of a few milliseconds: the burst peak applies

    def graph_us(fn, reps=10, iters=5):
        fn()
        torch.cuda.synchronize()
        stream = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                fn()
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (iters * reps)

    def rand_tile(q):
        return torch.randint(-2 ** 31, 2 ** 31 - 1, (B.tbn_tile_words(q),), device=dev, dtype=torch.int32, generator=gen)

    def linear_entry(T, n, m, k, x_dtype=torch.bfloat16, act=B.ACT_NONE):
        x = torch.randn(T, n, device=dev, generator=gen).to(x_dtype)
        y = torch.empty(T, m, device=dev, dtype=x_dtype)
        tile, alpha = rand_tile(n * m // k), torch.rand(k, device=dev, generator=gen) * 0.02
        xd = B.BF16 if x_dtype == torch.bfloat16 else B.F32
        ws = torch.empty(max(B.tbn_linear_workspace_bytes(T, n, m, k, xd), 16), dtype=torch.uint8, device=dev)
        us = graph_us(lambda: B.tbn_linear_fwd(x, m, tile, k, alpha, B.ALPHA_PER_TILE, act=act, y=y, workspace=ws))
        r = m // k
        flops, nbytes = 2.0 * T * r * n, (T * n + T * m) * x.element_size() + n * m // k / 8 + 4 * k
        bound_us = max(flops / tens, nbytes / hbm) * 1e6
        return dict(us=us, path=B.tbn_linear_select_path(T, n, m, k, xd), alg_tflops=flops / us / 1e6,
                    alg_gbs=nbytes / us / 1e3, bound="tensor" if flops / tens > nbytes / hbm else "hbm",
                    frac_of_binding_roofline=bound_us / us, l2="resident" if nbytes < 100e6 else "exceeds L2")

    out = {}
    out["single_fc_512x512_k4_T64_f32"] = linear_entry(64, 512, 512, 4, torch.float32)
    T, dims, ks = 4096, [1024, 2048, 2048, 10], [8, 8, 1]
    x = torch.randn(T, dims[0], device=dev, generator=gen).to(torch.bfloat16)
    tiles = [rand_tile(dims[l] * dims[l + 1] // ks[l]) for l in range(3)]
    alphas = [torch.rand(ks[l], device=dev, generator=gen) * 0.02 for l in range(3)]
    ws = torch.empty(B.tbn_mlp_workspace_bytes(T, dims, ks, B.BF16), dtype=torch.uint8, device=dev)
    y = torch.empty(T, dims[-1], device=dev, dtype=torch.bfloat16)
    us = graph_us(lambda: B.tbn_mlp_fwd(x, dims, tiles, ks, alphas, [1, 1, 1], workspace=ws, y=y))
    out["mlp_1024_2048_2048_10_T4096"] = dict(us=us, samples_per_s=T / us * 1e6, variant="compact chain (distinct hidden columns only, folded rows)",
                                              bound_us_compact_hbm=16.6e6 / hbm * 1e6)
    for name, (Cin, H, Cout, stride) in {"conv_64_128_s2_32x32": (64, 32, 128, 2), "conv_128_256_s2_16x16": (128, 16, 256, 2),
                                         "conv_64_128_s1_32x32": (64, 32, 128, 1)}.items():
        xc = torch.rand(256, Cin, H, H, device=dev, generator=gen).to(torch.bfloat16)
        tile, alpha = rand_tile(Cout * Cin * 9 // 4), torch.rand(4, device=dev, generator=gen) * 0.05
        us = graph_us(lambda: B.tbn_conv2d_fwd(xc, Cout, 3, 3, stride, 1, tile, 4, alpha, B.ALPHA_PER_TILE, act=B.ACT_RELU),
                      reps=3, iters=3)
        Ho = (H + 2 - 3) // stride + 1
        nbytes = xc.numel() * 2 + 256 * Cout * Ho * Ho * 2
        out[name] = dict(us=us, alg_gbs=nbytes / us / 1e3, images_per_s=256 / us * 1e6, bound="hbm",
                         frac_of_binding_roofline=nbytes / hbm * 1e6 / us)
    for name, (n, m) in {"vit_qkv_768_2304": (768, 2304), "vit_out_768_768": (768, 768), "vit_fc1_768_3072": (768, 3072),
                         "vit_fc2_3072_768": (3072, 768)}.items():
        out[name] = linear_entry(25216, n, m, 8)
    out["vit_fc1_768_3072_gelu"] = linear_entry(25216, 768, 3072, 8, act=B.ACT_GELU)
    # the whole ViT-B shaped encoder block (LayerNorm, tiled qkv, attention, tiled projection + residual, LayerNorm,
    # tiled fc1 + GELU, tiled fc2 + residual) and the whole convolution stack (full-precision first convolution, two
    # tiled stride-2 convolutions, global average pooling, full-precision classifier), each run as one chain
    Nb, S, d, heads, mlp, bks = 128, 197, 768, 12, 3072, [8, 8, 8, 8]
    xb_ = torch.randn(Nb * S, d, device=dev, generator=gen).to(torch.bfloat16)
    shapes = [(3 * d, d), (d, d), (mlp, d), (d, mlp)]
    btiles = [rand_tile(m_ * n_ // 8) for (m_, n_) in shapes]
    balphas = [torch.rand(8, device=dev, generator=gen) * 0.03 for _ in shapes]
    bws = torch.empty(B.tbn_vit_block_workspace_bytes(Nb, S, d, mlp, bks), dtype=torch.uint8, device=dev)
    by = torch.empty_like(xb_)
    us = graph_us(lambda: B.tbn_vit_block_fwd(xb_, Nb, S, heads, mlp, btiles, bks, balphas, [1, 1, 1, 1], workspace=bws, y=by),
                  reps=3, iters=3)
    out["vit_block_whole_T25216"] = dict(us=us, images_per_s=Nb / us * 1e6, launches=7,
                                         includes="LN + qkv + attention + proj(+res) + LN + fc1(GELU) + fc2(+res)")
    qkv_ = torch.randn(Nb * S, 3 * d, device=dev, generator=gen).to(torch.bfloat16)
    us = graph_us(lambda: B.tbn_attention_fwd(qkv_, Nb, S, heads, 64), reps=3, iters=3)
    out["vit_attention_only"] = dict(us=us, dense_tflops=4.0 * Nb * heads * S * S * 64 / us / 1e6, note="tcgen05 kernel; glue of the block, not a tiled layer")
    us = graph_us(lambda: B.tbn_layernorm_fwd(xb_), reps=3, iters=3)
    out["vit_layernorm_only"] = dict(us=us, alg_gbs=2.0 * xb_.numel() * 2 / us / 1e3)
    # the block's MLP with the first layer in compact form (its 384 distinct pre-activations only) and the second layer
    # rebuilding gelu(alpha_j z) on chip, against the full form timed above (fc1 with GELU + fc2)
    zc = torch.empty(Nb * S, mlp // 8, device=dev, dtype=torch.bfloat16)
    one = torch.ones(1, device=dev)
    us1 = graph_us(lambda: B.tbn_linear_fwd(xb_, mlp // 8, btiles[2], 1, one, B.ALPHA_PER_LAYER, y=zc), reps=3, iters=3)
    us2 = graph_us(lambda: B.tbn_linear_compact_fwd(zc, 8, balphas[2], B.ALPHA_PER_TILE, B.ACT_GELU, d, btiles[3], 8, balphas[3],
                                                    B.ALPHA_PER_TILE, y=by), reps=3, iters=3)
    out["vit_mlp_compact_gelu_chain"] = dict(us=us1 + us2, first_layer_us=us1, second_layer_us=us2,
                                             full_form_us=out["vit_fc1_768_3072_gelu"]["us"] + out["vit_fc2_3072_768"]["us"],
                                             note="measured slower than the full form, which the block therefore uses")
    del bws, qkv_, by, xb_, zc
    xc0 = torch.rand(256, 3, 32, 32, device=dev, generator=gen).to(torch.bfloat16)
    W0 = torch.randn(64, 3, 3, 3, device=dev, generator=gen) * 0.27
    ct1, ca1 = rand_tile(128 * 64 * 9 // 4), torch.rand(4, device=dev, generator=gen) * 0.05
    ct2, ca2 = rand_tile(256 * 128 * 9 // 4), torch.rand(4, device=dev, generator=gen) * 0.03
    Wfc = torch.randn(10 * 256, device=dev, generator=gen) * 0.06

    def stack():
        h = B.tbn_conv2d_dense_fwd(xc0, W0, 1, 1, act=B.ACT_RELU)
        h = B.tbn_conv2d_fwd(h, 128, 3, 3, 2, 1, ct1, 4, ca1, B.ALPHA_PER_TILE, act=B.ACT_RELU)
        h = B.tbn_conv2d_fwd(h, 256, 3, 3, 2, 1, ct2, 4, ca2, B.ALPHA_PER_TILE, act=B.ACT_RELU)
        return B.tbn_avgpool_linear_fwd(h, Wfc2d)

    Wfc2d = Wfc.reshape(10, 256)
    us = graph_us(stack, reps=3, iters=3)
    out["conv_stack_whole_batch256"] = dict(us=us, images_per_s=256 / us * 1e6, launches=4,
                                            includes="dense conv 3->64 + tiled 64->128 s2 + tiled 128->256 s2 + (avg pool + dense classifier)")
    us = graph_us(lambda: B.tbn_conv2d_dense_fwd(xc0, W0, 1, 1, act=B.ACT_RELU), reps=3, iters=3)
    out["conv_first_dense_3_64"] = dict(us=us, alg_gbs=(xc0.numel() * 2 + 256 * 64 * 1024 * 2) / us / 1e3, bound="hbm",
                                        frac_of_binding_roofline=(xc0.numel() * 2 + 256 * 64 * 1024 * 2) / hbm * 1e6 / us)
    # derived: images/s over the tiled layers only (LayerNorm, attention and residual adds of the block, and the
    # full-precision first convolution / classifier of the conv stack, are not tiled layers and are not run)
    vit_us = sum(out[n]["us"] for n in ("vit_qkv_768_2304", "vit_out_768_768", "vit_fc1_768_3072_gelu", "vit_fc2_3072_768"))
    out["vit_block_tiled_linears_only"] = dict(us=vit_us, images_per_s=128 / vit_us * 1e6, includes="qkv + out-proj + fc1 with fused GELU + fc2")
    conv_us = out["conv_64_128_s2_32x32"]["us"] + out["conv_128_256_s2_16x16"]["us"]
    out["conv_stack_tiled_convs_only"] = dict(us=conv_us, images_per_s=256 / conv_us * 1e6, includes="64->128 s2 + 128->256 s2")
    # prepare step (once per layer, outside the forward): W fp32 read once, packed tile written
    Wagg = torch.randn(N_FEAT * N_FEAT, device=dev, generator=gen) * 0.02
    for k in (2, 16):
        us = graph_us(lambda: B.tbn_aggregate_tile(Wagg, k, B.ALPHA_PER_TILE), reps=3, iters=3)
        nbytes = 4.0 * Wagg.numel() + Wagg.numel() / k / 8
        out[f"aggregate_8192x8192_k{k}"] = dict(us=us, alg_gbs=nbytes / us / 1e3, bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us)
    # training-side tiling module (Sec. 3): forward = one read of W + one write of B_hat; backward = G read twice, W read
    # once (sign for the alpha path), dW written once
    for k in (4,):
        us = graph_us(lambda: B.tbn_tile_fwd(Wagg, k, B.ALPHA_PER_TILE), reps=3, iters=3)
        nbytes = 8.0 * Wagg.numel() + Wagg.numel() / k / 8
        out[f"tile_fwd_8192x8192_k{k}"] = dict(us=us, alg_gbs=nbytes / us / 1e3, bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us)
        _, t_bits, t_alpha = B.tbn_tile_fwd(Wagg, k, B.ALPHA_PER_TILE)
        Gagg = torch.randn(Wagg.numel(), device=dev, generator=gen)
        us = graph_us(lambda: B.tbn_tile_bwd(Gagg, t_bits, t_alpha, Wagg, k, B.ALPHA_PER_TILE), reps=3, iters=3)
        nbytes = 16.0 * Wagg.numel()
        out[f"tile_bwd_8192x8192_k{k}"] = dict(us=us, alg_gbs=nbytes / us / 1e3, bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us)
        del Gagg
    del Wagg
    # full-precision tiled weights (Sec. 5.2): ViT fc1-shaped layer, k = 4, bf16 tile read in place
    T, n, m, k = 25216, 768, 3072, 4
    x = torch.randn(T, n, device=dev, generator=gen).to(torch.bfloat16)
    y = torch.empty(T, m, device=dev, dtype=torch.bfloat16)
    tv = (torch.randn(n * m // k, device=dev, generator=gen) * 0.02).to(torch.bfloat16)
    ws = torch.empty(max(B.tbn_linear_fp_tile_workspace_bytes(T, n, m, k, B.BF16, B.BF16), 16), dtype=torch.uint8, device=dev)
    us = graph_us(lambda: B.tbn_linear_fp_tile_fwd(x, m, tv, k, act=B.ACT_GELU, y=y, workspace=ws))
    flops, nbytes = 2.0 * T * (m // k) * n, (T * n + T * m) * 2 + tv.numel() * 2
    out["fp_tile_vit_fc1_768_3072_k4"] = dict(us=us, alg_tflops=flops / us / 1e6, alg_gbs=nbytes / us / 1e3,
                                              bound="tensor" if flops / tens > nbytes / hbm else "hbm",
                                              frac_of_binding_roofline=max(flops / tens, nbytes / hbm) * 1e6 / us)
    for T in (1, 16, 256, 4096):
        for k in (2, 16):
            out[f"large_linear_T{T}_k{k}"] = linear_entry(T, N_FEAT, N_FEAT, k)
    # binary activations (Sec. 7): threshold + packing, then the XNOR / popcount layer on the sweep's shape.  Integer
    # ops = 2*T*r*n.  Large batches run on the 8-bit integer tensor cores (peak taken as twice the measured bf16 burst
    # peak, the nominal ratio); the popcount rate of the CUDA cores (16 popcounts of 32 bits per clock and SM) is
    # quoted beside it as the bound a popcount kernel would have.
    T = 16384
    x = torch.randn(T, N_FEAT, device=dev, generator=gen).to(torch.bfloat16)
    xb = torch.empty((T, B.tbn_row_words(N_FEAT)), dtype=torch.int32, device=dev)
    beta = torch.empty(T, dtype=torch.float32, device=dev)
    us = graph_us(lambda: B.tbn_binarize_fwd(x, x_bits=xb, beta=beta), reps=3, iters=3)
    nbytes = x.numel() * 2 + xb.numel() * 4 + T * 4
    out["binarize_T16384_8192"] = dict(us=us, alg_gbs=nbytes / us / 1e3, bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us)
    y = torch.empty(T, N_FEAT, device=dev, dtype=torch.bfloat16)
    int8_peak = 2.0 * tens
    popc_peak = 148 * 16 * 32 * 2 * 1.965e9
    for k in (2, 16):
        tile, alpha = rand_tile(N_FEAT * N_FEAT // k), torch.rand(k, device=dev, generator=gen) * 0.02
        us = graph_us(lambda: B.tbn_linear_bin_fwd(xb, N_FEAT, N_FEAT, tile, k, alpha, B.ALPHA_PER_TILE, beta=beta, y=y),
                      reps=3, iters=3)
        ops = 2.0 * T * (N_FEAT // k) * N_FEAT
        nbytes = xb.numel() * 4 + y.numel() * 2 + N_FEAT * N_FEAT // k / 8
        t_bound = max(ops / int8_peak, nbytes / hbm)
        out[f"bin_linear_T{T}_k{k}"] = dict(us=us, alg_tops=ops / us / 1e6, alg_gbs=nbytes / us / 1e3,
                                            bound="tensor (int8)" if ops / int8_peak > nbytes / hbm else "hbm",
                                            frac_of_binding_roofline=t_bound * 1e6 / us,
                                            popcount_alu_peak_tops=popc_peak / 1e12)
    # the same layer with the activation signs expanded to bytes once (one pass over the bits) and staged by TMA
    xbytes = torch.empty((T, N_FEAT), dtype=torch.uint8, device=dev)
    xpop = torch.empty(T, dtype=torch.int32, device=dev)
    us = graph_us(lambda: B.tbn_bin_expand_fwd(xb, N_FEAT, x_bytes=xbytes, x_pop=xpop), reps=3, iters=3)
    nbytes = xb.numel() * 4 + xbytes.numel() + T * 4
    out["bin_expand_T16384_8192"] = dict(us=us, alg_gbs=nbytes / us / 1e3, bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us)
    us = graph_us(lambda: B.tbn_binarize_bytes_fwd(x), reps=3, iters=3)
    nbytes = x.numel() * 2 + xb.numel() * 4 + xbytes.numel() + T * 8
    out["binarize_with_bytes_T16384_8192"] = dict(us=us, alg_gbs=nbytes / us / 1e3, bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us,
                                                  note="threshold, packing, row scale, sign bytes and row popcounts in one pass")
    for k in (2, 16):
        tile, alpha = rand_tile(N_FEAT * N_FEAT // k), torch.rand(k, device=dev, generator=gen) * 0.02
        us = graph_us(lambda: B.tbn_linear_bin_bytes_fwd(xbytes, xpop, N_FEAT, N_FEAT, tile, k, alpha, B.ALPHA_PER_TILE, beta=beta,
                                                         y=y), reps=3, iters=3)
        ops = 2.0 * T * (N_FEAT // k) * N_FEAT
        nbytes = xbytes.numel() + y.numel() * 2 + N_FEAT * N_FEAT // k / 8
        t_bound = max(ops / int8_peak, nbytes / hbm)
        out[f"bin_linear_bytes_T{T}_k{k}"] = dict(us=us, alg_tops=ops / us / 1e6, alg_gbs=nbytes / us / 1e3,
                                                  bound="tensor (int8)" if ops / int8_peak > nbytes / hbm else "hbm",
                                                  frac_of_binding_roofline=t_bound * 1e6 / us)
    del x, y, xbytes
    xb16 = xb[:16].contiguous()
    y16 = torch.empty(16, N_FEAT, device=dev, dtype=torch.bfloat16)
    tile, alpha = rand_tile(N_FEAT * N_FEAT // 2), torch.rand(2, device=dev, generator=gen) * 0.02
    us = graph_us(lambda: B.tbn_linear_bin_fwd(xb16, N_FEAT, N_FEAT, tile, 2, alpha, B.ALPHA_PER_TILE, beta=beta[:16], y=y16))
    out["bin_linear_T16_k2_popcount_kernel"] = dict(us=us, alg_tops=2.0 * 16 * (N_FEAT // 2) * N_FEAT / us / 1e6,
                                                    alg_gbs=(N_FEAT * N_FEAT // 2 / 8 + 16 * N_FEAT * 2.125) / us / 1e3,
                                                    bound="launch / hbm", l2="resident")
    # Small batch against HBM: a CUDA-graph chain of distinct layers whose tiles (4 MiB each at k = 2) add up to
    # more than L2, so every layer's tile really comes from HBM; per-layer time and tile GB/s.
    for T in (1, 16):
        k, n_layers = 2, 40
        x = torch.randn(T, N_FEAT, device=dev, generator=gen).to(torch.bfloat16)
        ys = [torch.empty(T, N_FEAT, device=dev, dtype=torch.bfloat16) for _ in range(2)]
        tiles = [rand_tile(N_FEAT * N_FEAT // k) for _ in range(n_layers)]
        alpha = torch.rand(k, device=dev, generator=gen) * 0.02
        ws = torch.empty(max(B.tbn_linear_workspace_bytes(T, N_FEAT, N_FEAT, k, B.BF16), 16), dtype=torch.uint8, device=dev)

        def chain():
            cur = x
            for l in range(n_layers):
                B.tbn_linear_fwd(cur, N_FEAT, tiles[l], k, alpha, B.ALPHA_PER_TILE, act=B.ACT_RELU, y=ys[l & 1], workspace=ws)
                cur = ys[l & 1]

        us = graph_us(chain, reps=1, iters=5) / n_layers
        nbytes = N_FEAT * N_FEAT // k / 8 + 2 * T * N_FEAT * 2
        out[f"small_batch_chain_T{T}_k{k}_{n_layers}_layers"] = dict(
            us_per_layer=us, path=B.tbn_linear_select_path(T, N_FEAT, N_FEAT, k, B.BF16), alg_gbs=nbytes / us / 1e3,
            bound="hbm", frac_of_binding_roofline=nbytes / hbm * 1e6 / us, l2="tiles exceed L2 (160 MiB)")
    return out


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    from paper_2407_12075_b200 import binding as B
    from paper_2407_12075_b200 import build as tbn_build
    from paper_2407_12075_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        tbn_build.build()
    if world > 1:
        dist.barrier()
    B.lib()

    T = args.tokens
    peaks = read_peaks()
    # ---- seeded synthetic inputs, resident in HBM before the timed region -----------------------
    x_np = synth.to_bf16_bits(synth.normal(SEED, 0, T * N_FEAT).reshape(T, N_FEAT))
    W_np = synth.normal(SEED, 1, N_FEAT * N_FEAT, 0.02).reshape(N_FEAT, N_FEAT)
    x = torch.from_numpy(x_np.view(np.int16)).view(torch.bfloat16).to(dev)
    Wd = torch.from_numpy(W_np).to(dev)
    layers = {}
    for k in KS:
        layers[k] = B.tbn_aggregate_tile(Wd, k, B.ALPHA_PER_TILE)
    del Wd
    y = torch.empty((T, N_FEAT), dtype=torch.bfloat16, device=dev)
    ws = torch.empty(max(max(B.tbn_linear_workspace_bytes(T, N_FEAT, N_FEAT, k, B.BF16) for k in KS), 16),
                     dtype=torch.uint8, device=dev)
    path_names = {1: "generic", 2: "small-batch", 3: "tensor (tcgen05)"}
    path = path_names.get(B.tbn_linear_select_path(T, N_FEAT, N_FEAT, 2, B.BF16), "?")

    def step(events=None):
        for i, k in enumerate(KS):
            tile, alpha = layers[k]
            if events is not None:
                events[i][0].record()
            B.tbn_linear_fwd(x, N_FEAT, tile, k, alpha, B.ALPHA_PER_TILE, y=y, workspace=ws)
            if events is not None:
                events[i][1].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    code, detail = B.tbn_last_device_status()
    if code != 0:
        raise SystemExit(f"device-side status {code} (detail {detail}) after warm-up")

    # ---- timed region: K steps, CUDA events on the launching stream, clocks sampled meanwhile ----
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in KS]
          for _ in range(args.steps)]
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_first()
    barrier()
    sampler.mark()
    t_beg.record()
    for s in range(args.steps):
        step(ev[s])
    t_end.record()
    torch.cuda.synchronize()
    timed_rows = sampler.count()
    # a short timed region can end between two samples: keep the same load running (untimed) until a few samples exist
    extra = 0
    t_extra = time.time()
    while sampler.proc is not None and sampler.count() < 3 and time.time() - t_extra < 3.0:
        step()
        torch.cuda.synchronize()
        extra += 1
    barrier()
    clocks = sampler.stop()
    clocks["samples_timed_region"] = timed_rows
    clocks["samples_untimed_extension"] = max(clocks.get("samples", 0) - timed_rows, 0)
    if extra:
        clocks["note"] = (f"timed region shorter than the sampling interval: {extra} more untimed steps of the same load "
                          f"ran while sampling")
    total_ms = max_over_ranks(t_beg.elapsed_time(t_end), dev)
    ms_per_step = total_ms / args.steps
    per_k_ms = {k: float(np.mean([ev[s][i][0].elapsed_time(ev[s][i][1]) for s in range(args.steps)]))
                for i, k in enumerate(KS)}
    flops_step = sum(algorithmic_flops(T, k) for k in KS)
    value = whole_job_value(flops_step, world, ms_per_step)

    # ---- roofline of the dominant kernel (the forward kernel, averaged over the four k) --------
    # The denominator follows the timed region (see tensor_peak_for): boost clocks -> burst peak, power cap -> sustained
    # peak.  Both fractions are printed; `frac` is the one that applies.
    kern_ms = float(np.mean(list(per_k_ms.values())))
    achieved = flops_step / len(KS) / (kern_ms * 1e-3) / 1e12
    peak, peak_kind = tensor_peak_for(total_ms, peaks, clocks.get("sm_mhz") if timed_rows else None, clocks.get("sm_max_mhz"))
    per_k = {}
    for k in KS:
        tf = algorithmic_flops(T, k) / (per_k_ms[k] * 1e-3) / 1e12
        gbs = algorithmic_bytes(T, k) / (per_k_ms[k] * 1e-3) / 1e9
        t_hbm = algorithmic_bytes(T, k) / (peaks["hbm_gbs"] * 1e9)
        fr = {}
        for kind, pk in (("burst", peaks["bf16_tflops"]), ("sustained", peaks["bf16_tflops_sustained"])):
            fr[kind] = max(algorithmic_flops(T, k) / (pk * 1e12), t_hbm) / (per_k_ms[k] * 1e-3)
        per_k[str(k)] = dict(ms=per_k_ms[k], alg_tflops=tf, dense_equiv_tflops=tf * k, alg_gbs=gbs,
                             frac_of_binding_roofline=fr[peak_kind], frac_burst=fr["burst"], frac_sustained=fr["sustained"])
    roofline = dict(bound="tensor", achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                    frac_burst=achieved / peaks["bf16_tflops"], frac_sustained=achieved / peaks["bf16_tflops_sustained"],
                    traffic=measured_traffic(T), traffic_note="bytes per k = 2 launch, scaled from an ncu capture at T = 8192",
                    peak_source=f"{peaks['source']} ({peak_kind} bf16 GEMM: the timed region lasted {total_ms:.0f} ms)",
                    kernel_path=path, per_k=per_k)

    # ---- end to end: host buffers through the C-ABI, copies inside the timed region -------------
    e2e = None
    if args.e2e_steps > 0:
        xh = torch.from_numpy(x_np.view(np.int16)).view(torch.bfloat16).pin_memory()
        yh = torch.empty((T, N_FEAT), dtype=torch.bfloat16).pin_memory()
        hws = torch.empty(max(B.tbn_linear_host_workspace_bytes(T, N_FEAT, N_FEAT, k, B.BF16, B.BF16) for k in KS),
                          dtype=torch.uint8, device=dev)
        def host_step():
            for k in KS:
                tile, alpha = layers[k]
                B.tbn_linear_fwd_host(xh, yh, tile, k, alpha, B.ALPHA_PER_TILE, hws)
        host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / args.e2e_steps
        dt = max_over_ranks(dt, dev)
        nbytes = T * N_FEAT * 2 * len(KS)
        e2e = dict(value=world * flops_step / dt / 1e12, unit=UNIT, h2d_bytes_per_step=nbytes,
                   d2h_bytes_per_step=nbytes, ms_per_step=dt * 1e3, steps=args.e2e_steps)

    # ---- the oracle on the host cores, rank 0 at N = 1 only; its rows also check the timed kernel's output -------
    cpu = None
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        kp = 4 if 4 in KS else KS[0]
        # a short probe sizes the sample to roughly 12 s of CPU work on whatever host this is
        probe_dt = oracle_sample(x_np, W_np, kp, 32)[0]
        rows = int(min(max(32 * 12.0 / max(probe_dt, 1e-3), 96), 4096))
        dt, n, cores, pick, ref = oracle_sample(x_np, W_np, kp, rows)
        cpu = dict(value=algorithmic_flops(n, kp) / dt / 1e12, unit=UNIT, cores=cores, kind="oracle",
                   sample=f"{n} seeded token rows of {T} x all 8192 outputs at k={kp}, {dt:.1f} s; the oracle does the "
                          f"dense fp64 product ({2.0 * n * N_FEAT * N_FEAT / dt / 1e9:.2f} dense GFLOP/s), value "
                          f"counts algorithmic flops")
        # the same launch as in the timed step, once more, and its rows against the oracle's
        tile, alpha = layers[kp]
        B.tbn_linear_fwd(x, N_FEAT, tile, kp, alpha, B.ALPHA_PER_TILE, y=y, workspace=ws)
        torch.cuda.synchronize()
        got = y[torch.from_numpy(pick).to(dev)].to(torch.float64).cpu().numpy()
        worst = float((np.abs(got - ref) / (1e-2 * (1.0 + np.abs(ref)))).max())
        parity = dict(k=kp, rows=int(n), max_err_over_bound=worst, bound="1e-2 * (1 + |ref|)")
        if not worst <= 1.0:
            raise SystemExit(f"parity failure in the timed configuration: max err / bound = {worst}")

    others = None
    if rank == 0 and world == 1 and not args.no_other_configs:
        xh = yh = hws = None
        others = measure_other_configs(B, torch, dev, peaks)

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="bf16", data="synthetic",
                    config=workload_config(T),
                    clocks=clocks, e2e=e2e, gpu_launches=args.steps * len(KS), roofline=roofline,
                    cpu_baseline=cpu, parity=parity, other_configs=others)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
