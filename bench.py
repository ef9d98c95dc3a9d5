#!/usr/bin/env python
"""Benchmark of the BWLA W1A6 linear hot path on the Qwen3-32B-shaped linear stack.

A step is one pass over all 7 linears of all layers (rotate + quantise + binary contraction + low-rank + bf16
epilogue for every linear), back to back on one stream, replayed from a CUDA graph.  Inputs are seeded and
synthetic (no checkpoints or datasets exist here); all layers' weights stay resident in HBM (about 5 GB, far
larger than L2, so every step streams them from DRAM again).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the decode figure (algorithmic HBM bytes of the whole stack per second
at --decode-m tokens); `prefill` holds the INT8 TOPS figure at --prefill-m tokens; `roofline` is for the dominant
kernel (the tcgen05 contraction) timed with CUDA events around each of its launches.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_00422_b200 import inputs as gen  # noqa: E402

# DRAM bytes of one contraction launch from an ncu capture (profiles/), with the algorithmic bytes of that same launch and
# the hash of the kernel source the capture was taken from.  The ratio scales the average launch of the step; when the
# kernel source has changed since, the figure is dropped (null).
NCU_TRAFFIC = {
    "decode": {"dram_bytes": 19881728, "algorithmic_bytes": 20216896,          # gate_proj launch, M = 8
               "kernel_sha256": "c8b8ebb137de23f31e5bfe57756a613fbc1113d2d736c5cef58e013ed50bad3e"},
}

METRIC = "W1A6 linear: decode HBM GB/s & prefill INT8 TOPS vs B200 roofline, Qwen3-32B"
BITS = 6


# ----------------------------------------------------------------------------------------------
# workload arithmetic
# ----------------------------------------------------------------------------------------------
def call_bytes(sh: gen.LinearShape, M: int) -> int:
    """Algorithmic HBM bytes of one whole linear call: sign bits, low-rank factors, alpha, Kronecker factors,
    activations in, outputs out."""
    return (sh.N * sh.K // 8 + 2 * sh.r * (sh.N + sh.K) + 4 * sh.N + 4 * (sh.n1 ** 2 + sh.n2 ** 2)
            + 2 * M * sh.K + 2 * M * sh.N)


def contraction_kernel_bytes(sh: gen.LinearShape, M: int) -> int:
    """Algorithmic bytes of one launch of the contraction kernel (fused epilogue): sign bits, int8 codes, U, the three
    bf16 terms of T, alpha, per-token scale and code sum in; bf16 outputs out."""
    return sh.N * sh.K // 8 + M * sh.K + 2 * sh.r * sh.N + 6 * M * 64 + 4 * sh.N + 8 * M + 2 * M * sh.N


def kernel_source_hash() -> str:
    import hashlib
    with open(os.path.join(ROOT, "paper_2605_00422_b200", "csrc", "gemm_umma.cu"), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def measured_traffic(which: str, algorithmic_bytes_per_launch: float):
    t = NCU_TRAFFIC.get(which)
    if not t or not t["dram_bytes"] or t["kernel_sha256"] != kernel_source_hash():
        return None
    return t["dram_bytes"] / t["algorithmic_bytes"] * algorithmic_bytes_per_launch


def call_ops(sh: gen.LinearShape, M: int) -> int:
    return 2 * M * sh.K * sh.N


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------------------------
# replicas: N processes, one GPU each, no exchange on the data path
# ----------------------------------------------------------------------------------------------
def max_over_ranks(ms: float, world: int, device, dist, torch) -> float:
    """The slowest rank's time: what a job of `world` replicas that start together takes."""
    if world <= 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_rate(world: int, units_per_rank_per_step: float, steps: int, ms: float) -> float:
    """Whole-job units per second: every rank processes its own copy of the workload (weak scaling)."""
    return world * units_per_rank_per_step * steps / (ms * 1e-3)


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, mx = [], set(), None
        try:
            for ln in open(self.path):
                p = [v.strip() for v in ln.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0]))
                    mx = float(p[1])
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample
# ----------------------------------------------------------------------------------------------
def host_layer(layer: int):
    """Host tensors of one layer's 7 linears (numpy recipe of the parity tests)."""
    out = []
    for sh in gen.CONFIG_SHAPES[4]:
        lay = gen.make_layer(4, sh, BITS, layer=layer, direct_words=True)
        out.append((sh, lay))
    return out


def oracle_pass(layer_tensors, xs):
    import oracle
    for sh, lay in layer_tensors:
        oracle.linear(xs[sh.K], lay.P1, lay.P2, BITS, lay.packed, lay.alpha, lay.U, lay.V)


def run_reference(args):
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    M = args.decode_m
    lt = host_layer(0)
    xs = {}
    for sh, _ in lt:
        if sh.K not in xs:
            xs[sh.K] = gen.make_activations(4, sh, M)
    nbytes = sum(call_bytes(sh, M) for sh, _ in lt)
    for _ in range(max(1, min(args.warmup, 1))):
        oracle_pass(lt, xs)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_pass(lt, xs)
    dt = time.perf_counter() - t0
    val = nbytes * args.steps / dt / 1e9
    sample = f"one layer (7 linears) of the stack at M={M} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"qwen3-32b linear stack, decode M={M}, bounded sample: {sample}", "bits": BITS},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------
class Linear:
    __slots__ = ("shape", "P1", "P2", "packed", "alpha", "U", "V", "layer")


# the linears of one transformer block that read the same activations go through one grouped call
GROUPS = (("qkv", (0, 1, 2)), ("o", (3,)), ("gate_up", (4, 5)), ("down", (6,)))


def build_stack(layers: int, device, torch, bwla=None):
    """Per-layer seeded weights generated on the device (same distributions as the host recipe of the tests); with
    `bwla` every linear also gets its prepared-layer handle (constants put into kernel form once, not per call)."""
    stack = []
    for layer in range(layers):
        row = []
        for sh in gen.CONFIG_SHAPES[4]:
            g = torch.Generator(device=device)
            g.manual_seed(gen.ROOT_SEED * 1000003 + layer * 101 + sh.shape_id)
            lin = Linear()
            lin.shape = sh
            lin.P1 = torch.from_numpy(gen.orthogonal_f32(sh.n1, gen._rng(4, layer, sh.shape_id, gen.T_P1))).to(device)
            lin.P2 = torch.from_numpy(gen.orthogonal_f32(sh.n2, gen._rng(4, layer, sh.shape_id, gen.T_P2))).to(device)
            lin.packed = torch.randint(-2 ** 31, 2 ** 31, (sh.N, sh.K // 32), dtype=torch.int64, device=device,
                                       generator=g).to(torch.int32)
            lin.alpha = torch.exp(-4.0 + 0.3 * torch.randn(sh.N, device=device, generator=g))
            lin.U = (0.01 * torch.randn(sh.N, sh.r, device=device, generator=g)).to(torch.bfloat16)
            lin.V = (0.01 * torch.randn(sh.r, sh.K, device=device, generator=g)).to(torch.bfloat16)
            lin.layer = bwla.Layer(lin.P1, lin.P2, BITS, lin.packed, lin.alpha, lin.U, lin.V) if bwla is not None else None
            row.append(lin)
        stack.append(row)
    return stack


def student_t_activations(M: int, K: int, device, torch, seed: int):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    z = torch.randn(M, K, device=device, generator=g)
    chi = (torch.randn(3, M, K, device=device, generator=g) ** 2).sum(0)
    x = z / torch.sqrt(chi / 3.0)
    ch = torch.randperm(K, device=device, generator=g)[:8]
    x[:, ch] *= 50.0
    return x.to(torch.bfloat16)


def oracle_spot_check(stack, xs, M, bwla, torch, tokens=8):
    """Outside every timed region: the first layer's seven linears on a few tokens against the CPU oracle, through
    the same grouped calls the timed step makes.  Returns counts for the JSON line (nothing is asserted here; the
    parity tests assert)."""
    import oracle
    nt = min(tokens, M)
    rep = {"layer": 0, "tokens": nt, "elements_codes": 0, "near_ties": 0, "code_mismatches": 0,
           "code_mismatches_outside_window": 0, "outputs": 0, "over_literal_bound": 0, "max_abs_over_rms": 0.0, "rel_l2_max": 0.0}
    window = oracle.near_tie_window(BITS)
    for _, idx in GROUPS:
        lins = [stack[0][i] for i in idx]
        x = xs[lins[0].shape.K][:nt].contiguous()
        outs = bwla.bwla_w1ax_linear_group([l.layer for l in lins], x)
        torch.cuda.synchronize()
        xb = x.view(torch.int16).cpu().numpy().view(np.uint16)
        for lin, out in zip(lins, outs):
            packed = lin.packed.cpu().numpy().view(np.uint32)
            U = lin.U.view(torch.int16).cpu().numpy().view(np.uint16)
            V = lin.V.view(torch.int16).cpu().numpy().view(np.uint16)
            ref = oracle.linear(xb, lin.P1.cpu().numpy(), lin.P2.cpu().numpy(), BITS, packed, lin.alpha.cpu().numpy(), U, V)
            codes, _, _ = bwla.bwla_layer_rotate_quant(lin.layer, x)
            q = oracle.quantize(ref["Y"], BITS, "f64")
            bad = codes.cpu().numpy().astype(np.int32) != q["codes"].astype(np.int32)
            flagged = q["dist"] <= window
            got = gen.f32_from_bf16_bits(out.view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
            err = np.abs(got - ref["y"])
            rms = float(np.sqrt(np.mean(ref["y"] ** 2)))
            rep["elements_codes"] += int(bad.size)
            rep["near_ties"] += int(flagged.sum())
            rep["code_mismatches"] += int(bad.sum())
            rep["code_mismatches_outside_window"] += int((bad & ~flagged).sum())
            rep["outputs"] += int(err.size)
            rep["over_literal_bound"] += int(np.count_nonzero(err > 1e-2 * rms))
            rep["max_abs_over_rms"] = max(rep["max_abs_over_rms"], float(err.max() / rms))
            rep["rel_l2_max"] = max(rep["rel_l2_max"], float(np.linalg.norm(got - ref["y"]) / np.linalg.norm(ref["y"])))
    return rep


def cublas_bf16_context(shapes, layers, Ms, device, torch, distinct=8, reps=3):
    """Context only: the same stack as plain bf16 GEMMs (torch.matmul -> cuBLAS), x [M][K] times W^T [K][N] for the 7
    shapes of every layer.  62 GB of bf16 weights would be needed for 64 distinct layers; `distinct` layers (7.8 GB, far
    above L2) are cycled instead."""
    out = {"distinct_layers": distinct, "note": "torch.matmul bf16, weights of %d distinct layers cycled over %d layers" % (distinct, layers)}
    W = [[torch.randn(sh.N, sh.K, device=device, dtype=torch.bfloat16) for sh in shapes] for _ in range(distinct)]
    for M in Ms:
        xs = {sh.K: torch.randn(M, sh.K, device=device, dtype=torch.bfloat16) for sh in shapes}
        ys = [torch.empty(M, sh.N, device=device, dtype=torch.bfloat16) for sh in shapes]

        def run():
            for l in range(layers):
                for i, sh in enumerate(shapes):
                    torch.matmul(xs[sh.K], W[l % distinct][i].t(), out=ys[i])
        run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        flops = layers * sum(2 * M * sh.K * sh.N for sh in shapes)
        wbytes = layers * sum(2 * sh.K * sh.N for sh in shapes)
        out[f"M{M}"] = {"ms_per_step": ms, "tflops": flops / (ms * 1e-3) / 1e12, "weight_gb_per_s": wbytes / (ms * 1e-3) / 1e9}
    del W
    return out


def run_per_shape(args):
    """Every shape of workload configs 1-3 at its token counts and bit widths, one linear at a time: whole call (CUDA
    events around a graph of calls over layers with distinct weights) and kernel-only times (events around each launch),
    for the chosen contraction path and, up to four tokens, for the other one.  Prints a markdown table; not part of the
    one-line benchmark contract."""
    import torch
    from paper_2605_00422_b200 import bwla
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    peaks = measured_peaks()
    NL = 6                                            # layers with distinct sign words per shape (cold weights)
    rows = []
    print("| config | shape | bits | M | path | whole call us | prologue us | contraction us | GB/s (call bytes) | TOPS (2MKN) | "
          "% of measured HBM | % of 8 TB/s | % of 2x burst bf16 | % of 4.5 POP/s | other path us |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for cfg in (1, 2, 3):
        if args.cfg and cfg != args.cfg:
            continue
        for sh in gen.CONFIG_SHAPES[cfg]:
            if args.shape and sh.name != args.shape:
                continue
            for bits in gen.CONFIG_BITS[cfg]:
                g = torch.Generator(device=device)
                g.manual_seed(1000 * cfg + sh.shape_id)
                P1 = torch.from_numpy(gen.orthogonal_f32(sh.n1, gen._rng(cfg, 0, sh.shape_id, gen.T_P1))).to(device)
                P2 = torch.from_numpy(gen.orthogonal_f32(sh.n2, gen._rng(cfg, 0, sh.shape_id, gen.T_P2))).to(device)
                alpha = torch.exp(-4.0 + 0.3 * torch.randn(sh.N, device=device, generator=g))
                U = (0.01 * torch.randn(sh.N, sh.r, device=device, generator=g)).to(torch.bfloat16)
                V = (0.01 * torch.randn(sh.r, sh.K, device=device, generator=g)).to(torch.bfloat16)
                layers = []
                for _ in range(NL):
                    pk = torch.randint(-2 ** 31, 2 ** 31, (sh.N, sh.K // 32), dtype=torch.int64, device=device, generator=g).to(torch.int32)
                    layers.append(bwla.Layer(P1, P2, bits, pk, alpha, U, V))
                for M in gen.CONFIG_TOKENS[cfg]:
                    if args.m and M != args.m:
                        continue
                    x = student_t_activations(M, sh.K, device, torch, 99 + M)
                    out = [torch.empty(M, sh.N, dtype=torch.bfloat16, device=device)]
                    ws = torch.zeros(bwla.bwla_group_workspace_bytes([layers[0]], M), dtype=torch.uint8, device=device)

                    def measure(path):
                        bwla.bwla_force_path(path)
                        try:
                            run = lambda: [bwla.bwla_w1ax_linear_group([L], x, outs=out, workspace=ws) for L in layers]
                            run()
                            torch.cuda.synchronize()
                            gr = torch.cuda.CUDAGraph()
                            with torch.cuda.graph(gr):
                                run()
                            reps = 5 if M <= 512 else 2
                            gr.replay()
                            torch.cuda.synchronize()
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            e0.record()
                            for _ in range(reps):
                                gr.replay()
                            e1.record()
                            torch.cuda.synchronize()
                            whole = e0.elapsed_time(e1) / reps / NL * 1e3
                            bwla.bwla_profile_enable(True)
                            run()
                            prof = bwla.bwla_profile_collect()
                            bwla.bwla_profile_enable(False)
                            return whole, prof["prologue"][0] / NL * 1e3, prof["contraction"][0] / NL * 1e3
                        finally:
                            bwla.bwla_force_path(bwla.BWLA_PATH_AUTO)

                    chosen = bwla.bwla_chosen_path(M, sh.K, sh.N, sh.r, bits)
                    whole, pro, con = measure(bwla.BWLA_PATH_AUTO)
                    other = ""
                    if M <= 4:
                        alt = bwla.BWLA_PATH_BITPLANE if chosen == bwla.BWLA_PATH_I8 else bwla.BWLA_PATH_I8
                        other = "%.1f (%s)" % (measure(alt)[0], {2: "bit-plane", 3: "tcgen05"}[alt])
                    gbs = call_bytes(sh, M) / (whole * 1e-6) / 1e9
                    tops = call_ops(sh, M) / (whole * 1e-6) / 1e12
                    name = {1: "simple", 2: "bit-plane", 3: "tcgen05 i8"}[chosen]
                    print(f"| {cfg} | {sh.name} {sh.K}->{sh.N} | {bits} | {M} | {name} | {whole:.1f} | {pro:.1f} | {con:.1f} | {gbs:.0f} | "
                          f"{tops:.1f} | {100 * gbs / peaks['hbm_gbs']:.1f} | {100 * gbs / 8000.0:.1f} | "
                          f"{100 * tops / (2 * peaks['bf16_tflops']):.1f} | {100 * tops / 4500.0:.1f} | {other} |", flush=True)
                del layers
                torch.cuda.empty_cache()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2605_00422_b200 import bwla

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    peaks = measured_peaks()
    shapes = gen.CONFIG_SHAPES[4]
    stack = build_stack(args.layers, device, torch, bwla)
    torch.cuda.synchronize()
    Ks = sorted({sh.K for sh in shapes})

    def make_io(M):
        xs = {K: student_t_activations(M, K, device, torch, 7000 + K + M) for K in Ks}
        outs = {sh.name: torch.empty(M, sh.N, dtype=torch.bfloat16, device=device) for sh in shapes}
        ws_bytes = max(bwla.bwla_group_workspace_bytes([stack[0][i].layer for i in idx], M) for _, idx in GROUPS)
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=device)
        return xs, outs, ws

    def step(xs, outs, ws, layers=None):
        n = 0
        for row in (stack if layers is None else stack[:layers]):
            for _, idx in GROUPS:
                lins = [row[i] for i in idx]
                bwla.bwla_w1ax_linear_group([l.layer for l in lins], xs[lins[0].shape.K],
                                            outs=[outs[l.shape.name] for l in lins], workspace=ws)
                n += bwla.bwla_last_launch_count()
        return n

    def capture(xs, outs, ws, layers=None):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step(xs, outs, ws, 1)        # sets per-kernel attributes before capture
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            launches = step(xs, outs, ws, layers)
        return g, launches

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, device, dist, torch)

    def kernel_profile(xs, outs, ws, passes=1, layers=None):
        bwla.bwla_profile_enable(True)
        for _ in range(passes):
            step(xs, outs, ws, layers)
        prof = bwla.bwla_profile_collect()
        bwla.bwla_profile_enable(False)
        return {k: (ms / passes, n // passes) for k, (ms, n) in prof.items() if n and not k.startswith('unused')}

    uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid).replace("GPU-", "")
    sampler = ClockSampler(uuid)

    # ------------------------------ decode ------------------------------
    # the weight-only operating point (Table 1, upper half): W1A16, rotated activations kept in bf16
    def measure_w1a16():
        def a16_step(xs_, outs_, ws_, layers_):
            for row in stack[:layers_]:
                for lin in row:
                    bwla.bwla_layer_w1a16_linear(lin.layer, xs_[lin.shape.K], out=outs_[lin.shape.name], workspace=ws_)
        res = {"workload": "same stack, W1A16 (bf16 rotated activations against the packed signs, bf16 tensor-core contraction)"}
        for Ma, La in ((args.decode_m, args.layers), (args.prefill_m, min(args.layers, 16))):
            if Ma <= 0:
                continue
            xs_a, outs_a, _ = make_io(Ma)
            ws_a = torch.zeros(max(bwla.bwla_w1a16_workspace_bytes(l.layer, Ma) for l in stack[0]), dtype=torch.uint8, device=device)
            a16_step(xs_a, outs_a, ws_a, 1)
            torch.cuda.synchronize()
            g_a = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_a):
                a16_step(xs_a, outs_a, ws_a, La)
            ms_a = timed(g_a.replay, 3, 2) / 3 * (args.layers / La)
            res[f"M{Ma}"] = {"ms_per_step": ms_a, "layers_timed": La,
                             "GB/s": world * args.layers * sum(call_bytes(sh, Ma) for sh in shapes) / (ms_a * 1e-3) / 1e9,
                             "TFLOP/s (2MKN)": world * args.layers * sum(call_ops(sh, Ma) for sh in shapes) / (ms_a * 1e-3) / 1e12,
                             "status": bwla.bwla_check_status(ws_a)}
            del g_a, ws_a, xs_a, outs_a
            torch.cuda.empty_cache()
        return res

    if args.only_w1a16:
        if rank == 0:
            print(json.dumps({"w1a16": measure_w1a16()}))
        if world > 1:
            dist.destroy_process_group()
        return

    M = args.decode_m
    xs, outs, ws = make_io(M)
    graph, launches_per_step = capture(xs, outs, ws)
    sampler.start()
    ms = timed(graph.replay, args.steps, max(args.warmup, 3))
    clocks = sampler.stop()
    status = bwla.bwla_check_status(ws)
    step_bytes = args.layers * sum(call_bytes(sh, M) for sh in shapes)
    value = replica_rate(world, step_bytes, args.steps, ms) / 1e9

    # end to end: activations arrive from pinned host memory and the last layer's outputs go back, every step
    h_xs = {K: xs[K].cpu().pin_memory() for K in Ks}
    h_outs = {n: torch.empty_like(o, device="cpu").pin_memory() for n, o in outs.items()}

    def e2e_step():
        for K in Ks:
            xs[K].copy_(h_xs[K], non_blocking=True)
        graph.replay()
        for n in h_outs:
            h_outs[n].copy_(outs[n], non_blocking=True)

    e2e_ms = timed(e2e_step, args.steps, 3)
    h2d = sum(h_xs[K].numel() * 2 for K in Ks)
    d2h = sum(h.numel() * 2 for h in h_outs.values())
    e2e_value = replica_rate(world, step_bytes, args.steps, e2e_ms) / 1e9

    prof = kernel_profile(xs, outs, ws)
    k_ms, k_n = prof.get("contraction", (0.0, 0))
    k_bytes = args.layers * sum(contraction_kernel_bytes(sh, M) for sh in shapes)
    achieved = k_bytes / (k_ms * 1e-3) / 1e9 if k_ms > 0 else None
    roofline = {"bound": "hbm", "kernel": "umma_w1a_kernel (tcgen05 kind::i8 contraction), decode stack",
                "achieved": achieved, "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": (achieved / peaks["hbm_gbs"]) if achieved else None,
                "traffic": measured_traffic("decode", k_bytes / k_n) if k_n else None,
                "launches_per_step": k_n, "avg_launch_us": (k_ms / k_n * 1e3) if k_n else None,
                "algorithmic_bytes_per_launch": (k_bytes / k_n) if k_n else None,
                "algorithmic_bytes_per_step": k_bytes,
                # the same launches charged with the whole call's algorithmic bytes (sign bits, U and V, alpha, Kronecker
                # factors, activations in, outputs out) instead of what the contraction kernel itself reads and writes
                "achieved_with_call_bytes": (step_bytes / (k_ms * 1e-3) / 1e9) if k_ms > 0 else None,
                "whole_step_frac": value / world / peaks["hbm_gbs"]}
    del graph
    spot = oracle_spot_check(stack, xs, M, bwla, torch) if (rank == 0 and not args.no_cpu_baseline) else None

    # the other decode batch sizes of the workload, whole-step only
    decode_other = {}
    for Mo in args.decode_also:
        if Mo == M:
            continue
        xs_o, outs_o, ws_o = make_io(Mo)
        graph_o, _ = capture(xs_o, outs_o, ws_o)
        ms_o = timed(graph_o.replay, max(3, args.steps // 2), 3) / max(3, args.steps // 2)
        bytes_o = args.layers * sum(call_bytes(sh, Mo) for sh in shapes)
        decode_other[f"M{Mo}"] = {"value": world * bytes_o / (ms_o * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms_o,
                                  "status": bwla.bwla_check_status(ws_o)}
        del graph_o

    # both contraction paths at one and four tokens (the bit-plane kernel takes at most four); AUTO picks per shape
    decode_paths = {}
    if not args.skip_extras:
        for Mo in (1, 4):
            xs_o, outs_o, ws_o = make_io(Mo)
            for name, path in (("bitplane", bwla.BWLA_PATH_BITPLANE), ("i8", bwla.BWLA_PATH_I8)):
                bwla.bwla_force_path(path)
                try:
                    graph_o, _ = capture(xs_o, outs_o, ws_o)
                    ms_o = timed(graph_o.replay, 5, 3) / 5
                finally:
                    bwla.bwla_force_path(bwla.BWLA_PATH_AUTO)
                bytes_o = args.layers * sum(call_bytes(sh, Mo) for sh in shapes)
                decode_paths[f"M{Mo}_{name}"] = {"ms_per_step": ms_o, "value": world * bytes_o / (ms_o * 1e-3) / 1e9, "unit": "GB/s",
                                                 "status": bwla.bwla_check_status(ws_o)}
                del graph_o
        decode_paths["M8"] = "the bit-plane kernel takes at most four tokens; see decode_other_batches for the tcgen05 path"
        decode_paths["chosen"] = {f"M{Mo}": {sh.name: bwla.bwla_chosen_path(Mo, sh.K, sh.N, sh.r, BITS) for sh in shapes} for Mo in (1, 4, 8, 16)}

    # the operating point of the paper's end-to-end figure (Sec. 4.4): W1A8 at batch 4, decode
    w1a8 = None
    if not args.skip_extras:
        for row in stack:
            for lin in row:
                lin.layer = bwla.Layer(lin.P1, lin.P2, 8, lin.packed, lin.alpha, lin.U, lin.V)
        torch.cuda.synchronize()
        xs_8, outs_8, ws_8 = make_io(4)
        graph_8, _ = capture(xs_8, outs_8, ws_8)
        ms_8 = timed(graph_8.replay, 5, 3) / 5
        bytes_8 = args.layers * sum(call_bytes(sh, 4) for sh in shapes)
        w1a8 = {"workload": "same stack, 8-bit codes, 4 tokens (batch 4 decode)", "ms_per_step": ms_8,
                "value": world * bytes_8 / (ms_8 * 1e-3) / 1e9, "unit": "GB/s", "status": bwla.bwla_check_status(ws_8)}
        del graph_8
        for row in stack:
            for lin in row:
                lin.layer = bwla.Layer(lin.P1, lin.P2, BITS, lin.packed, lin.alpha, lin.U, lin.V)
        torch.cuda.synchronize()

    w1a16 = measure_w1a16() if not args.skip_extras else None

    # ------------------------------ prefill ------------------------------
    prefill = None
    if args.prefill_m > 0:
        Mp = args.prefill_m
        xs_p, outs_p, ws_p = make_io(Mp)
        Lp = min(args.prefill_layers or args.layers, args.layers)
        graph_p, _ = capture(xs_p, outs_p, ws_p, Lp)
        steps_p = max(2, args.steps // 5)
        sampler_p = ClockSampler(uuid)
        sampler_p.start()
        ms_p = timed(graph_p.replay, steps_p, 3)
        clocks_p = sampler_p.stop()
        ops = Lp * sum(call_ops(sh, Mp) for sh in shapes)
        tops = world * ops * steps_p / (ms_p * 1e-3) / 1e12
        prof_p = kernel_profile(xs_p, outs_p, ws_p, layers=Lp)
        kp_ms, kp_n = prof_p.get("contraction", (0.0, 0))
        k_tops = ops / (kp_ms * 1e-3) / 1e12 if kp_ms > 0 else None
        # int8 dense = 2 x bf16 (nominal ratio) of the measured bf16 rate; the burst figure is the denominator (the
        # clocks stay at their maximum in this step), the sustained and the nominal ones are printed beside it
        i8_peak = 2.0 * peaks["bf16_tflops"]
        prefill = {"metric": "prefill INT8 TOPS (2*M*K*N of the contraction / whole-step time)", "value": tops,
                   "unit": "TOPS", "M": Mp, "layers": Lp, "steps": steps_p, "ms_per_step": ms_p / steps_p, "clocks": clocks_p,
                   "roofline": {"bound": "tensor", "kernel": "umma_w1a_persistent_kernel (tcgen05 kind::i8 contraction), prefill stack", "achieved": k_tops,
                                "peak": i8_peak, "peak_source": peaks["source"] + " bf16 burst x 2 (int8:bf16 nominal ratio)",
                                "unit": "TOP/s", "frac": (k_tops / i8_peak) if k_tops else None, "traffic": None,
                                "frac_of_sustained": (k_tops / (2.0 * peaks["bf16_tflops_sustained"])) if k_tops else None,
                                "frac_of_nominal_4500": (k_tops / 4500.0) if k_tops else None,
                                "whole_call_frac_of_nominal_4500": tops / 4500.0,
                                "launches_per_step": kp_n},
                   "kernel_ms_per_step": {k: round(v[0], 4) for k, v in prof_p.items()},
                   "status": bwla.bwla_check_status(ws_p)}
        del graph_p

    # ------------------------------ CPU baseline (rank 0, N = 1) ------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        lt = host_layer(0)
        hx = {}
        for sh, _ in lt:
            if sh.K not in hx:
                hx[sh.K] = gen.make_activations(4, sh, M)
        t0 = time.perf_counter()
        reps = 0
        while reps < 1 or (time.perf_counter() - t0 < 10.0 and reps < 50):
            oracle_pass(lt, hx)
            reps += 1
        dt = time.perf_counter() - t0
        cpu = {"value": reps * sum(call_bytes(sh, M) for sh, _ in lt) / dt / 1e9, "unit": "GB/s",
               "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"{reps} pass(es) over one layer (7 linears) at M={M}; {dt:.1f} s"}

    cublas = None
    if rank == 0 and world == 1 and not args.no_cublas:
        del stack
        torch.cuda.empty_cache()
        cublas = cublas_bf16_context(shapes, args.layers, [M] + ([args.prefill_m] if args.prefill_m > 0 else []), device, torch)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "dtype_detail": "int8 codes x 1-bit signs -> int32 (fp32 rotation, bf16 in/out)", "data": "synthetic",
            "config": {"workload": f"qwen3-32b linear stack (config 4): {args.layers} layers x 7 W1A6 linears, decode M={M}, "
                                   f"rank 64, all weights resident ({step_bytes / 1e9:.2f} GB algorithmic bytes per step)",
                       "bits": BITS, "l2": "inputs larger than L2 (weights of all layers are streamed every step)",
                       "launch": "one CUDA graph per step, one stream", "parallelism": "replicas only"},
            "clocks": clocks, "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                                      "ms_per_step": e2e_ms / args.steps},
            "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
            "kernel_ms_per_step": {k: round(v[0], 4) for k, v in prof.items()},
            "cpu_baseline": cpu, "decode_other_batches": decode_other, "prefill": prefill, "device_status": status,
            "parity_spot_check": spot, "cublas_bf16_context": cublas, "decode_paths": decode_paths, "w1a8_batch4": w1a8, "w1a16": w1a16,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=gen.QWEN3_32B_LAYERS)
    ap.add_argument("--decode-m", type=int, default=16)
    ap.add_argument("--decode-also", type=int, nargs="*", default=[1, 64], help="further decode batch sizes (whole-step time only)")
    ap.add_argument("--prefill-m", type=int, default=2048)
    ap.add_argument("--prefill-layers", type=int, default=0, help="layers in the prefill step (0 = all)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cublas", action="store_true", help="skip the cuBLAS bf16 context measurement")
    ap.add_argument("--skip-extras", action="store_true", help="skip the forced-path, W1A8 batch-4 and W1A16 steps")
    ap.add_argument("--only-w1a16", action="store_true", help="time only the W1A16 (weight-only) stack and print its figures")
    ap.add_argument("--per-shape", action="store_true", help="time every shape of workload configs 1-3 on its own and print a table")
    ap.add_argument("--shape", default=None, help="with --per-shape: only the shape of this name (e.g. q_gate)")
    ap.add_argument("--cfg", type=int, default=0, help="with --per-shape: only this workload config (1, 2 or 3)")
    ap.add_argument("--m", type=int, default=0, help="with --per-shape: only this token count")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.per_shape:
        run_per_shape(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
