#!/usr/bin/env python
"""Benchmark of the SPARQ hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras] [--full]
                    [--section NAME]

A step is one pass of the whole hot path -- vSPARQ transform (n = 4, five placements, round to
nearest) inside the u8 x s8 -> s32 implicit-GEMM convolution, fp32 scale + bias + ReLU +
requantize to uint8 -- over one batch of the largest single-GPU workload of the ablation config:
128 x 28 x 28 x 128 NHWC uint8 activations (50 % zeros) -> 128 filters of 3x3, stride 1, pad 1
(29.6 GOP).  One fused kernel launch per step.  Prints ONE JSON line; the other configs (tiny
GEMM, ResNet-18 layer, ResNet-50 sweep, 2^30-byte transform, the ablation grid) are compact
entries of its `extra` object, and `--section NAME` prints one of them in full.

With --impl reference the CPU oracle is timed instead (rank 0 only): each step is the same layer
on a bounded number of images.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import sparq_synth as synth  # noqa: E402

METRIC = "fused SPARQ INT8 conv TOPS"
UNIT = "TOPS"
WORKLOAD = "cfg5 conv3x3 128x28x28x128->128 s1 p1, fused vSPARQ n=4 5opt +R, 50% zeros, requant u8"

# the layer the headline is quoted on (ablation config, fused vSPARQ 5opt +R, 50 % zeros)
HEAD = dict(nb=128, h=28, w=28, c=128, cout=128, r=3, s=3, stride=1, pad=1, zf=0.5, seed=500)
# ResNet-18-style layer (32 x 56 x 56 x 64 -> 64, 45 % zeros)
RN18 = dict(nb=32, h=56, w=56, c=64, cout=64, r=3, s=3, stride=1, pad=1, zf=0.45, seed=1)
L2_BYTES = 126 * 1024 * 1024
OPS_PER_STEP = 2 * 128 * 28 * 28 * 128 * 3 * 3 * 128       # the headline layer; dense count: no MAC is skipped
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0
NOMINAL_INT8_TOPS = 4500.0          # dense, datasheet (2 x the 2.25 PFLOP/s bf16 figure)
MIN_TIMED_MS = 50.0                 # device time every reported figure is the median over, at least

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarized under
# profiles/; None whenever the kernel has changed since its capture.
TRAFFIC = {"head": 13077504 + 0,                # profiles/sparq_conv_window_kernel_cfg5.txt (output still dirty in L2)
           "rn18": 6542336 + 0,                  # profiles/sparq_conv_window_kernel_cfg2.txt
           "layer1x1": 12931584 + 2800256,        # profiles/sparq_gemm_kernel_layer1x1.txt (mean of the two launches)
           "transform_per_2p28": 268445184 + 214811392}   # profiles/quantize_vec_kernel_2p28.txt


def ops_of(L):
    ho = (L["h"] + 2 * L["pad"] - L["r"]) // L["stride"] + 1
    wo = (L["w"] + 2 * L["pad"] - L["s"]) // L["stride"] + 1
    return 2 * L["nb"] * ho * wo * L["cout"] * L["r"] * L["s"] * L["c"]


def bytes_of(L):
    ho = (L["h"] + 2 * L["pad"] - L["r"]) // L["stride"] + 1
    wo = (L["w"] + 2 * L["pad"] - L["s"]) // L["stride"] + 1
    return L["nb"] * L["h"] * L["w"] * L["c"], L["nb"] * ho * wo * L["cout"], L["cout"] * L["r"] * L["s"] * L["c"]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]), source="measured")
    return dict(hbm=FALLBACK_HBM_GBS, bf16=FALLBACK_BF16_TFLOPS, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(self.gpu_index)],
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
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ---- timing ------------------------------------------------------------------------------------

def time_region(fn, steps, warmup, sync):
    """Eager loop, CUDA events on the current stream (for kernels that take >= 100 us)."""
    import torch
    for i in range(warmup):
        fn(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync()
    e0.record()
    for i in range(steps):
        fn(warmup + i)
    e1.record()
    sync()
    return e0.elapsed_time(e1)      # ms


class GraphTimer:
    """`steps` calls captured once into a CUDA graph (Python needs ~15 us to enqueue one call,
    more than a small layer takes on the device).  Each replay runs exactly `steps` steps and
    is timed by its own event pair on the launching stream; replays are enqueued back to back
    until at least `min_ms` of device time has been covered, and the median replay is reported."""

    def __init__(self, fn, steps, warmup):
        import torch
        self.steps = steps
        # warm-up on the stream the capture will use: the library sets up per-stream state
        # (workspaces) on a stream's first call, which must not happen inside a capture
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(warmup):
                fn(i)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph, stream=side):
            for i in range(steps):
                fn(warmup + i)
        self.graph.replay()            # the first replay also uploads the graph
        torch.cuda.synchronize()
        self.replays = 0

    def run(self, min_ms=None, barrier=None):
        import torch
        min_ms = MIN_TIMED_MS if min_ms is None else min(min_ms, MIN_TIMED_MS)
        probe0, probe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        probe0.record(); self.graph.replay(); probe1.record()
        torch.cuda.synchronize()
        one = max(probe0.elapsed_time(probe1), 1e-3)
        n = int(min(2000, max(5, np.ceil(1.2 * min_ms / one))))
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        torch.cuda.synchronize()
        if barrier:
            barrier()
        ev[0].record()
        for i in range(n):
            self.graph.replay()
            ev[i + 1].record()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        times = [ev[i].elapsed_time(ev[i + 1]) for i in range(n)]
        self.replays = n
        return statistics.median(times) / self.steps, sum(times), n


def device_activations(device, shape, zf, seed):
    """The config's value recipe drawn on the device (seeded torch generator): zeros with
    probability zf, else clip(round(|N(0,1)| * 40), 1, 255)."""
    import torch
    g = torch.Generator(device=device).manual_seed(seed)
    n = int(np.prod(shape))
    z = torch.randn(n, generator=g, device=device)
    v = torch.clamp(torch.round(z.abs() * 40.0), 1, 255).to(torch.uint8)
    if zf > 0:
        v[torch.rand(n, generator=g, device=device) < zf] = 0
    return v.view(*shape)


class ConvLayer:
    """One convolution workload with `sets` rotating input / output buffer pairs, so that
    consecutive steps never find their operands in the 126 MiB L2."""

    def __init__(self, device, L, sets=None, host_recipe=False):
        import torch
        self.L = L
        in_b, out_b, _ = bytes_of(L)
        if sets is None:
            sets = max(2, min(24, int(1.3 * L2_BYTES // (in_b + out_b)) + 1))
        self.sets = sets
        ho = (L["h"] + 2 * L["pad"] - L["r"]) // L["stride"] + 1
        wo = (L["w"] + 2 * L["pad"] - L["s"]) // L["stride"] + 1
        shape = (L["nb"], L["h"], L["w"], L["c"])
        if host_recipe:
            self.xs = [torch.from_numpy(synth.activations(L["seed"], shape, L["zf"], stream=10 + i)).to(device)
                       for i in range(sets)]
        else:
            self.xs = [device_activations(device, shape, L["zf"], L["seed"] * 64 + i) for i in range(sets)]
        self.outs = [torch.empty((L["nb"], ho, wo, L["cout"]), dtype=torch.uint8, device=device) for _ in range(sets)]
        self.wt = torch.from_numpy(synth.weights(L["seed"], (L["cout"], L["r"], L["s"], L["c"]))).to(device)
        self.scale = torch.from_numpy(synth.scales(L["seed"], L["cout"])).to(device)
        self.bias = torch.from_numpy(synth.bias(L["seed"], L["cout"])).to(device)
        self.inv = synth.inv_out_scale(L["r"] * L["s"] * L["c"], L["zf"])
        self.scratch = None

    def fused(self, params):
        import paper_2105_11010_b200 as sparq
        L = self.L

        def step(i):
            j = i % self.sets
            sparq.sparq_conv2d_nhwc_s8(self.xs[j], self.wt, (L["stride"], L["stride"]), (L["pad"], L["pad"]), params,
                                       scale=self.scale, bias=self.bias, relu=True, inv_out_scale=self.inv,
                                       u8_out=self.outs[j])
        return step

    def unfused(self, params):
        """Separate transform kernel into a scratch tensor, then the plain A8W8 convolution."""
        import torch
        import paper_2105_11010_b200 as sparq
        L = self.L
        if self.scratch is None:
            self.scratch = [torch.empty_like(self.xs[0]) for _ in range(min(self.sets, 4))]
        none = sparq.SparqParams(sparq.MODE_NONE)
        rows, row_len = L["nb"] * L["h"] * L["w"], L["c"]

        def step(i):
            j = i % self.sets
            t = self.scratch[i % len(self.scratch)]
            sparq.sparq_quantize(self.xs[j], t, rows, row_len, params)
            sparq.sparq_conv2d_nhwc_s8(t, self.wt, (L["stride"], L["stride"]), (L["pad"], L["pad"]), none,
                                       scale=self.scale, bias=self.bias, relu=True, inv_out_scale=self.inv,
                                       u8_out=self.outs[j])
        return step


def roofline_tensor(ops, ms, mma, pk, clocks_mhz, traffic, kernel, alg_bytes):
    """Roofline object of a contraction: achieved TOP/s of one step in a back-to-back stream
    against the measured tcgen05.mma kind::i8 rate at the SM clock sampled during the run."""
    tops = ops / (ms * 1e-3) / 1e12
    clk = clocks_mhz or pk.get("sm_max_mhz") or 1965.0
    peak = mma["mac_per_clk_sm"] * mma["sms"] * 2 * clk * 1e6 / 1e12 if mma else pk["bf16"] * 2
    return {
        "bound": "tensor", "achieved": round(tops, 1), "peak": round(peak, 1), "unit": "TOP/s",
        "frac": round(tops / peak, 4), "traffic": traffic,
        "peak_source": (f"measured: own MMA-only i8 loop, {mma['mac_per_clk_sm']:.0f} MAC/clk/SM x {mma['sms']} SMs x "
                        f"{clk:.0f} MHz sampled" if mma else f"{pk['source']} bf16 burst x 2"),
        "frac_of_nominal_4500": round(tops / NOMINAL_INT8_TOPS, 4),
        "per": "step in a back-to-back stream",
        "kernel": kernel, "ops": ops, "bytes": alg_bytes,
    }


# ---- sections ------------------------------------------------------------------------------------

def mma_peak_section(device, bns=(64, 128, 256), iters=2000):
    """The tensor core's own rate: the library's MMA-only loop on every SM (operands resident in
    shared memory).  MAC/clk/SM from the slowest CTA's cycle count; TOP/s from CUDA events."""
    import torch
    import paper_2105_11010_b200 as sparq
    cyc = torch.zeros(256, dtype=torch.int64, device=device)
    out = {}
    for bn in bns:
        sms = sparq.sparq_selftest_mma_rate(bn, iters, cyc)      # warm-up
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        sms = sparq.sparq_selftest_mma_rate(bn, iters, cyc)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        worst = int(cyc[:sms].max().item())
        macs_cta = iters * 4 * 128 * bn * 32
        out[f"n{bn}"] = {"mac_per_clk_sm": round(macs_cta / worst, 1), "ms": round(ms, 4),
                         "tops_by_events": round(2 * macs_cta * sms / ms / 1e9, 1)}
    sparq.sparq_check()
    best = max(out.values(), key=lambda d: d["mac_per_clk_sm"])
    out["sms"] = sms
    out["mac_per_clk_sm"] = best["mac_per_clk_sm"]
    out["implied_mhz"] = round(best["tops_by_events"] * 1e12 / (2 * best["mac_per_clk_sm"] * sms) / 1e6, 0)
    return out


def transform_section(device, pk, n, steps, warmup):
    """Standalone transform on n uint8 activations (50 % zeros), bSPARQ and vSPARQ, n = 4,
    five placements, round to nearest; rows of 1024.  Bytes = n read + n written."""
    import torch
    import paper_2105_11010_b200 as sparq
    sync = torch.cuda.synchronize
    x = torch.empty(n, dtype=torch.uint8, device=device)
    chunk = min(n, 1 << 26)
    for k, lo in enumerate(range(0, n, chunk)):
        x[lo:lo + chunk] = device_activations(device, (chunk,), 0.5, 4000 + k)
    y = torch.empty_like(x)
    tr = {"activations": n}
    for name, mode in (("bsparq", sparq.MODE_BSPARQ), ("vsparq", sparq.MODE_VSPARQ)):
        p = sparq.SparqParams(mode, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
        reps = max(steps, int(np.ceil(MIN_TIMED_MS / (2 * n / (pk["hbm"] * 1e6)))))
        ms = time_region(lambda i: sparq.sparq_quantize(x, y, n // 1024, 1024, p), reps, warmup, sync) / reps
        gbs = 2 * n / ms / 1e6
        tr[name] = {"ms": round(ms, 4), "gbs": round(gbs, 1),
                    "roofline": {"bound": "hbm", "achieved": round(gbs, 1), "peak": pk["hbm"], "unit": "GB/s",
                                 "frac": round(gbs / pk["hbm"], 4), "frac_of_nominal_8000": round(gbs / 8000.0, 4),
                                 "traffic": (TRAFFIC["transform_per_2p28"] * (n >> 28) if name == "bsparq" and n >= (1 << 28) else None),
                                 "peak_source": pk["source"] + " copy"}}
    sparq.sparq_check()
    return tr


def pack_section(device, pk, n, steps, warmup):
    """Packed stream codec on n uint8 activations (50 % zeros, rows of 1024), vSPARQ, round to
    nearest, for 4-, 3- and 2-bit windows with their full placement sets.  Algorithmic bytes of
    either direction = n (raw or unpacked activations) + n/16 * 2w (data plane) + n/16 * ctrl_bits
    (control plane), w = window bits."""
    import torch
    import paper_2105_11010_b200 as sparq
    sync = torch.cuda.synchronize
    x = device_activations(device, (n // 1024, 1024), 0.5, 6)
    y = torch.empty_like(x)
    out = {"activations": n}
    for w, mask in ((4, sparq.SET_5OPT), (3, sparq.SET_6OPT), (2, sparq.SET_7OPT)):
        p = sparq.SparqParams(sparq.MODE_VSPARQ, w, mask, sparq.ROUND_NEAREST)
        cb = sparq.sparq_packed_ctrl_bits(p)
        data = torch.empty(n // 16 * 2 * w, dtype=torch.uint8, device=device)
        ctrl = torch.empty(n // 16 * cb, dtype=torch.uint8, device=device)
        nbytes = n + n // 16 * 2 * w + n // 16 * cb
        res = {"ctrl_bits_per_pair": cb, "bits_per_activation": w + cb / 2}
        for name, fn in (("pack", lambda i: sparq.sparq_pack(x, p, data, ctrl)),
                         ("unpack", lambda i: sparq.sparq_unpack(data, ctrl, p, y))):
            ms = time_region(fn, steps, warmup, sync) / steps
            gbs = nbytes / ms / 1e6
            res[name] = {"ms": round(ms, 4), "gbs": round(gbs, 1), "frac_of_copy": round(gbs / pk["hbm"], 4)}
        out[f"n{w}"] = res
    sparq.sparq_check()
    return out


def frontend_section(device, pk, n, steps, warmup):
    """Min-max quantization front end on n activations (post-ReLU normal, fp32 and bf16):
    absmax (bytes = the input read once) and u8 quantization (input read + n bytes written)."""
    import torch
    import paper_2105_11010_b200 as sparq
    sync = torch.cuda.synchronize
    gen = torch.Generator(device=device).manual_seed(7)
    x32 = torch.randn(n, generator=gen, device=device).clamp_(min=0)
    out = torch.empty(n, dtype=torch.uint8, device=device)
    mx = torch.zeros(1, dtype=torch.float32, device=device)
    res = {"activations": n}
    for name, x in (("f32", x32), ("bf16", x32.to(torch.bfloat16))):
        eb = x.element_size()
        for op, fn, nbytes in (("absmax", lambda i: sparq.sparq_absmax(x, mx), n * eb),
                               ("quantize_u8", lambda i: sparq.sparq_quantize_act_u8(x, mx, out), n * eb + n)):
            ms = time_region(fn, steps, warmup, sync) / steps
            gbs = nbytes / ms / 1e6
            res[f"{op}_{name}"] = {"ms": round(ms, 4), "gbs": round(gbs, 1), "frac_of_copy": round(gbs / pk["hbm"], 4)}
    sparq.sparq_check()
    return res


def sparse24_section(device, pk, steps, warmup):
    """vSPARQ on 2:4 sparse weights, shape of the 28x28x128 -> 128 3x3 layer at batch 128
    (M 100352, K 1152, N 128): expansion of the activations (bytes = M*K read + 3*M*K
    written), then the dense contraction over the expanded operands.  Ops are counted as
    the sparse tensor core would: 2*M*N*K/2."""
    import torch
    import paper_2105_11010_b200 as sparq
    sync = torch.cuda.synchronize
    M, K, N = 100352, 1152, 128
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
    A = device_activations(device, (M, K), 0.5, 8)
    vals, pos = synth.sparse24_weights(8, N, K)
    w = torch.empty((N, 3 * K), dtype=torch.int8, device=device)
    sparq.sparq_sparse24_expand_weights(torch.from_numpy(vals).to(device), torch.from_numpy(pos).to(device), p, w)
    ws = torch.empty(M * 3 * K, dtype=torch.uint8, device=device)
    sc = torch.from_numpy(synth.scales(8, N)).to(device)
    out = torch.empty((M, N), dtype=torch.uint8, device=device)
    inv = synth.inv_out_scale(K // 2)
    ms_e = time_region(lambda i: sparq.sparq_sparse24_expand_activations(A, p, ws), steps, warmup, sync) / steps
    ms_t = time_region(lambda i: sparq.sparq_gemm_s8_sparse24(A, w, p, workspace=ws, scale=sc, relu=True,
                                                              inv_out_scale=inv, u8_out=out), steps, warmup, sync) / steps
    sparq.sparq_check()
    gbs = 4 * M * K / ms_e / 1e6
    return {"shape": {"M": M, "K": K, "N": N},
            "expand_activations": {"ms": round(ms_e, 4), "gbs": round(gbs, 1), "frac_of_copy": round(gbs / pk["hbm"], 4)},
            "gemm_sparse24": {"ms": round(ms_t, 4), "sparse_tops": round(M * N * K / ms_t / 1e9, 1),
                              "dense_equivalent_tops_executed": round(2 * M * N * 3 * K / ms_t / 1e9, 1)}}


def layer1x1_section(device, pk, steps, warmup):
    """The fused GEMM kernel on an output-heavy 1x1 layer of the ResNet-50 stack at batch 64
    (56x56x64 -> 256: M 200704, K 64, N 256; vSPARQ n = 4, five placements, round; scale + bias +
    ReLU + requantize).  Bandwidth-side roofline: bytes = input + output + weights."""
    import paper_2105_11010_b200 as sparq
    L = dict(nb=64, h=56, w=56, c=64, cout=256, r=1, s=1, stride=1, pad=0, zf=0.5, seed=9)
    layer = ConvLayer(device, L, sets=4)
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
    ms, _, _ = GraphTimer(layer.fused(p), steps, warmup).run()
    sparq.sparq_check()
    nbytes = sum(bytes_of(L))
    gbs = nbytes / ms / 1e6
    return {"layer": "56x56x64->256 1x1/s1, batch 64", "ms": round(ms, 4), "tops": round(ops_of(L) / ms / 1e9, 1),
            "roofline": {"bound": "hbm", "achieved": round(gbs, 1), "peak": pk["hbm"], "unit": "GB/s",
                         "frac": round(gbs / pk["hbm"], 4), "traffic": TRAFFIC["layer1x1"],
                         "peak_source": pk["source"] + " copy", "kernel": "sparq_gemm_kernel (fused 1x1 layer)",
                         "algorithmic_bytes_per_launch": nbytes}}


def cfg1_section(device, steps=200, warmup=10):
    """Tiny GEMM of config 1 (256 x 576 x 64, 50 % zeros, vSPARQ n = 4 5opt +R; int32 and fp32
    outputs): microseconds per launch in a back-to-back stream.  Launch-latency bound."""
    import torch
    import paper_2105_11010_b200 as sparq
    A = torch.from_numpy(synth.activations(0, (256, 576), 0.5)).to(device)
    B = torch.from_numpy(np.ascontiguousarray(synth.weights(0, (576, 64)).T)).to(device)
    sc = torch.from_numpy(synth.scales(0, 64)).to(device)
    acc = torch.empty((256, 64), dtype=torch.int32, device=device)
    f32 = torch.empty((256, 64), dtype=torch.float32, device=device)
    out = {}
    for name, mode in (("vsparq", sparq.MODE_VSPARQ), ("none", sparq.MODE_NONE)):
        p = sparq.SparqParams(mode, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
        ms, _, _ = GraphTimer(lambda i: sparq.sparq_gemm_s8(A, B, p, scale=sc, acc_out=acc, f32_out=f32), steps, warmup).run(20.0)
        out[name + "_us"] = round(ms * 1e3, 2)
    sparq.sparq_check()
    return out


def cfg5_section(device, steps=20, warmup=3, full=True):
    """Ablation grid on the 128 x 28 x 28 x 128 -> 128 3x3 layer: microseconds per step, fused
    (transform inside the convolution kernel) / unfused (transform kernel into a scratch tensor,
    then the plain convolution), for the window widths, placement sets and roundings at 50 %
    zeros, and for the zero fractions with n = 4, five placements, round.  Restricted sets for
    n = 3 and n = 2 are this library's extension, not the paper's."""
    import paper_2105_11010_b200 as sparq
    V, B_ = sparq.MODE_VSPARQ, sparq.MODE_BSPARQ
    grid = [("v4_5opt_R", V, 4, 0x1F, 1), ("v4_5opt_T", V, 4, 0x1F, 0), ("v4_3opt_R", V, 4, 0x15, 1),
            ("v4_2opt_R", V, 4, 0x11, 1), ("b4_5opt_R", B_, 4, 0x1F, 1), ("b4_5opt_T", B_, 4, 0x1F, 0),
            ("v3_6opt_R", V, 3, 0x3F, 1), ("v3_6opt_T", V, 3, 0x3F, 0), ("v3_x35_R", V, 3, 0x35, 1),
            ("v3_x29_R", V, 3, 0x29, 1), ("v2_7opt_R", V, 2, 0x7F, 1), ("v2_7opt_T", V, 2, 0x7F, 0),
            ("v2_x55_R", V, 2, 0x55, 1)]
    if not full:
        grid = grid[:1] + grid[6:7] + grid[10:11]
    out = {"us_fused_unfused": {}, "zero_frac_v4_5opt_R": {}}    # microseconds: [fused, unfused]
    layer = ConvLayer(device, HEAD)
    for name, mode, n, mask, rnd in grid:
        p = sparq.SparqParams(mode, n, mask, rnd)
        f, _, _ = GraphTimer(layer.fused(p), steps, warmup).run()
        u, _, _ = GraphTimer(layer.unfused(p), steps, warmup).run()
        out["us_fused_unfused"][name] = [round(f * 1e3, 1), round(u * 1e3, 1)]
    none, _, _ = GraphTimer(layer.fused(sparq.SparqParams(sparq.MODE_NONE)), steps, warmup).run()
    out["none_us"] = round(none * 1e3, 2)
    del layer
    p = sparq.SparqParams(V, 4, 0x1F, 1)
    for zf in (0.0, 0.25, 0.5, 0.75, 0.9):
        L = dict(HEAD, zf=zf, seed=520 + int(zf * 100))
        layer = ConvLayer(device, L)
        f, _, _ = GraphTimer(layer.fused(p), steps, warmup).run()
        u, _, _ = GraphTimer(layer.unfused(p), steps, warmup).run()
        out["zero_frac_v4_5opt_R"][str(zf)] = [round(f * 1e3, 1), round(u * 1e3, 1)]
        del layer
    sparq.sparq_check()
    return out


def sweep_section(device, pk, mma, clk, steps=10, detail=False, only=None):
    """ResNet-50 sweep, batch 64, every conv shape (22 shapes, 52 instances), fused vSPARQ n = 4
    5opt +R with requantization.  Each layer against its own floor max(ops / tensor peak,
    bytes / measured copy bandwidth)."""
    import torch
    import paper_2105_11010_b200 as sparq
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
    peak_tops = mma["mac_per_clk_sm"] * mma["sms"] * 2 * (clk or 1965.0) * 1e6 / 1e12 if mma else pk["bf16"] * 2
    layers, total_ms, total_ops, total_floor = [], 0.0, 0, 0.0
    for li, S in enumerate(synth.resnet50_conv_layers()):
        zf = float(np.random.default_rng(100 + li).uniform(0.3, 0.7))
        L = dict(nb=64, h=S.h, w=S.w, c=S.cin, cout=S.cout, r=S.r, s=S.s, stride=S.stride, pad=S.pad, zf=zf, seed=100 + li)
        if only and only not in f"{S.h}x{S.w}x{S.cin}->{S.cout} {S.r}x{S.s}/s{S.stride}":
            continue
        layer = ConvLayer(device, L)
        ms, _, _ = GraphTimer(layer.fused(p), steps, 3).run(25.0)
        ops, nbytes = ops_of(L), sum(bytes_of(L))
        floor = max(ops / (peak_tops * 1e12), nbytes / (pk["hbm"] * 1e9)) * 1e3
        layers.append({"layer": f"{S.h}x{S.w}x{S.cin}->{S.cout} {S.r}x{S.s}/s{S.stride}", "count": S.count,
                       "us": round(ms * 1e3, 2), "tops": round(ops / ms / 1e9, 1), "floor_us": round(floor * 1e3, 2),
                       "frac_of_floor": round(floor / ms, 3)})
        total_ms += ms * S.count
        total_ops += ops * S.count
        total_floor += floor * S.count
        del layer
        torch.cuda.empty_cache()
    sparq.sparq_check()
    tops = total_ops / total_ms / 1e9
    worst = sorted(layers, key=lambda d: d["frac_of_floor"])[:3]
    out = {"ms_per_pass": round(total_ms, 4), "tops": round(tops, 1), "frac_of_int8_peak": round(tops / peak_tops, 4),
           "floor_ms_per_pass": round(total_floor, 4),
           "worst3": [[d["layer"], d["us"], d["floor_us"]] for d in worst]}
    if detail:
        out["layers"] = layers
    return out


def head_cpu_baseline(budget_s: float = 10.0):
    """The oracle as it stands on the host cores: whole passes over the full 128-image batch of
    the headline layer (transform, direct convolution, epilogue) until `budget_s` has gone by."""
    import oracle
    L = HEAD
    x = synth.activations(L["seed"], (L["nb"], L["h"], L["w"], L["c"]), L["zf"], stream=10)
    wt = synth.weights(L["seed"], (L["cout"], L["r"], L["s"], L["c"]))
    scale, bias = synth.scales(L["seed"], L["cout"]), synth.bias(L["seed"], L["cout"])
    inv = synth.inv_out_scale(L["r"] * L["s"] * L["c"], L["zf"])
    passes = 0
    t0 = time.perf_counter()
    while True:
        acc = oracle.conv2d_nhwc(x, wt, (1, 1), (1, 1), oracle.MODE_VSPARQ, 4, 0x1F, 1)
        oracle.epilogue(acc, scale, bias, True, inv)
        passes += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or passes >= 64:
            break
    return passes * ops_of(L) / dt / 1e12, dt, passes, oracle.num_threads()


def reference_step(images: int):
    import oracle
    L = HEAD
    x = synth.activations(L["seed"], (images, L["h"], L["w"], L["c"]), L["zf"], stream=10)
    wt = synth.weights(L["seed"], (L["cout"], L["r"], L["s"], L["c"]))
    scale, bias = synth.scales(L["seed"], L["cout"]), synth.bias(L["seed"], L["cout"])
    inv = synth.inv_out_scale(L["r"] * L["s"] * L["c"], L["zf"])
    t0 = time.perf_counter()
    acc = oracle.conv2d_nhwc(x, wt, (1, 1), (1, 1), oracle.MODE_VSPARQ, 4, 0x1F, 1)
    oracle.epilogue(acc, scale, bias, True, inv)
    return time.perf_counter() - t0, oracle.num_threads()


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """The slowest rank's time: every rank times the same K steps on its own shard, and the
    job is as slow as its slowest replica.  Works on any initialized process group (NCCL on
    GPUs, gloo in the CPU tests)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ms_per_step: float, world: int) -> float:
    """Weak scaling: each of the `world` replicas does one full workload per step."""
    return world * ops_of(HEAD) / (ms_per_step * 1e-3) / 1e12


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    images = 8
    for _ in range(args.warmup):
        reference_step(images)
    total, cores = 0.0, 1
    for _ in range(args.steps):
        dt, cores = reference_step(images)
        total += dt
    ops = 2 * images * HEAD["h"] * HEAD["w"] * HEAD["cout"] * 9 * HEAD["c"]
    value = args.steps * ops / total / 1e12
    sample = f"{images} of {HEAD['nb']} images per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": "CPU oracle, " + sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


SECTIONS = ["main", "transform", "pack", "frontend", "sparse24", "layer1x1", "mma_peak", "cfg1", "cfg2", "cfg5", "sweep"]


def main():
    global MIN_TIMED_MS
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="headline only")
    ap.add_argument("--full", action="store_true", help="also the codec, front-end and 2:4 sections, and per-layer sweep detail")
    ap.add_argument("--section", default="main", choices=SECTIONS,
                    help="print one section in full instead of the headline line (small runs for profiling)")
    ap.add_argument("--log2n", type=int, default=28, help="activations for the streaming sections (2^log2n)")
    ap.add_argument("--only", default=None, help="with --section sweep: only the layers whose name contains this text")
    ap.add_argument("--min-ms", type=float, default=MIN_TIMED_MS,
                    help="device time each graph-timed figure covers at least (lower it for profiler runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    MIN_TIMED_MS = args.min_ms
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2105_11010_b200 as sparq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SPARQ library has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()

    sync = torch.cuda.synchronize
    pk = peaks()
    VS = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
    if args.section != "main":
        sec = args.section
        if sec == "transform":
            res = transform_section(device, pk, 1 << args.log2n, args.steps, args.warmup)
        elif sec == "pack":
            res = pack_section(device, pk, 1 << args.log2n, args.steps, args.warmup)
        elif sec == "frontend":
            res = frontend_section(device, pk, 1 << args.log2n, args.steps, args.warmup)
        elif sec == "sparse24":
            res = sparse24_section(device, pk, args.steps, args.warmup)
        elif sec == "layer1x1":
            res = layer1x1_section(device, pk, args.steps, args.warmup)
        elif sec == "mma_peak":
            res = mma_peak_section(device)
        elif sec == "cfg1":
            res = cfg1_section(device)
        elif sec == "cfg5":
            res = cfg5_section(device, args.steps, args.warmup)
        elif sec == "sweep":
            res = sweep_section(device, pk, mma_peak_section(device), None, args.steps, detail=True, only=args.only)
        else:   # cfg2
            layer = ConvLayer(device, RN18, sets=20, host_recipe=True)
            ms, _, _ = GraphTimer(layer.fused(VS), args.steps, args.warmup).run()
            sparq.sparq_check()
            res = {"us": round(ms * 1e3, 2), "tops": round(ops_of(RN18) / ms / 1e9, 1)}
        print(json.dumps(res))
        return

    mma = mma_peak_section(device)
    layer = ConvLayer(device, HEAD, host_recipe=True)
    step = layer.fused(VS)
    timer = GraphTimer(step, args.steps, args.warmup)
    sparq.sparq_check()
    sampler = ClockSampler(local)
    sampler.start()
    ms_step, timed_ms, replays = timer.run(MIN_TIMED_MS, barrier)
    # keep the same load running a little longer so that the 50 ms sampler has samples under it
    t_end = time.time() + 0.4
    while time.time() < t_end:
        timer.graph.replay()
        sync()
    clocks = sampler.stop()
    # the same K steps enqueued one by one from Python (launch-bound on small layers)
    eager_ms_step = time_region(step, args.steps, 0, sync) / args.steps
    sparq.sparq_check()
    ms_step = max_over_ranks(ms_step, world, device)
    value = whole_job_tops(ms_step, world)

    # end to end: pinned host input -> device -> fused kernel -> uint8 result back on the host
    L = HEAD
    in_b, out_b, w_b = bytes_of(L)
    x_host = torch.from_numpy(synth.activations(L["seed"], (L["nb"], L["h"], L["w"], L["c"]), L["zf"], stream=10)).pin_memory()
    y_host = torch.empty((L["nb"], L["h"], L["w"], L["cout"]), dtype=torch.uint8).pin_memory()

    def e2e_step():
        sparq.sparq_conv2d_nhwc_s8_host(x_host, layer.wt, (1, 1), (1, 1), VS, scale=layer.scale, bias=layer.bias,
                                        relu=True, inv_out_scale=layer.inv, u8_out=y_host)
    e2e_steps = max(10, min(args.steps, 100))
    for _ in range(3):
        e2e_step()
    sync(); barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(e2e_steps):
        e2e_step()
    f1.record()
    sync(); barrier()
    e2e_ms = max_over_ranks(f0.elapsed_time(f1), world, device)
    e2e_value = whole_job_tops(e2e_ms / e2e_steps, world)

    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 6), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {
            "workload": WORKLOAD,
            "global_batch": L["nb"] * world,
            "l2": f"{layer.sets} rotating in/out sets, {layer.sets * (in_b + out_b) >> 20} MiB > 126 MiB L2",
            "parallelism": f"replicas x{world}",
            "timing": f"median of {replays} graph replays of K steps ({timed_ms:.0f} ms)",
            "eager_ms_per_step": round(eager_ms_step, 5),
        },
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"]},
        "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": in_b, "d2h_bytes_per_step": out_b,
                "steps": e2e_steps},
        "gpu_launches": args.steps * replays,
        "roofline": roofline_tensor(ops_of(L), ms_step, mma, pk, clocks["sm_mhz"], TRAFFIC["head"],
                                    "sparq_conv_window_kernel<128,128,VSPARQ,4,round,resident>", in_b + out_b + w_b),
    }
    if rank == 0 and world == 1:
        tops, dt, passes, cores = head_cpu_baseline()
        line["cpu_baseline"] = {"value": round(tops, 5), "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{passes} passes over the full {L['nb']}-image batch, {dt:.1f} s"}
        if not args.no_extras:
            del layer, timer
            torch.cuda.empty_cache()
            ex = {"mma_peak_mac_per_clk_sm": {k: mma[k]["mac_per_clk_sm"] for k in ("n64", "n128", "n256")}}
            ex["cfg1_gemm_256x576x64"] = cfg1_section(device)
            rn = ConvLayer(device, RN18, sets=20, host_recipe=True)
            ms2, _, _ = GraphTimer(rn.fused(VS), args.steps, 3).run()
            r2 = roofline_tensor(ops_of(RN18), ms2, mma, pk, clocks["sm_mhz"], TRAFFIC["rn18"], "", sum(bytes_of(RN18)))
            ex["cfg2_resnet18_conv"] = {"us": round(ms2 * 1e3, 2), "tops": r2["achieved"], "frac": r2["frac"],
                                        "traffic": r2["traffic"]}
            del rn
            torch.cuda.empty_cache()
            ex["cfg3_resnet50_b64"] = sweep_section(device, pk, mma, clocks["sm_mhz"], 10, detail=args.full)
            tr = transform_section(device, pk, 1 << 30, 20, 3)
            ex["cfg4_transform_2p30"] = {m: {"ms": tr[m]["ms"], "gbs": tr[m]["gbs"], "frac_of_copy": tr[m]["roofline"]["frac"],
                                             "frac_of_8000": tr[m]["roofline"]["frac_of_nominal_8000"]} for m in ("bsparq", "vsparq")}
            ex["cfg4_transform_2p30"].update(bound="hbm", peak_gbs=pk["hbm"], traffic=tr["bsparq"]["roofline"]["traffic"])
            ex["cfg5_ablation"] = cfg5_section(device, 20, 3, full=True)
            if args.full:
                ex["packed_stream_2p28"] = pack_section(device, pk, 1 << 28, 20, 3)
                ex["minmax_frontend_2p28"] = frontend_section(device, pk, 1 << 28, 20, 3)
                ex["sparse24_vsparq"] = sparse24_section(device, pk, 20, 3)
                ex["gemm_layer1x1"] = layer1x1_section(device, pk, 20, 3)
            line["extra"] = ex
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
