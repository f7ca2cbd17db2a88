#!/usr/bin/env python
"""Benchmark of the MXInt linear-layer hot path (arXiv 2307.15517) on B200.

One *step* = the whole hot path over one batch of synthetic input: for each of the four
OPT-1.3B-shaped prefill linears (2048 tokens; 2048->6144, 2048->2048, 2048->8192, 8192->2048;
MXInt4, block 16) the activations are quantized on the fly and multiplied with the layer's
pre-quantized weights (``mx_linear`` of the C ABI).  Weights are quantized once before the timed
region (they are static at inference); activations are quantized in every step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  ``value`` = effective TOPS (2*M*N*K summed over the four layers and all
ranks / device time of the steps).  With N > 1 (torchrun) every rank runs the same step on its own
token batch: independent problems, no data-path collective, weak scaling.
``--impl reference`` times the plain CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mx_linear_effective_tops"
UNIT = "TOPS"
WORKLOAD = "opt-1.3b prefill linears, 2048 tokens, MXInt4 block 16 (4 layers per step)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, averaged over the four launches of a step, from the
# ncu captures summarised under profiles/ (gemm_tc_kernel_opt13b_prefill.md, launch_list_bench.md)
GEMM_TC_DRAM_BYTES_PER_LAUNCH = 48.1e6
PREP_DRAM_BYTES_PER_LAUNCH = 38.9e6
# Dense bf16 tensor throughput of one SM per clock (tcgen05, 128x256x16 per 128 clocks): 8192 flop.
# SMs x this x the SM clock sampled during the timed region = the hardware bound the fractions below use
# beside the measured rate of the vendor's GEMM (which itself runs power-capped near 1.35 GHz).
TENSOR_FLOP_PER_CLK_PER_SM = 8192


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------ clocks sampler
class ClockSampler:
    """Polls NVML (SM clock, power, clock-event reasons) from a thread while the timed region
    runs; read-only queries, nothing on the GPU is changed."""
    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"),
               (0x4, "sw_power_cap"))

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.samples = []
        self.stop_flag = False
        self.thread = None
        self.sm_max = None
        self.error = None

    def _run(self, nv, handle):
        while not self.stop_flag:
            try:
                clk = nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(handle)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(handle)
                self.samples.append((clk, int(mask)))
            except Exception as e:                      # keep the benchmark alive
                self.error = repr(e)
                return
            time.sleep(0.002)

    def start(self):
        try:
            import threading

            import pynvml as nv
            nv.nvmlInit()
            handle = nv.nvmlDeviceGetHandleByUUID(self.uuid)
            self.sm_max = nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM)
            self.thread = threading.Thread(target=self._run, args=(nv, handle), daemon=True)
            self.thread.start()
        except Exception as e:
            self.error = repr(e)

    def stop(self):
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "samples": 0,
                    "reasons": ["no samples: %s" % self.error]}
        clocks = [c for c, _ in self.samples]
        reasons = sorted({name for _, m in self.samples for bit, name in self.REASONS if m & bit})
        return {"sm_mhz": statistics.median(clocks), "sm_min_mhz": min(clocks),
                "sm_max_mhz": self.sm_max, "samples": len(clocks), "reasons": reasons}


# ------------------------------------------------------------------------------ workload
def layer_flops(tokens, spec):
    return 2.0 * tokens * spec.N * spec.K


N_SETS = 3      # rotating input/weight/output sets: ~450 MB each, together far beyond the L2


def build_device_workload(mxb, synth, torch, seed):
    """Per layer: fp32 activations (device + pinned host copy), pre-quantized weights, output."""
    layers = []
    for li, spec in enumerate(synth.opt13b_prefill_layers()):
        x, w, _ = synth.opt13b_inputs(li, seed=seed)
        fa, fw = mxb.MxFormat(spec.block, spec.w_act), mxb.MxFormat(spec.block, spec.w_wgt)
        w_mant, w_exp = mxb.mx_quantize(w.cuda(), fw)
        xd = x.cuda()
        y = torch.empty((x.shape[0], spec.N), dtype=torch.float32, device="cuda")
        ws = mxb.alloc_workspace(mxb.mx_workspace_bytes(x.shape[0], spec.N, spec.K, fa, fw))
        M = x.shape[0]
        layers.append(dict(spec=spec, fa=fa, fw=fw, x=xd, x_host=x.pin_memory(), w_mant=w_mant,
                           w_exp=w_exp, y=y, ws=ws,
                           y_host=torch.empty((M, spec.N), dtype=torch.float32).pin_memory(),
                           # the same layer with an MXInt8 result (blocks of `block` along N)
                           fy=mxb.MxFormat(spec.block, 8),
                           yq_mant=torch.empty((M, spec.N), dtype=torch.uint8, device="cuda"),
                           yq_exp=torch.empty((M, spec.N // spec.block), dtype=torch.uint8, device="cuda"),
                           yq_mant_host=torch.empty((M, spec.N), dtype=torch.uint8).pin_memory(),
                           yq_exp_host=torch.empty((M, spec.N // spec.block), dtype=torch.uint8).pin_memory()))
    torch.cuda.synchronize()
    return layers


def run_step(mxb, layers):
    for L in layers:
        mxb.mx_linear(L["x"], L["fa"], L["w_mant"], L["w_exp"], L["fw"], L["spec"].N, y=L["y"],
                      workspace=L["ws"])


def run_step_q(mxb, layers):
    """The same four layers with the result quantized in the product's epilogue (MXInt8, same block)."""
    for L in layers:
        mxb.mx_linear_q(L["x"], L["fa"], L["w_mant"], L["w_exp"], L["fw"], L["spec"].N, L["fy"],
                        y_mant=L["yq_mant"], y_exp=L["yq_exp"], workspace=L["ws"])


class E2EPipeline:
    """The end-to-end leg: every layer's activations come from pinned host memory and every result
    goes back to pinned host memory, every step.  Three streams -- host-to-device copies, the
    library calls, device-to-host copies -- are chained per layer by events, so the two PCIe
    directions and the kernels overlap; a buffer is only rewritten after its last reader is done."""

    def __init__(self, torch):
        self.torch = torch
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream() for _ in range(3))

    def begin(self):
        cur = self.torch.cuda.current_stream()
        for st in (self.s_in, self.s_run, self.s_out):
            st.wait_stream(cur)

    def end(self):
        cur = self.torch.cuda.current_stream()
        for st in (self.s_in, self.s_run, self.s_out):
            cur.wait_stream(st)

    def step(self, mxb, layers, quantized=False):
        """quantized: the layer returns MXInt8 (mx_linear_q) and only its packed bytes go back to the host."""
        torch = self.torch
        for L in layers:
            with torch.cuda.stream(self.s_in):
                if "ev_run" in L:
                    self.s_in.wait_event(L["ev_run"])        # the product that last read x has finished
                L["x"].copy_(L["x_host"], non_blocking=True)
                L["ev_in"] = self.s_in.record_event()
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(L["ev_in"])
                if "ev_out" in L:
                    self.s_run.wait_event(L["ev_out"])       # y's previous contents have reached the host
                if quantized:
                    mxb.mx_linear_q(L["x"], L["fa"], L["w_mant"], L["w_exp"], L["fw"], L["spec"].N, L["fy"],
                                    y_mant=L["yq_mant"], y_exp=L["yq_exp"], workspace=L["ws"], stream=self.s_run)
                else:
                    mxb.mx_linear(L["x"], L["fa"], L["w_mant"], L["w_exp"], L["fw"], L["spec"].N, y=L["y"],
                                  workspace=L["ws"], stream=self.s_run)
                L["ev_run"] = self.s_run.record_event()
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(L["ev_run"])
                if quantized:
                    L["yq_mant_host"].copy_(L["yq_mant"], non_blocking=True)
                    L["yq_exp_host"].copy_(L["yq_exp"], non_blocking=True)
                else:
                    L["y_host"].copy_(L["y"], non_blocking=True)
                L["ev_out"] = self.s_out.record_event()


# ------------------------------------------------------------------------------ secondary metrics
def decode_sweep(mxb, synth, torch, hbm_gbs, iters=10):
    """Decode-shaped sweep: token batches 1/4/16 against 32 layers' worth of weight matrices
    (4 x 4096->4096 and 2 x 4096->11008 per layer, MXInt4 block 32, pre-quantized; activations fp32,
    quantized to MXInt8 inside the call), one grouped launch.  GB/s counts the packed weight bytes
    (mantissas + exponent bytes) that have to be streamed, nothing else."""
    fw = mxb.MxFormat(synth.DECODE_SPEC["block"], synth.DECODE_SPEC["w_wgt"])
    fa = mxb.MxFormat(synth.DECODE_SPEC["block"], synth.DECODE_SPEC["w_act"])
    g = torch.Generator(device="cuda")
    g.manual_seed(1234)
    mats = []
    for layer in range(synth.DECODE_LAYERS):
        for _, K, N in synth.decode_layer_shapes():
            w = torch.randn(N, K, generator=g, device="cuda", dtype=torch.float32) * 0.02
            mats.append((K, N) + tuple(mxb.mx_quantize(w, fw)))
            del w
    wbytes = sum(m[2].numel() + m[3].numel() for m in mats)
    out = {"weight_bytes": wbytes, "matrices": len(mats)}
    per_layer = len(synth.decode_layer_shapes())
    for T in synth.DECODE_TOKEN_BATCHES:
        xs = [synth.decode_activations(T, 4096, seed=l).cuda() for l in range(synth.DECODE_LAYERS)]
        layers = [dict(x=xs[i // per_layer], fa=fa, fw=fw, N=N, w_mant=wm, w_exp=we,
                       y=torch.empty(T, N, device="cuda")) for i, (K, N, wm, we) in enumerate(mats)]
        args = mxb.make_linear_args(layers)
        ws = mxb.alloc_workspace(mxb.mx_linear_grouped_workspace_bytes(args))
        for _ in range(3):
            mxb.mx_linear_grouped(args, ws)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            mxb.mx_linear_grouped(args, ws)
        b.record()
        torch.cuda.synchronize()
        ms_call = a.elapsed_time(b) / iters
        # the same calls again with the library's per-kernel events (they add gaps between launches)
        mxb.mx_profile_begin()
        for _ in range(iters):
            mxb.mx_linear_grouped(args, ws)
        torch.cuda.synchronize()
        prof = mxb.mx_profile_end()
        ms_kernel = prof["gemm_stream"][0] / iters
        out["tokens_%d" % T] = {
            "ms_per_call": ms_call, "gbs_call": wbytes / ms_call / 1e6,
            "ms_stream_kernel": ms_kernel, "gbs_stream_kernel": wbytes / ms_kernel / 1e6,
            "frac_hbm_stream_kernel": wbytes / ms_kernel / 1e6 / hbm_gbs,
            "frac_hbm_call": wbytes / ms_call / 1e6 / hbm_gbs, "launches_per_call": sum(n for _, n in prof.values()) / iters}
    return out


def llama7b_rate(mxb, synth, torch, iters=10):
    """The seven LLaMA-7B-shaped linears at 4096 tokens with the per-layer widths and block sizes drawn
    for seed 0 (mean width about 4 bits), Student-t activations: one pass = seven mx_linear calls.
    Inputs, weights and outputs of a pass take ~1.2 GB, far beyond the L2."""
    layers = []
    for li, spec in enumerate(synth.llama7b_mixed_layers(0)):
        x, w = synth.llama7b_inputs(spec, li, seed=0)
        fa, fw = mxb.MxFormat(spec.block, spec.w_act), mxb.MxFormat(spec.block, spec.w_wgt)
        wm, we = mxb.mx_quantize(w.cuda(), fw)
        M = x.shape[0]
        layers.append(dict(spec=spec, fa=fa, fw=fw, x=x.cuda(), wm=wm, we=we,
                           y=torch.empty((M, spec.N), dtype=torch.float32, device="cuda"),
                           ws=mxb.alloc_workspace(mxb.mx_workspace_bytes(M, spec.N, spec.K, fa, fw))))
        del x, w

    def one_pass():
        for L in layers:
            mxb.mx_linear(L["x"], L["fa"], L["wm"], L["we"], L["fw"], L["spec"].N, y=L["y"], workspace=L["ws"])

    for _ in range(2):
        one_pass()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        one_pass()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / iters
    mxb.mx_profile_begin()
    for _ in range(iters):
        one_pass()
    torch.cuda.synchronize()
    prof = mxb.mx_profile_end()
    flops = sum(2.0 * L["x"].shape[0] * L["spec"].N * L["spec"].K for L in layers)
    gemm_ms = prof["gemm_tc"][0] / iters
    return {"ms_per_pass": ms, "tops": flops / ms / 1e9, "flops": flops,
            "gemm_ms_per_pass": gemm_ms, "gemm_tflops": flops / gemm_ms / 1e9,
            "layers": [[L["spec"].name, L["spec"].K, L["spec"].N, L["spec"].block, L["spec"].w_act, L["spec"].w_wgt]
                       for L in layers]}


def block_scaled_rate(mxb, synth, torch, peak_bf16, iters=10):
    """The LLaMA-7B-shaped layers of the seed-0 draw that the hardware's block-scaled tensor-core path holds
    exactly (block 32, both widths <= 5): mx_linear with MX_ALGO_TCGEN05_MXF8 beside the default bf16 path.
    The roofline of the 8-bit path is the bf16 peak times the nominal fp8 : bf16 ratio of 2."""
    out = {"layers": []}
    for li, spec in enumerate(synth.llama7b_mixed_layers(0)):
        if spec.block != 32 or spec.w_act > 5 or spec.w_wgt > 5 or spec.K % 128:
            continue
        x, w = synth.llama7b_inputs(spec, li, seed=0)
        fa, fw = mxb.MxFormat(spec.block, spec.w_act), mxb.MxFormat(spec.block, spec.w_wgt)
        wm, we = mxb.mx_quantize(w.cuda(), fw)
        xd = x.cuda()
        M = x.shape[0]
        y = torch.empty((M, spec.N), dtype=torch.float32, device="cuda")
        flops = 2.0 * M * spec.N * spec.K
        rec = {"name": spec.name, "K": spec.K, "N": spec.N, "w_act": spec.w_act, "w_wgt": spec.w_wgt}
        for key, algo in (("bf16_path", mxb.MX_ALGO_AUTO), ("mxf8_path", mxb.MX_ALGO_TCGEN05_MXF8)):
            ws = mxb.alloc_workspace(mxb.mx_workspace_bytes_ex(M, spec.N, spec.K, fa, fw, algo))
            for _ in range(3):
                mxb.mx_linear(xd, fa, wm, we, fw, spec.N, y=y, workspace=ws, algo=algo)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(iters):
                mxb.mx_linear(xd, fa, wm, we, fw, spec.N, y=y, workspace=ws, algo=algo)
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / iters
            mxb.mx_profile_begin()
            for _ in range(iters):
                mxb.mx_linear(xd, fa, wm, we, fw, spec.N, y=y, workspace=ws, algo=algo)
            torch.cuda.synchronize()
            gemm_ms = mxb.mx_profile_end()["gemm_tc"][0] / iters
            rec[key] = {"ms_per_call": ms, "tops": flops / ms / 1e9, "gemm_ms": gemm_ms, "gemm_tflops": flops / gemm_ms / 1e9}
        rec["mxf8_path"]["gemm_frac_of_2x_bf16_burst"] = rec["mxf8_path"]["gemm_tflops"] / (2.0 * peak_bf16)
        out["layers"].append(rec)
        del x, w, xd, wm, we, y
    return out


def single_layer_latency(mxb, synth, torch, iters=200):
    """The single 128 x 768 x 768 MXInt4/B16 layer (151 MFLOP: latency-bound, two launches)."""
    x, w, spec = synth.single_layer(0)
    fa, fw = mxb.MxFormat(spec.block, spec.w_act), mxb.MxFormat(spec.block, spec.w_wgt)
    xd = x.cuda()
    wm, we = mxb.mx_quantize(w.cuda(), fw)
    y = torch.empty((x.shape[0], spec.N), dtype=torch.float32, device="cuda")
    ws = mxb.alloc_workspace(mxb.mx_workspace_bytes(x.shape[0], spec.N, spec.K, fa, fw))
    for _ in range(10):
        mxb.mx_linear(xd, fa, wm, we, fw, spec.N, y=y, workspace=ws)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        mxb.mx_linear(xd, fa, wm, we, fw, spec.N, y=y, workspace=ws)
    b.record()
    torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / iters
    return {"us_per_call": us, "tops": 2.0 * x.shape[0] * spec.N * spec.K / us / 1e6,
            "note": "back-to-back calls on one stream, operands L2-resident; a roofline fraction is not meaningful here"}


def quantize_rate(mxb, torch, hbm_gbs, iters=20):
    """Quantizer throughput on activation-sized tensors (fp32 in, packed MXInt4/B16 out):
    algorithmic bytes = 4 read + 0.5 + 1/16 written per element."""
    out = {}
    for rows, K in ((2048, 8192), (16384, 8192)):
        xs = [torch.randn(rows, K, device="cuda") for _ in range(3)]       # rotate: inputs beyond L2
        f = mxb.MxFormat(16, 4)
        mant = torch.empty(rows, K // 2, dtype=torch.uint8, device="cuda")
        ex = torch.empty(rows, K // 16, dtype=torch.uint8, device="cuda")
        for i in range(3):
            mxb.mx_quantize(xs[i], f, mant, ex)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(iters):
            mxb.mx_quantize(xs[i % 3], f, mant, ex)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / iters
        gbs = rows * K * (4 + 0.5 + 1 / 16) / ms / 1e6
        out["%dx%d" % (rows, K)] = {"ms": ms, "gbs": gbs, "frac_hbm": gbs / hbm_gbs}
    return out


def decoder_block_rate(mxb, synth, torch, iters=5):
    """One full decoder block in MX at OPT-6.7B shapes (hidden 4096, 32 heads x 128, FFN 16384,
    sequence 2048): six linears (A8/W4/B16), Q K^T and P V per head (A8/A8/B16), fp32 glue."""
    from paper_2307_15517_b200 import decoder_block as db
    sh = synth.decoder_block_shapes()
    cfg = db.BlockConfig(hidden=sh["hidden"], heads=sh["heads"], head_dim=sh["head_dim"], ffn=sh["ffn"],
                         block=sh["block"], w_act=sh["w_act"], w_wgt=sh["w_wgt"])
    seq, hid, ffn = sh["seq"], sh["hidden"], sh["ffn"]
    g = torch.Generator(device="cuda")
    g.manual_seed(77)
    rnd = lambda *shape: torch.randn(*shape, generator=g, device="cuda", dtype=torch.float32)
    qw = db.quantize_weights(cfg, {n: rnd(o, i) * 0.02 for n, o, i in
                                   (("wq", hid, hid), ("wk", hid, hid), ("wv", hid, hid), ("wo", hid, hid),
                                    ("w1", ffn, hid), ("w2", hid, ffn))})
    params = {n: rnd(sz) * 0.02 for n, sz in (("bq", hid), ("bk", hid), ("bv", hid), ("bo", hid), ("b1", ffn),
                                              ("b2", hid), ("ln1_b", hid), ("ln2_b", hid))}
    params["ln1_g"] = torch.ones(hid, device="cuda")
    params["ln2_g"] = torch.ones(hid, device="cuda")
    params = db.prepare_params(params)
    x = synth.outlier_activations(seq, hid, 4, -(-hid * 5 // 1000), 40.0).cuda()
    for _ in range(2):
        db.run(cfg, x, qw, params)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        db.run(cfg, x, qw, params)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / iters
    # once more with every launch bracketed by events (per-kind durations; the brackets serialise launches
    # that otherwise overlap as programmatic dependents, so these do not add up to `ms`)
    mxb.mx_profile_begin()
    for _ in range(iters):
        db.run(cfg, x, qw, params)
    torch.cuda.synchronize()
    prof = mxb.mx_profile_end()
    fl = db.flops(cfg, seq)
    return {"ms_per_block": ms, "tops": fl / ms / 1e9, "flops": fl,
            "kernels_ms": {k: v[0] / iters for k, v in prof.items() if v[1]},
            "launches": sum(v[1] for v in prof.values()) / iters,
            "note": "nominal flops of the block (both attention products counted in full; the fused kernel skips "
                    "the masked key tiles of the causal rows and computes the score tiles twice); includes torch "
                    "allocations of the intermediates; gemm_tc includes the fused attention kernel"}


# ------------------------------------------------------------------------------ oracle (CPU)
def oracle_inputs(orc, synth, sample_rows):
    """Untimed set-up: the first `sample_rows` tokens of every layer and its quantized weights."""
    out = []
    for li, spec in enumerate(synth.opt13b_prefill_layers()):
        x, w, _ = synth.opt13b_inputs(li, seed=0)
        qw, ew, _ = orc.quantize(w.numpy(), spec.block, spec.w_wgt)
        out.append(dict(spec=spec, x=x[:sample_rows].contiguous().numpy(), qw=qw, ew=ew))
    return out


def oracle_step(orc, inputs):
    """One pass of the hot path on the CPU: quantize the sampled activations, then the
    block-scaled product against the full weights.  Returns (seconds, operations)."""
    t_total, macs = 0.0, 0
    for L in inputs:
        spec = L["spec"]
        t0 = time.perf_counter()
        qa, ea, _ = orc.quantize(L["x"], spec.block, spec.w_act)
        orc.gemm(qa, ea, spec.w_act, L["qw"], L["ew"], spec.w_wgt, spec.block)
        t_total += time.perf_counter() - t0
        macs += L["x"].shape[0] * spec.N * spec.K
    return t_total, 2.0 * macs


def cpu_baseline(sample_rows=2048):
    from oracle import mx_oracle as orc
    from paper_2307_15517_b200 import synth
    t, ops = oracle_step(orc, oracle_inputs(orc, synth, sample_rows))
    return {"value": ops / t / 1e12, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
            "sample": "first %d of 2048 tokens of each of the 4 layers, all output columns, "
                      "one pass, %.1f s of CPU time" % (sample_rows, t)}


def run_reference(args):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import mx_oracle as orc
    from paper_2307_15517_b200 import synth
    rows = 64
    inputs = oracle_inputs(orc, synth, rows)
    for _ in range(max(args.warmup, 1)):
        oracle_step(orc, inputs)
    t, ops = 0.0, 0.0
    for _ in range(args.steps):
        dt, o = oracle_step(orc, inputs)
        t += dt
        ops += o
    value = ops / t / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64/f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": "first %d tokens of each layer per step" % rows},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
                         "sample": "first %d of 2048 tokens of each of the 4 layers per step" % rows},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------ multi-rank bookkeeping
def rank_seed(rank: int, set_index: int) -> int:
    """Every rank works on its own token batches: distinct seeds per (rank, rotating set)."""
    return N_SETS * rank + set_index


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of `values` (a list of floats) over all ranks of the default group;
    the identity when no process group is up.  The slowest rank defines the job's time."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_tops(world: int, flops_per_rank_step: float, steps: int, ms_total: float) -> float:
    """Whole-job throughput: every rank does the same work on its own batch (weak scaling)."""
    return world * flops_per_rank_step * steps / (ms_total * 1e-3) / 1e12


# ------------------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2307_15517_b200 import binding as mxb
    from paper_2307_15517_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the MXInt kernels have no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks, peaks_kind = load_peaks()
    # Step i works on set i % N_SETS (own activations, weights, workspace and outputs), so what a
    # step reads was last touched N_SETS steps ago and has long left the 126 MB L2.
    sets = [build_device_workload(mxb, synth, torch, seed=rank_seed(rank, i)) for i in range(N_SETS)]
    layers = sets[0]
    tokens = synth.OPT13B_TOKENS
    flops_step = sum(layer_flops(tokens, L["spec"]) for L in layers)
    h2d = sum(L["x_host"].numel() * 4 for L in layers)
    d2h = sum(L["y_host"].numel() * 4 for L in layers)
    d2h_q = sum(L["yq_mant_host"].numel() + L["yq_exp_host"].numel() for L in layers)
    layer_list = [[L["spec"].name, L["spec"].K, L["spec"].N] for L in layers]
    counter = [0]

    def next_set():
        counter[0] += 1
        return sets[counter[0] % N_SETS]

    def timed_steps(step_fn, steps, profile):
        """One event pair around `steps` back-to-back steps on the current stream.  With `profile`
        the library also brackets each of its kernel launches with events (per-kernel durations);
        those extra event records cost stream time, so that pass is never the one `value` comes from."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if profile:
            mxb.mx_profile_begin()
        a.record()
        for _ in range(steps):
            step_fn(mxb, next_set())
        b.record()
        torch.cuda.synchronize()
        prof = mxb.mx_profile_end() if profile else None
        return a.elapsed_time(b), prof

    # ---- device-resident timing ----
    for _ in range(args.warmup):
        run_step(mxb, next_set())
    assert mxb.mx_poll_status() == 0, "device status after warm-up"
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid))
    barrier()
    if rank == 0:
        sampler.start()
    ms_total, _ = timed_steps(run_step, args.steps, profile=False)
    barrier()
    # the same steps once more with every kernel launch bracketed by events: per-kernel durations
    ms_instr, prof = timed_steps(run_step, args.steps, profile=True)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    assert mxb.mx_poll_status() == 0, "device status after the timed region"

    # ---- end to end: pinned host inputs in, results out, every step ----
    ms_e2e = ms_e2e_q = float("nan")
    if not args.skip_e2e:
        pipe = E2EPipeline(torch)
        pipe.begin()
        for _ in range(2):
            pipe.step(mxb, next_set())
        pipe.end()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()                       # on the current stream; the three pipeline streams start behind it
        pipe.begin()
        for _ in range(args.steps):
            pipe.step(mxb, next_set())
        pipe.end()                       # ... and the current stream waits for all three before the end event
        b.record()
        torch.cuda.synchronize()
        ms_e2e = a.elapsed_time(b)
        barrier()
        # the same leg with the layer's own result type: MXInt8 mantissas + exponent bytes go back, not fp32
        for L in (L for S in sets for L in S):
            L.pop("ev_run", None), L.pop("ev_out", None), L.pop("ev_in", None)
        pipe.begin()
        for _ in range(2):
            pipe.step(mxb, next_set(), quantized=True)
        pipe.end()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        pipe.begin()
        for _ in range(args.steps):
            pipe.step(mxb, next_set(), quantized=True)
        pipe.end()
        b.record()
        torch.cuda.synchronize()
        ms_e2e_q = a.elapsed_time(b)
        barrier()

    secondary = None
    linear_q = None
    if world == 1 and not args.skip_secondary:          # single-GPU runs only
        # the prefill step once more with MXInt8 results instead of fp32 (no fp32 Y is written)
        for _ in range(3):
            run_step_q(mxb, next_set())
        torch.cuda.synchronize()
        ms_q, _ = timed_steps(run_step_q, args.steps, profile=False)
        linear_q = {"ms_per_step": ms_q / args.steps, "tops": flops_step * args.steps / (ms_q * 1e-3) / 1e12,
                    "result": "MXInt8, blocks of 16 along N, written by the product's epilogue"}
        # ... and with the paper's own block shape: activations MXInt((16,2),8,7), weights MXInt((16,2),8,3)
        for S in sets:
            for L in S:
                b = L["spec"].block
                L["fa2"], L["fw2"] = mxb.MxFormat(b, 8, 8, 2), mxb.MxFormat(b, 4, 8, 2)
                w_hat = mxb.mx_dequantize(L["w_mant"], L["w_exp"], L["spec"].K, L["fw"])
                L["w2_mant"], L["w2_exp"] = mxb.mx_quantize(w_hat, L["fw2"])
                del w_hat

        def run_step_2d(mxb_, layers_):
            for L in layers_:
                mxb_.mx_linear(L["x"], L["fa2"], L["w2_mant"], L["w2_exp"], L["fw2"], L["spec"].N, y=L["y"],
                               workspace=L["ws"])

        for _ in range(3):
            run_step_2d(mxb, next_set())
        torch.cuda.synchronize()
        ms_2d, _ = timed_steps(run_step_2d, args.steps, profile=False)
        block_16x2 = {"ms_per_step": ms_2d / args.steps, "tops": flops_step * args.steps / (ms_2d * 1e-3) / 1e12,
                      "formats": "activations MXInt((16,2),8,7), weights MXInt((16,2),8,3): two-row blocks"}
        # ... and with one tensor-memory accumulator per block (bit-identical to the sequential fp32 sum)
        def run_step_bw(mxb_, layers_):
            for L in layers_:
                mxb_.mx_linear(L["x"], L["fa"], L["w_mant"], L["w_exp"], L["fw"], L["spec"].N, y=L["y"],
                               workspace=L["ws"], algo=mxb_.MX_ALGO_TCGEN05_BLOCKWISE)

        for _ in range(3):
            run_step_bw(mxb, next_set())
        torch.cuda.synchronize()
        ms_bw, _ = timed_steps(run_step_bw, args.steps, profile=False)
        blockwise = {"ms_per_step": ms_bw / args.steps, "tops": flops_step * args.steps / (ms_bw * 1e-3) / 1e12,
                     "algo": "MX_ALGO_TCGEN05_BLOCKWISE: exact block sums, fp32 block adds in ascending order"}
        del sets, layers
        torch.cuda.empty_cache()
        secondary = {"linear_q": linear_q, "block_16x2": block_16x2, "blockwise": blockwise,
                     "decode_sweep": decode_sweep(mxb, synth, torch, peaks["hbm_gbs"]),
                     "quantize": quantize_rate(mxb, torch, peaks["hbm_gbs"]),
                     "single_layer": single_layer_latency(mxb, synth, torch),
                     "llama7b_mixed": llama7b_rate(mxb, synth, torch),
                     "block_scaled": block_scaled_rate(mxb, synth, torch, peaks["bf16_tflops"]),
                     "decoder_block": decoder_block_rate(mxb, synth, torch),
                     "hbm_peak_gbs": peaks["hbm_gbs"], "peak_kind": peaks_kind}
        # every configuration's whole call against the vendor-GEMM rate (tensor-bound ones)
        for key in ("linear_q", "block_16x2", "blockwise", "llama7b_mixed", "decoder_block"):
            secondary[key]["frac_of_bf16_burst"] = secondary[key]["tops"] / peaks["bf16_tflops"]
        secondary["llama7b_mixed"]["gemm_frac_of_bf16_burst"] = secondary["llama7b_mixed"]["gemm_tflops"] / peaks["bf16_tflops"]
        assert mxb.mx_poll_status() == 0, "device status after the secondary metrics"
    barrier()

    ms_total, ms_e2e, ms_e2e_q = max_over_ranks([ms_total, ms_e2e, ms_e2e_q], dist, device="cuda")

    if rank == 0:
        value = aggregate_tops(world, flops_step, args.steps, ms_total)
        e2e_value = aggregate_tops(world, flops_step, args.steps, ms_e2e)
        e2e_q_value = aggregate_tops(world, flops_step, args.steps, ms_e2e_q)
        gemm_ms, gemm_n = prof["gemm_tc"]
        achieved = flops_step * args.steps / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
        peak = peaks["bf16_tflops"]          # burst figure: the timed region lasts well under a second
        # hardware bound at the clock this run actually had: SMs x 8192 flop per clock x sampled SM MHz
        sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
        mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        peak_clock = sms * TENSOR_FLOP_PER_CLK_PER_SM * mhz * 1e6 / 1e12
        per_gpu = value / world
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 (exact MXInt decode) x bf16 -> f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens_per_gpu": tokens,
                       "layers": layer_list,
                       "weights": "pre-quantized once outside the timed region",
                       "l2": "inputs larger than L2: %d rotating sets of activations, weights, workspace "
                             "and outputs (~450 MB each); one CUDA event pair around the K steps" % N_SETS,
                       "parallelism": "replicas over token batches (no collective)"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps,
                    "note": "pinned host X in and fp32 Y out for every layer of every step; copies in both "
                            "directions and the kernels run on three event-chained streams (PCIe-bound)",
                    "mxint8_results": {"value": e2e_q_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                                       "d2h_bytes_per_step": d2h_q, "ms_per_step": ms_e2e_q / args.steps,
                                       "note": "the same leg through mx_linear_q: the layer's MXInt8 result "
                                               "(mantissas + exponent bytes) goes back instead of fp32"}},
            "gpu_launches": sum(n for _, n in prof.values()),
            "gpu_launches_note": "counted by the library over an instrumented repeat of the K timed steps",
            "kernels": {k: {"ms_per_step": ms / args.steps, "launches_per_step": n / args.steps}
                        for k, (ms, n) in prof.items() if n},
            "kernels_note": "per-kernel CUDA events over an instrumented repeat of the same K steps "
                            "(%.4f ms per step with the extra event records in the stream)" % (ms_instr / args.steps),
            "roofline": {"bound": "tensor", "kernel": "gemm_tc2_kernel / gemm_tc_kernel", "achieved": achieved,
                         "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_kind": "rate of the vendor's bf16 GEMM (burst), %s" % peaks_kind,
                         "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                         # the bound the silicon sets at the clock sampled during the timed region
                         "peak_clock_derived": peak_clock, "frac_of_clock_derived_peak": achieved / peak_clock,
                         "clock_derived_note": "%d SMs x %d flop/clk x %.0f MHz (median sampled under load)"
                                               % (sms, TENSOR_FLOP_PER_CLK_PER_SM, mhz),
                         "traffic": GEMM_TC_DRAM_BYTES_PER_LAUNCH,
                         "algorithmic_flops_per_launch": flops_step / 4.0,
                         # the whole call (operand preparation + product) against the same peaks
                         "call": {"achieved": per_gpu, "frac": per_gpu / peak,
                                  "frac_of_sustained_peak": per_gpu / peaks["bf16_tflops_sustained"],
                                  "frac_of_clock_derived_peak": per_gpu / peak_clock,
                                  "traffic_per_step": None if PREP_DRAM_BYTES_PER_LAUNCH is None else
                                  4 * (GEMM_TC_DRAM_BYTES_PER_LAUNCH + PREP_DRAM_BYTES_PER_LAUNCH)}},
            "secondary": secondary,
            "cpu_baseline": None if args.skip_cpu_baseline else cpu_baseline(),
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--skip-cpu-baseline", action="store_true",
                    help="leave the CPU oracle timing out (profiler runs)")
    ap.add_argument("--skip-e2e", action="store_true", help="leave the host-buffer leg out")
    ap.add_argument("--skip-secondary", action="store_true",
                    help="leave the decode sweep and the quantizer rate out")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
