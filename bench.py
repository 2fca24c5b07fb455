#!/usr/bin/env python
"""Benchmark of the melded FP8-LoRA hot path on B200.

Workload (one "step"): forward, backward and row-wise proxy update of the seven linear layers of one
LLaMA-7B decoder layer (q, k, v, o 4096->4096; gate, up 4096->11008; down 11008->4096) at 4096 tokens,
rank 64, top-256 rows per matrix -- synthetic seeded inputs with 1% outlier channels.  The metric is
the algorithmic fwd+bwd FLOP rate 2T[n(m+r) + mn + mr] summed over the matrices, divided by the time
of the whole step (quantization of X, dY, O_A and the proxy update are inside the timed region, their
arithmetic is not counted as useful FLOPs).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line.  N > 1 (under torchrun) runs independent replicas, one per GPU (the path has no
exchange step); the reported value is the aggregate over ranks with the max-over-ranks time.
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_24061_b200 import synth  # noqa: E402

METRIC = "melded FP8-LoRA layer fwd+bwd TFLOP/s (7B projection set, T=4096, r=64)"
UNIT = "TFLOP/s"
FP8_OVER_BF16 = 2.0        # nominal dense FP8 : bf16 tensor throughput on B200 (4.5 : 2.25 PFLOP/s)
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one forward and one dX launch of gemm_fp8_pair_kernel, measured with ncu on
# the three projection shapes of the workload, in bytes:
GEMM_DRAM_BYTES = {   # (n, m): (forward, dX)
    (4096, 4096): (33950976 + 2122240, 33630720 + 351488),
    (4096, 11008): (62336256 + 53340160, 136442624 + 18720512),
    (11008, 4096): (139000064 + 23043328, 62110720 + 49093120),
}


def layer_flops(T, n, m, r):
    """Algorithmic FLOPs of one fwd+bwd of one matrix: forward 2Tn(m+r), dX 2Tmn, dB 2Tmr."""
    return 2.0 * T * (n * (m + r) + m * n + m * r)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            d = json.load(fh)
        return dict(bf16_sustained=float(d["bf16_tflops_sustained"]), bf16_burst=float(d["bf16_tflops"]),
                    hbm=float(d["hbm_gbs"]), source="measured")
    except Exception:
        return dict(bf16_sustained=FALLBACK_BF16_TFLOPS * 1.4 / 1.59, bf16_burst=FALLBACK_BF16_TFLOPS,
                    hbm=FALLBACK_HBM_GBS, source="fallback")


class ClockSampler:
    """Samples SM clock, power and clock-event reasons of one GPU every 10 ms on a host thread (NVML; reading only), each
    sample stamped with the host clock, so that every timed pass gets the record of its own window."""
    REASONS = [("hw_slowdown", "nvmlClocksEventReasonHwSlowdown"), ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown"),
               ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown"), ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap")]

    def __init__(self, cuda_index: int, period_s: float = 0.01):
        self.cuda_index, self.period = cuda_index, period_s
        self.samples = []          # (t, sm_mhz, power_w, reason bits)
        self.sm_max = None
        self._stop = threading.Event()
        self.thread = None
        self.error = None

    def _handle(self, nv):
        try:
            uuid = str(torch.cuda.get_device_properties(self.cuda_index).uuid)
            return nv.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
        except Exception:
            return nv.nvmlDeviceGetHandleByIndex(self.cuda_index)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = self._handle(nv)
            self.sm_max = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            masks = [(name, getattr(nv, attr)) for name, attr in self.REASONS]
        except Exception as exc:      # no NVML: the record says so
            self.error = f"NVML unavailable: {exc}"
            return

        def pump():
            while not self._stop.is_set():
                try:
                    sm = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                    pw = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                    self.samples.append((time.perf_counter(), sm, pw, tuple(name for name, m in masks if bits & m)))
                except Exception as exc:
                    self.error = str(exc)
                    return
                time.sleep(self.period)
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    @staticmethod
    def now():
        return time.perf_counter()

    def window(self, t0: float, t1: float):
        """Record of the samples taken between two host times (the caller synchronizes the device at both)."""
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": [self.error or "no sampler"]}
        rows = [r for r in self.samples if t0 <= r[0] <= t1]
        reasons = sorted({name for r in rows for name in r[3]})
        return {"sm_mhz": statistics.median(r[1] for r in rows) if rows else None, "sm_max_mhz": self.sm_max,
                "power_w_max": max((r[2] for r in rows), default=None), "samples": len(rows), "seconds": round(t1 - t0, 4),
                "reasons": reasons}

    def stop(self):
        self._stop.set()
        if self.thread is not None:
            self.thread.join(timeout=2)
        if self.samples:
            return self.window(self.samples[0][0], self.samples[-1][0])
        return self.window(0.0, 0.0)


def aggregate_over_ranks(ms_local: float, flops_per_rank: float, dist=None, device=None):
    """Replica aggregation: every rank runs its own batch; the job's time is the slowest rank's (max-reduce of the
    device-timed milliseconds), the job's work is the sum over ranks.  Returns (ms, TFLOP/s of the whole job)."""
    world = 1
    ms = float(ms_local)
    if dist is not None and dist.is_initialized():
        world = dist.get_world_size()
        t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return ms, world * flops_per_rank / (ms * 1e-3) / 1e12


def build_workload(fq, device, seed, T, r, k, linears, outlier_frac, per_row=False, heavy_tailed=False, flags=0):
    layers = []
    for idx, (name, n, m) in enumerate(linears):
        W = synth.backbone(seed, idx, m, n, device, heavy_tailed=heavy_tailed)
        A = synth.adapter_a(seed, idx, r, n, device)
        B = synth.adapter_b(seed, idx, m, r, device)
        layer = fq.setup_layer(W, A, B, 1.0, per_row=per_row)
        layer.flags = flags
        del W
        X = synth.activations(seed, idx, T, n, round(outlier_frac * n), device)
        dY = synth.out_grad(seed, idx, 0, T, m, device)
        out_f = (torch.empty((T, m), dtype=torch.bfloat16, device=device),
                 torch.empty((T, r), dtype=torch.float32, device=device),
                 torch.empty(1, dtype=torch.float32, device=device), torch.empty(1, dtype=torch.float32, device=device))
        out_b = (torch.empty((T, n), dtype=torch.bfloat16, device=device),
                 torch.empty((m, r), dtype=torch.float32, device=device), torch.empty(1, dtype=torch.float32, device=device))
        idx_out = torch.empty(k, dtype=torch.int32, device=device)
        layers.append(dict(name=name, n=n, m=m, layer=layer, X=X, dY=dY, out_f=out_f, out_b=out_b, idx=idx_out,
                           ws=layer.workspace(T)))
    return layers


def run_step_fused_update(fq, layers, lr, k, batch):
    """The step with Alg. 3 line 4 and the row scores inside the adapter-gradient kernel (falqon_melded_backward_update) and
    one batched selection + merge (falqon_proxy_update_scored_batched)."""
    for L in layers:
        _, OA, amax_oa, _ = fq.melded_forward(L["layer"], L["X"], ws=L["ws"], out=L["out_f"])
        fq.melded_backward_update(L["layer"], L["dY"], OA, amax_oa, lr, ws=L["ws"], out=L["out_b"])
    batch.run_scored()


def run_step_exact_merge(fq, layers, lr, k, batch):
    """The step with the correctly rounded tensor-core merge for the whole projection set in one batched call
    (falqon_proxy_update_batched_exact, the bf16 copy of every layer's A~ prepared once at set-up)."""
    for L in layers:
        _, OA, amax_oa, _ = fq.melded_forward(L["layer"], L["X"], ws=L["ws"], out=L["out_f"])
        fq.melded_backward(L["layer"], L["dY"], OA, amax_oa, ws=L["ws"], out=L["out_b"])
    batch.run_exact(lr)


def run_step(fq, layers, lr, k, batch=None):
    """Forward and backward of every projection, and the proxy update of each: one batched call for the whole set
    (batch: a ProxyBatch over the layers' gradient buffers), or one call per projection when batch is None."""
    for L in layers:
        _, OA, amax_oa, _ = fq.melded_forward(L["layer"], L["X"], ws=L["ws"], out=L["out_f"])
        _, dB, _ = fq.melded_backward(L["layer"], L["dY"], OA, amax_oa, ws=L["ws"], out=L["out_b"])
        if batch is None:
            fq.proxy_update(L["layer"], dB, lr, k, ws=L["ws"], idx_out=L["idx"])
    if batch is not None:
        batch.run(lr)


def make_proxy_batch(fq, layers, k):
    return fq.ProxyBatch([L["layer"] for L in layers], [L["out_b"][1] for L in layers], [k] * len(layers),
                         wss=[L["ws"] for L in layers], idx_outs=[L["idx"] for L in layers])


def run_step_e2e(fq, layers, host, lr, k, pipe, batch=None):
    """Same step, but every input starts in pinned host memory and the results are read back.  The uploads run on a
    copy stream one projection ahead of the compute stream (each projection has its own device buffers; an event
    per projection says when its inputs have landed, another when the compute no longer reads them)."""
    compute = torch.cuda.current_stream()
    copy = pipe["copy_stream"]
    for i, (L, H) in enumerate(zip(layers, host)):
        with torch.cuda.stream(copy):
            copy.wait_event(pipe["consumed"][i])          # the previous step's kernels are done with these buffers
            L["X"].copy_(H["X"], non_blocking=True)
            L["dY"].copy_(H["dY"], non_blocking=True)
            pipe["landed"][i].record(copy)
    for i, (L, H) in enumerate(zip(layers, host)):
        compute.wait_event(pipe["landed"][i])
        _, OA, amax_oa, _ = fq.melded_forward(L["layer"], L["X"], ws=L["ws"], out=L["out_f"])
        _, dB, _ = fq.melded_backward(L["layer"], L["dY"], OA, amax_oa, ws=L["ws"], out=L["out_b"])
        pipe["consumed"][i].record(compute)
        if batch is None:
            fq.proxy_update(L["layer"], dB, lr, k, ws=L["ws"], idx_out=L["idx"])
        H["dB"].copy_(dB, non_blocking=True)
        if batch is None:
            H["idx"].copy_(L["idx"], non_blocking=True)
    if batch is not None:
        batch.run(lr)
        for L, H in zip(layers, host):
            H["idx"].copy_(L["idx"], non_blocking=True)


def make_e2e_pipe(n_layers):
    pipe = dict(copy_stream=torch.cuda.Stream(), landed=[torch.cuda.Event() for _ in range(n_layers)],
                consumed=[torch.cuda.Event() for _ in range(n_layers)])
    for ev in pipe["consumed"]:
        ev.record(torch.cuda.current_stream())
    return pipe


def time_oracle_sample(T_sample, r, k, lr, seed=0):
    """The CPU oracle, as it stands, on a token slice of the q projection (4096 -> 4096): quantize,
    forward, backward and proxy update.  Returns (TFLOP/s, seconds, threads, description)."""
    import numpy as np
    from oracle import falqon_oracle as orc
    n = m = 4096
    W = synth.backbone(seed, 0, m, n).float().numpy()
    A = synth.adapter_a(seed, 0, r, n).float().numpy()
    X = synth.activations(seed, 0, T_sample, n, round(0.01 * n)).float().numpy()
    dY = synth.out_grad(seed, 0, 0, T_sample, m).float().numpy()
    wq, s_w, dbuf = orc.setup_layer(W, A, None, 1.0)   # set-up is not timed (not on the per-step path)
    t0 = time.perf_counter()
    f = orc.layer_forward(X, wq, s_w, m, r)
    b = orc.layer_backward(dY, f["OA"], wq, s_w, m, r)
    orc.proxy_update(wq, dbuf, b["dB"].astype(np.float32), lr, k, m, r)
    dt = time.perf_counter() - t0
    flops = layer_flops(T_sample, n, m, r)
    desc = f"q projection 4096->4096, first {T_sample} of 4096 tokens, r={r}, top-{k}: quantize+fwd+bwd+proxy update"
    return flops / dt / 1e12, dt, orc.num_threads(), desc


def run_sweep(args):
    """configs[4]: 4096 -> 11008, rank x tokens x top-k.  Forward and backward depend on (rank, tokens), the proxy
    update on (rank, top-k); each is timed alone with CUDA events (warm L2 state of a step loop: the calls run back
    to back on one stream) and set against the FP8 tensor roofline or the HBM / fp32-ALU rooflines."""
    from paper_2510_24061_b200 import binding as fq
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    tensor_peak = peaks["bf16_burst"] * FP8_OVER_BF16          # kernels timed in isolation: burst figure
    n, m = 4096, 11008
    ranks = [8, 16, 32, 64, 128]
    tokens = [512, 2048, 8192, 32768]
    topks = [0, 64, 512, 4096]
    iters = 10

    def timed(fn, graph=True):
        """ms per call, calls back to back on one stream: as replays of a CUDA graph of the call (forward and backward:
        three to five kernels per call, timed without their launch gaps) or, for the proxy update and with --eager, as plain
        calls (its two kernels overlap from one call to the next under programmatic stream serialization, which separate
        graph launches do not allow: 24 against 43 us at top-64).  A first batch of calls sizes the run: at least 10 calls
        and about 20 ms, and the timed batch follows the warm one without a pause -- a call of 35 us timed ten times after
        an idle gap measures the clock ramp of the GPU, not the call."""
        for _ in range(3):
            fn()
        run = fn
        if graph and not args.eager:
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            run = g.replay
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters):
            run()
        e1.record()
        e1.synchronize()
        est = max(e0.elapsed_time(e1) / iters, 1e-3)
        n_timed = max(iters, min(2000, int(20.0 / est)))
        for _ in range(n_timed):          # warm batch, same length, no pause before the timed one
            run()
        e1.record()
        for _ in range(n_timed):
            run()
        e2.record()
        torch.cuda.synchronize()
        return e1.elapsed_time(e2) / n_timed

    W = synth.backbone(0, 4, m, n, dev)
    for r in ranks:
        A = synth.adapter_a(0, 4, r, n, dev)
        layer = fq.setup_layer(W, A, None, 1.0)
        for T in tokens:
            X = synth.activations(0, 4, T, n, round(0.01 * n), dev)
            dY = synth.out_grad(0, 4, 0, T, m, dev)
            ws = layer.workspace(T)
            out_f = (torch.empty((T, m), dtype=torch.bfloat16, device=dev), torch.empty((T, r), dtype=torch.float32, device=dev),
                     torch.empty(1, dtype=torch.float32, device=dev), torch.empty(1, dtype=torch.float32, device=dev))
            out_b = (torch.empty((T, n), dtype=torch.bfloat16, device=dev), torch.empty((m, r), dtype=torch.float32, device=dev),
                     torch.empty(1, dtype=torch.float32, device=dev))
            t_f = timed(lambda: fq.melded_forward(layer, X, ws=ws, out=out_f))
            _, OA, amax_oa, _ = out_f
            t_b = timed(lambda: fq.melded_backward(layer, dY, OA, amax_oa, ws=ws, out=out_b))
            f_f = 2.0 * T * n * (m + r)
            f_b = 2.0 * T * m * n + 2.0 * T * m * r
            print(json.dumps({"sweep": "fwd_bwd", "n": n, "m": m, "rank": r, "tokens": T,
                              "fwd_ms": t_f, "fwd_tflops": f_f / t_f / 1e9, "fwd_frac_tensor_peak": f_f / t_f / 1e9 / tensor_peak,
                              "bwd_ms": t_b, "bwd_tflops": f_b / t_b / 1e9, "bwd_frac_tensor_peak": f_b / t_b / 1e9 / tensor_peak,
                              "tensor_peak_tflops": tensor_peak}), flush=True)
            del X, dY, out_f, out_b, ws
            layer._ws = None
            torch.cuda.empty_cache()
        dB = synth.normal_bf16(0, 77, (m, r), 1e-3, dev).float()
        ws = layer.workspace(1)
        for k in topks:
            idx = torch.empty(max(k, 1), dtype=torch.int32, device=dev)
            t_p = timed(lambda: fq.proxy_update(layer, dB, 2e-4, k, ws=ws, idx_out=idx if k > 0 else None), graph=False)
            t_x = t_xp = None
            if k > 0:   # the same update with the correctly rounded merge on the tensor cores
                scratch = torch.empty(int(fq.lib.falqon_exact_merge_scratch_bytes(m, n, r)), dtype=torch.uint8, device=dev)
                t_x = timed(lambda: fq.proxy_update_exact(layer, dB, 2e-4, k, ws=ws, idx_out=idx, scratch=scratch, want_count=False), graph=False)
                del scratch
                one = fq.ProxyBatch([layer], [dB], [k], wss=[ws], idx_outs=[idx])
                one.prepare_exact()           # the bf16 copy of A~ built once: 4 launches per update instead of 6
                t_xp = timed(lambda: one.run_exact(2e-4), graph=False)
                del one
            bytes_p = 12.0 * m * r + 4.0 * m + k * (2.0 * n + 8.0 * r) + r * n   # optimizer+score pass, merged rows, A~ once
            fma = float(k) * n * r
            alu_peak = 148 * 128 * peaks_clock_ghz() * 1e9                    # fp32 fma per second
            print(json.dumps({"sweep": "proxy", "n": n, "m": m, "rank": r, "topk": k, "proxy_ms": t_p, "proxy_exact_merge_ms": t_x, "proxy_exact_merge_prepared_ms": t_xp,
                              "algorithmic_gbs": bytes_p / t_p / 1e6, "frac_hbm_peak": bytes_p / t_p / 1e6 / peaks["hbm"],
                              "merge_gfma_per_s": fma / t_p / 1e6, "frac_fp32_fma_peak": fma / (t_p * 1e-3) / alu_peak,
                              "hbm_peak_gbs": peaks["hbm"]}), flush=True)


def measure_tensor_ceiling(fq, seconds, fills, gpu_index=0):
    """Back-to-back launches of the MMA-issue-only kernel (the product kernels' 256 x 256 x 32 E4M3 instruction on
    operands resident in shared memory) for `seconds` per operand fill.  Per fill: the rate over the first ten launches
    (burst), over the last second (sustained, under the power cap) and over the whole run, with the clocks seen."""
    import time
    dev = torch.device("cuda", torch.cuda.current_device())
    sink = torch.zeros(4 * fq.tensor_ceiling_ctas(), dtype=torch.float32, device=dev)
    kblocks = 20000            # about 10 ms per launch
    out = {"kblocks_per_launch": kblocks, "seconds_per_fill": seconds, "ctas": fq.tensor_ceiling_ctas()}
    codes = {"zeros": 0, "uniform_codes": 1, "bell_shaped_codes": 2}
    traffic = None
    for name in fills:
        load_src = None
        if name.endswith("+operand_traffic"):     # 64 MB of codes (stays in L2), streamed into the operand slots
            if traffic is None:
                traffic = torch.randint(0, 120, (64 << 20,), dtype=torch.uint8, device=dev)
            load_src = traffic
        fill = codes[name.split("+")[0]]
        for _ in range(3):
            flops = fq.tensor_ceiling(kblocks, 1, fill, sink, load_src)
        torch.cuda.synchronize()
        time.sleep(1.0)        # let the power average settle before the burst figure
        sampler = ClockSampler(gpu_index)
        sampler.start()
        events = [torch.cuda.Event(enable_timing=True)]
        events[0].record()
        t0 = time.time()
        while time.time() - t0 < seconds:
            for _ in range(10):
                fq.tensor_ceiling(kblocks, 1, fill, sink, load_src)
            ev = torch.cuda.Event(enable_timing=True)
            ev.record()
            events.append(ev)
            ev.synchronize()
        clocks = sampler.stop()
        ms = [events[i].elapsed_time(events[i + 1]) for i in range(len(events) - 1)]     # each: 10 launches
        rate = lambda chunk: 10.0 * len(chunk) * flops / (sum(chunk) * 1e-3) / 1e12
        n_last = max(1, int(len(ms) * min(1.0, 1.0 / seconds)))
        out[name] = {"burst": rate(ms[:1]), "sustained": rate(ms[-n_last:]), "whole_run": rate(ms), "launches": 10 * len(ms),
                     "clocks": clocks}
    return out


def run_tensor_ceiling(args):
    """The FP8 tensor pipe with nothing else in the way, for zero operands, uniformly random codes and the codes of a
    bell-shaped variable under absmax scaling.  One JSON line."""
    from paper_2510_24061_b200 import binding as fq
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    out = {"metric": "FP8 tensor ceiling (tcgen05.mma kind::f8f6f4, 256x256x32 over CTA pairs, operands in shared memory)",
           "unit": "TFLOP/s",
           "bf16_x2_reference": {"burst": peaks["bf16_burst"] * FP8_OVER_BF16, "sustained": peaks["bf16_sustained"] * FP8_OVER_BF16,
                                 "source": peaks["source"]}, "nominal": 4500.0}
    out.update(measure_tensor_ceiling(fq, args.tensor_ceiling, ["zeros", "uniform_codes", "bell_shaped_codes",
                                                                  "bell_shaped_codes+operand_traffic"]))
    out["device_status"] = fq.last_device_status()
    print(json.dumps(out), flush=True)


def run_stack(args):
    """configs[2]: 32 decoder-shaped blocks of the 7B projection set, activations chained (see
    paper_2510_24061_b200/stack.py), one training step = forward through all blocks, backward, and each block's
    seven proxy updates right after its backward.  One JSON line: step ms, TFLOP/s over the algorithmic FLOP of the
    224 melded layers, both peak fractions, memory in use."""
    from paper_2510_24061_b200 import binding as fq
    from paper_2510_24061_b200 import stack as st
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = synth.config1()
    T, r, k, lr = cfg["T"], cfg["r"], cfg["k"], cfg["lr"]
    H, F, n_layers = 4096, 11008, args.stack_layers
    peaks = measured_peaks()
    stack = st.Stack(n_layers, H, F, T, r, k, seed=cfg["seed"], device=dev, lr=lr, producer_amax=not args.stack_own_absmax,
                     batched_proxy=not args.proxy_per_layer, fuse_chain=not args.stack_unfused_chain,
                     fuse_cast=not (args.stack_separate_casts or args.stack_own_absmax or args.stack_unfused_chain),
                     layer_flags=fq.LAYER_DB_OWN_KERNEL if args.own_db else 0,
                     adamw=dict(beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0) if args.stack_adamw else None)
    h0 = synth.normal_bf16(cfg["seed"], 9001, (T, H), 1.0, dev)
    G = synth.normal_bf16(cfg["seed"], 9002, (T, H), 1.0e-2, dev)
    steps, warmup = max(1, min(args.steps, 20)), max(3, min(args.warmup, 5))
    for _ in range(warmup):
        stack.step(h0, G)
    torch.cuda.synchronize()
    one_step = lambda: stack.step(h0, G)
    use_graph = not args.eager and not args.stack_adamw     # AdamW's step count is a call argument: not captured
    if use_graph:
        step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(step_graph):
            stack.step(h0, G)
        one_step = step_graph.replay
        for _ in range(2):
            one_step()
        torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def soak(run, seconds):     # the same loop for `seconds` right before a timed region: the clocks of a long job
        t0 = sampler.now()
        while sampler.now() - t0 < seconds:
            run()
            e1.record()
            e1.synchronize()
        return sampler.window(t0, sampler.now())

    def timed(run, n):
        torch.cuda.synchronize()
        t0 = sampler.now()
        e0.record()
        for _ in range(n):
            run()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n, sampler.window(t0, sampler.now())

    t_soak = sampler.now()
    clocks_soak = soak(one_step, args.soak)
    ms, clocks_timed = timed(one_step, steps)
    clocks = sampler.window(t_soak, sampler.now())
    clocks["soak_before"] = clocks_soak
    clocks["timed_steps_only"] = clocks_timed
    # forward alone and backward (+ updates) alone, same protocol
    ms_f, _ = timed(lambda: stack.forward(h0), steps)
    # where the step goes: the same step call by call with the library's stages bracketed by events (the brackets cost the
    # launch overlap, so this pass is slower); what the brackets do not cover is the chain between the layers
    eager = lambda: stack.step(h0, G)
    soak(eager, min(args.soak, 1.0))
    n_rec = 12 * 7 * n_layers * 2
    fq.profile_start(n_rec, None)
    ms_inst, clocks_inst = timed(eager, 2)
    recs = fq.profile_stop(n_rec)
    fam = {"products": 0.0, "casts": 0.0, "adapter_gradient": 0.0, "proxy_update": 0.0}
    names = {"gemm_fwd": "products", "gemm_dx": "products", "quant_x": "casts", "quant_dy": "casts", "quant_oa": "casts",
             "gemm_db": "adapter_gradient", "reduce_db": "adapter_gradient", "sgd_score": "proxy_update", "topk": "proxy_update",
             "merge": "proxy_update"}
    for name, t in recs:
        fam[names[name]] += t / 2.0
    fam["chain_kernels_and_gaps"] = max(ms_inst - sum(fam.values()), 0.0)
    shares = {k_: {"ms_per_step": round(v, 3), "share": round(v / ms_inst, 4)} for k_, v in fam.items()}
    f_products = stack.flops_per_step()
    products_tf = f_products / (fam["products"] * 1e-3) / 1e12 if fam["products"] > 0 else 0.0
    flops = stack.flops_per_step()
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms,
        "forward_ms": ms_f, "backward_and_updates_ms": ms - ms_f, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp8", "data": "synthetic",
        "config": {"workload": f"configs[2]: {n_layers} chained blocks of the LLaMA-7B projection set, tokens=4096, rank=64, "
                               "top-k=256, q/k/v and gate/up share one quantized input, bf16 chain kernels between the layers",
                   "tokens": T, "rank": r, "topk": k, "matrices": 7 * n_layers, "tflop_per_step": flops / 1e12,
                   "l2": "working set far larger than L2 (every step touches the whole stack)", "parallelism": "single GPU",
                   "optimizer": "AdamW on the DeltaBuffers" if args.stack_adamw else "SGD on the DeltaBuffers",
                   "proxy_update": "one call per projection" if args.proxy_per_layer else "one batched call per block",
                   "casts": ("inside the chain kernels that produce the tensors (two phases around a grid barrier)"
                             if stack.fuse_cast else "single-pass kernels of their own (the producing kernel hands over the absmax)"),
                   "launch": "replays of one CUDA graph of the step" if use_graph else "one library call after another"},
        "clocks": clocks, "gpu_launches": stack.launches_per_step() * steps,
        "regime": "sustained: %.1f s of the same step loop ran right before the timed steps" % args.soak,
        "frac_of_fp8_peak": {"of_measured_sustained_x2": tf / (peaks["bf16_sustained"] * FP8_OVER_BF16),
                             "of_nominal_4500": tf / 4500.0,
                             "target": "north_star: >= 0.60 of dense FP8 peak on this stack -- not met"},
        "where_the_step_goes": {"pass_ms_per_step": ms_inst, "clocks": clocks_inst, "families": shares,
                                "products_alone_tflops": products_tf,
                                "products_alone_frac_of_measured_sustained_x2": products_tf / (peaks["bf16_sustained"] * FP8_OVER_BF16),
                                "products_alone_frac_of_nominal_4500": products_tf / 4500.0,
                                "note": "call-by-call pass with the library's stages bracketed by CUDA events (slower than the "
                                        "graph replay above: no launch overlap across brackets); chain = what no bracket covers"},
        "memory": {"layers_bytes": stack.bytes_resident(), "allocated_bytes": torch.cuda.memory_allocated(dev),
                   "peak_allocated_bytes": torch.cuda.max_memory_allocated(dev)},
        "device_status": fq.last_device_status()}))


def peaks_clock_ghz():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["sm_max_mhz"]) / 1e3
    except Exception:
        return 1.965


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="falqon", choices=["falqon", "reference"])
    ap.add_argument("--oracle-tokens", type=int, default=4096,
                    help="token rows of the q projection the CPU oracle is timed on (4096 = the whole projection, 10-30 s of CPU work)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="configs[4]: sweep rank x tokens x top-k on the 4096->11008 projection; one JSON line per point")
    ap.add_argument("--stack", action="store_true",
                    help="configs[2]: the 32-block chained stack of the 7B projection set; one JSON line")
    ap.add_argument("--stack-layers", type=int, default=32)
    ap.add_argument("--stack-own-absmax", action="store_true",
                    help="with --stack: every layer takes the absmax of its input itself (the chain kernels do not hand it over)")
    ap.add_argument("--stack-unfused-chain", action="store_true",
                    help="with --stack: residual sums and the normalisations (or their gradients) that follow them as separate kernels")
    ap.add_argument("--stack-separate-casts", action="store_true",
                    help="with --stack: every cast is a kernel of its own (default: the casts run inside the chain kernels that "
                         "produce the tensors, all but those of the gated MLP's two gradients)")
    ap.add_argument("--own-db", action="store_true",
                    help="the adapter gradient as a kernel of its own (FALQON_LAYER_DB_OWN_KERNEL) instead of riding on the "
                         "input-gradient product's launch")
    ap.add_argument("--stack-adamw", action="store_true",
                    help="with --stack: AdamW (beta 0.9 / 0.999, eps 1e-8, no weight decay) on every DeltaBuffer instead of plain SGD")
    ap.add_argument("--config3", action="store_true",
                    help="configs[3] instead of configs[1]: the LLaMA-13B projection set, 8192 tokens, per-row-scaled "
                         "heavy-tailed backbone, top-512 (not the headline line)")
    ap.add_argument("--tensor-ceiling", type=float, default=0.0, metavar="SECONDS",
                    help="measure the FP8 tensor pipe alone (MMA issue on shared-memory operands) for SECONDS per fill; one JSON line")
    ap.add_argument("--no-tensor-ceiling", action="store_true",
                    help="skip the 3 s measurement of the FP8 tensor pipe alone that the default line reports beside the roofline")
    ap.add_argument("--eager", action="store_true",
                    help="time the step as one library call after another instead of as replays of one CUDA graph of the "
                         "step (the library's calls only enqueue kernels, so a step can be captured; replays are about 2 %% faster)")
    ap.add_argument("--proxy-per-layer", action="store_true",
                    help="run one falqon_proxy_update per projection instead of one falqon_proxy_update_batched per step")
    ap.add_argument("--exact-merge", action="store_true",
                    help="merge with the correctly rounded tensor-core merge, batched over the projection set "
                         "(falqon_proxy_update_batched_exact) -- a different rounding of the merged rows than the default fp32 chain")
    ap.add_argument("--fused-update", action="store_true",
                    help="run the optimizer step and the row scores inside the adapter-gradient kernel "
                         "(falqon_melded_backward_update + falqon_proxy_update_scored_batched)")
    ap.add_argument("--soak", type=float, default=2.0, metavar="SECONDS",
                    help="how long the step loop runs right before the timed steps, so that they see the clocks of a long job")
    ap.add_argument("--fused", action="store_true",
                    help="cast X and dY inside the producers of the tensor-core products (FALQON_LAYER_FUSED_CAST) instead of "
                         "in cast kernels of their own")
    ap.add_argument("--only", default=None, help="profiling aid: restrict the workload to one projection (q,k,v,o,gate,up,down)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = synth.config3() if args.config3 else synth.config1()
    T, r, k, lr = cfg["T"], cfg["r"], cfg["k"], cfg["lr"]
    linears = cfg["linears"]
    if args.only is not None:
        linears = [l for l in linears if l[0] == args.only]
    flops_step = sum(layer_flops(T, n, m, r) for _, n, m in linears)
    workload = {"workload": ("configs[3]: LLaMA-13B projection set (q,k,v,o,gate,up,down), tokens=8192, rank=64, top-k=512, "
                             "per-row-scaled heavy-tailed backbone" if args.config3 else
                             "configs[1]: LLaMA-7B projection set (q,k,v,o,gate,up,down), tokens=4096, rank=64, top-k=256")
                            + ("" if args.only is None else f" -- RESTRICTED to '{args.only}' (profiling aid, not a bench line)"),
                "tokens": T, "rank": r, "topk": k, "matrices": len(linears), "gflop_per_step": flops_step / 1e9,
                "l2": "inputs larger than L2 (%.2f GB of inputs and outputs touched per step)" %
                      (sum(2.0 * T * (n + m) * 2 for _, n, m in linears) / 1e9),
                "parallelism": f"replicas x{world}",
                "proxy_update": "one call per projection" if args.proxy_per_layer else "one batched call per step",
                "launch": "one library call after another" if args.eager else "replays of one CUDA graph of the step"}

    if args.tensor_ceiling > 0:
        if rank == 0:
            run_tensor_ceiling(args)
        return
    if args.sweep:
        if rank == 0:
            run_sweep(args)
        return
    if args.stack:
        if rank == 0:
            run_stack(args)
        return

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 3))
        for _ in range(min(args.warmup, 1)):
            time_oracle_sample(min(args.oracle_tokens, 64), r, k, lr)
        vals = [time_oracle_sample(args.oracle_tokens, r, k, lr) for _ in range(steps)]
        tf = statistics.mean(v[0] for v in vals)
        secs = statistics.mean(v[1] for v in vals)
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": secs * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8 (software E4M3/E5M2, fp64 accumulate)", "data": "synthetic",
            "config": workload,
            "cpu_baseline": {"value": tf, "unit": UNIT, "cores": vals[0][2], "kind": "oracle", "sample": vals[0][3]},
            "e2e": {"value": tf, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the melded FP8-LoRA path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2510_24061_b200 import binding as fq

    layers = build_workload(fq, device, cfg["seed"] + rank, T, r, k, linears, cfg["outlier_frac"],
                            per_row=cfg.get("per_row", False), heavy_tailed=cfg.get("heavy_tailed", False),
                            flags=(fq.LAYER_FUSED_CAST if args.fused else 0) | (fq.LAYER_DB_OWN_KERNEL if args.own_db else 0))
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return aggregate_over_ranks(ms, 0.0, dist, device)[0]

    batch = None if args.proxy_per_layer else make_proxy_batch(fq, layers, k)
    sampler = ClockSampler(local_rank)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(run, steps):
        """EXACTLY `steps` calls of run() between two events, a barrier and a device synchronize on both sides; returns
        (ms per step as the max over ranks, clock record of that window)."""
        barrier()
        t0 = sampler.now()
        ev0.record()
        for _ in range(steps):
            run()
        ev1.record()
        barrier()
        t1 = sampler.now()
        return max_over_ranks(ev0.elapsed_time(ev1)) / steps, sampler.window(t0, t1)

    def soak(run, seconds):
        """Runs run() back to back for at least `seconds` (device busy the whole time), so that what is timed next sees
        the clocks of a long job -- the board's power cap pulls the SM clock down within a second or so -- and not those
        of a GPU that has just been idle.  Returns the clock record of the soak."""
        t0 = sampler.now()
        while True:
            for _ in range(20):
                run()
            ev1.record()
            ev1.synchronize()
            if sampler.now() - t0 >= seconds:
                break
        return sampler.window(t0, sampler.now())

    def with_cycles(ms, clocks):
        """time x median SM clock of the pass: passes that ran at different clocks compare in cycles."""
        mhz = clocks.get("sm_mhz")
        return None if mhz is None else ms * mhz * 1e-3      # ms x MHz = thousand cycles; / 1000 = million SM cycles per step

    step_fn = run_step
    if args.fused_update:
        step_fn = lambda fq_, layers_, lr_, k_, batch_: run_step_fused_update(fq_, layers_, lr_, k_, batch_)
    if args.exact_merge:
        batch.prepare_exact()
        step_fn = lambda fq_, layers_, lr_, k_, batch_: run_step_exact_merge(fq_, layers_, lr_, k_, batch_)
    for _ in range(max(args.warmup, 3)):
        step_fn(fq, layers, lr, k, batch)
    barrier()
    one_step = lambda: step_fn(fq, layers, lr, k, batch)
    if not args.eager:
        step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(step_graph):
            step_fn(fq, layers, lr, k, batch)
        one_step = step_graph.replay
    for _ in range(max(args.warmup, 3)):      # the W warm-up steps proper, in the form that is timed
        one_step()

    # ---- burst: the first steps after an idle second (clocks at their maximum, power average still low)
    burst_steps = 20
    barrier()
    time.sleep(1.0)
    ms_burst, clocks_burst = timed(one_step, burst_steps)

    # ---- sustained (the headline): the same step loop for SOAK seconds first, then EXACTLY --steps steps
    t_soak = sampler.now()
    clocks_soak = soak(one_step, args.soak)
    ms_step, clocks_timed = timed(one_step, args.steps)
    clocks = sampler.window(t_soak, sampler.now())       # the soak and the timed steps: one continuous stretch of the same loop
    clocks["soak_before"] = clocks_soak
    clocks["timed_steps_only"] = clocks_timed
    value = world * flops_step / (ms_step * 1e-3) / 1e12
    # ---- the spread of single steps, right after the timed region (same regime): an event after every step
    n_spread = max(args.steps, 20)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_spread + 1)]
    marks[0].record()
    for i in range(n_spread):
        one_step()
        marks[i + 1].record()
    torch.cuda.synchronize()
    singles = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(n_spread))
    per_step = {"n": n_spread, "median_ms": singles[n_spread // 2], "min_ms": singles[0], "max_ms": singles[-1],
                "note": "this rank's steps one by one, an event after each, right after the timed region"}

    # ---- forward and backward alone (quantization included, no proxy update): the quantity the metric's name describes;
    # `value` above is the whole hot path, proxy update included
    def run_fwd_bwd():
        for L in layers:
            _, OA, amax_oa, _ = fq.melded_forward(L["layer"], L["X"], ws=L["ws"], out=L["out_f"])
            fq.melded_backward(L["layer"], L["dY"], OA, amax_oa, ws=L["ws"], out=L["out_b"])
    soak(run_fwd_bwd, min(args.soak, 1.0))
    ms_fwd_bwd, clocks_fwd_bwd = timed(run_fwd_bwd, args.steps)

    # ---- the same steps again, call by call, with EVERY stage bracketed by CUDA events on the launching stream (an event
    # between two kernels removes their launch overlap, so this pass is slower per step): after a soak of its own, so
    # that the kernel durations it records are those of the sustained regime too
    eager_step = lambda: step_fn(fq, layers, lr, k, batch)
    soak(eager_step, min(args.soak, 1.0))
    n_records = 12 * len(layers) * args.steps
    fq.profile_start(n_records, None)
    ms_step_instrumented, clocks_instrumented = timed(eager_step, args.steps)
    records = fq.profile_stop(n_records)
    # ---- for reference: the adapter gradient as a kernel of its own (the default runs it inside the dX launch, where it
    # has no duration of its own): the same instrumented steps with FALQON_LAYER_DB_OWN_KERNEL on every layer
    own_db_records = []
    if not args.own_db and not args.fused:
        for L in layers:
            L["layer"].flags |= fq.LAYER_DB_OWN_KERNEL
        for _ in range(3):
            eager_step()
        fq.profile_start(n_records, None)
        timed(eager_step, args.steps)
        own_db_records = fq.profile_stop(n_records)
        for L in layers:
            L["layer"].flags &= ~fq.LAYER_DB_OWN_KERNEL
    status = fq.last_device_status()
    sampler.stop()

    # ---- what one proxy update does to a backbone (bookkeeping outside every timed region, first projection):
    # codes that changed, and codes sitting at the largest finite magnitude (saturation of the requantized rows)
    L0 = layers[0]
    before = L0["layer"].wq[: L0["m"]].clone()
    _, OA0, amax0, _ = fq.melded_forward(L0["layer"], L0["X"], ws=L0["ws"], out=L0["out_f"])
    _, dB0, _ = fq.melded_backward(L0["layer"], L0["dY"], OA0, amax0, ws=L0["ws"], out=L0["out_b"])
    fq.proxy_update(L0["layer"], dB0, lr, k, ws=L0["ws"], idx_out=L0["idx"])
    after = L0["layer"].wq[: L0["m"]]
    rows = L0["idx"][:k].long()
    proxy_effect = {"projection": L0["name"], "rows_merged": int(k),
                    "changed_codes": int((before != after).sum().item()),
                    "changed_codes_outside_merged_rows": int((before != after).sum().item() - (before[rows] != after[rows]).sum().item()),
                    "saturated_codes_in_merged_rows": int(((after[rows] & 0x7F) == 0x7E).sum().item())}

    # ---- roofline of the dominant kernel: the tcgen05 FP8 GEMM in its two tensor-bound roles.  Its launches were timed
    # by the library's stage events inside the soaked, instrumented pass above, so the matching peak is the SUSTAINED one.
    peaks = measured_peaks()
    t_big = sum(ms for name, ms in records if name in ("gemm_fwd", "gemm_dx"))
    db_rides = not any(name == "gemm_db" for name, _ in records)      # the adapter gradient ran inside the dX launches
    f_big = args.steps * sum(2.0 * T * n * (m + r) + 2.0 * T * m * n + (2.0 * T * m * r if db_rides else 0.0) for _, n, m in linears)
    launches_big = sum(1 for name, _ in records if name in ("gemm_fwd", "gemm_dx"))
    achieved = f_big / (t_big * 1e-3) / 1e12 if t_big > 0 else 0.0
    peak = peaks["bf16_sustained"] * FP8_OVER_BF16
    gemm_name = "gemm_fp8_pair_fused_kernel" if args.fused else "gemm_fp8_pair_kernel"
    roofline = {"kernel": f"{gemm_name} (forward and input-gradient products)", "bound": "tensor",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "regime": "sustained: launch durations recorded by CUDA events on the launching stream inside a step loop that "
                          "had been running for %.1f s; clocks of that pass under instrumented_pass" % min(args.soak, 1.0),
                "peak_source": f"{peaks['source']} bf16 sustained x{FP8_OVER_BF16:g} (nominal FP8:bf16 ratio)",
                "frac_of_nominal_4500": achieved / 4500.0,
                "launches": launches_big, "avg_launch_ms": t_big / max(launches_big, 1),
                "gflop_per_launch": f_big / max(launches_big, 1) / 1e9,
                "traffic": (sum(sum(GEMM_DRAM_BYTES[(n, m)]) for _, n, m in linears) / (2.0 * len(linears))
                            if all((n, m) in GEMM_DRAM_BYTES for _, n, m in linears) and not args.fused else None),
                "traffic_note": "dram read+write bytes per average launch, from an ncu capture of the forward and the dX "
                                "launch of each projection shape (un-fused kernel); "
                                "algorithmic bytes per average launch: %.1f MB of FP8 operands + %.1f MB of bf16 / fp32 "
                                "outputs (an operand the preceding cast left in L2, or an output still in L2 when the "
                                "kernel ends, does not show up as DRAM traffic)" %
                                (sum((T * n + (m + r) * n) + (T * m + m * n) for _, n, m in linears) / (2.0 * len(linears)) / 1e6,
                                 sum((2 * T * m + 4 * T * r) + 2 * T * n for _, n, m in linears) / (2.0 * len(linears)) / 1e6)}

    # ---- stage breakdown of the same pass, and the HBM-bound stages against the measured copy rate
    breakdown = {}
    for name, ms in records:
        breakdown[name] = breakdown.get(name, 0.0) + ms / args.steps
    t_db = breakdown.get("gemm_db", 0.0)
    L2_BYTES = 126e6

    def cast_bytes(elems, per_elt_small, per_elt_large):
        return elems * (per_elt_small if 2.0 * elems <= L2_BYTES else per_elt_large)
    # un-fused: the tensor is read once from DRAM (2 B), its codes written (1 B); a tensor larger than L2 is read a second
    # time for the cast (5 B).  fused: only the absmax pass reads it (2 B).
    lo, hi = (2, 2) if args.fused else (3, 5)
    q_bytes = sum(cast_bytes(T * n, lo, hi) + cast_bytes(T * m, lo, hi) for _, n, m in linears)
    q_bytes_5 = sum(5.0 * T * (n + m) for _, n, m in linears)
    t_quant = (breakdown.get("quant_x", 0) + breakdown.get("quant_dy", 0)) * 1e-3
    quant_gbs = q_bytes / t_quant / 1e9 if t_quant > 0 else 0.0
    n_beyond_l2 = sum((2.0 * T * n > L2_BYTES) + (2.0 * T * m > L2_BYTES) for _, n, m in linears)
    quantize = {"bound": "hbm", "achieved_gbs": quant_gbs, "peak_gbs": peaks["hbm"], "frac": quant_gbs / peaks["hbm"],
                "frac_of_nominal_8000": quant_gbs / 8000.0, "ms_per_step": t_quant * 1e3,
                "bytes_per_elt": lo if n_beyond_l2 == 0 else f"{lo} for {2 * len(linears) - n_beyond_l2} tensors that fit L2, {hi} for {n_beyond_l2} beyond it",
                "bytes_per_step": q_bytes,
                "frac_if_counted_at_5_bytes_per_elt": (q_bytes_5 / t_quant / 1e9 / peaks["hbm"]) if t_quant > 0 and not args.fused else None,
                "note": ("absmax pass over X and dY (the casts run inside the products)" if args.fused else
                         "absmax + cast of X and dY in one kernel each: a tensor that fits L2 is read from DRAM once (2 B/elt) and its "
                         "codes written once (1 B/elt); beyond L2 (126 MB of bf16) the cast pass reads it again: 5 B/elt") +
                        "; the O_A cast rides in the same stage"}
    db_bytes = sum(T * m + T * r + 4.0 * m * r for _, n, m in linears)
    db = {"bound": "hbm", "kernel": "db_fused_kernel", "bytes_per_step": db_bytes, "ms_per_step": t_db,
          "achieved_gbs": db_bytes / (t_db * 1e-3) / 1e9 if t_db > 0 else 0.0, "peak_gbs": peaks["hbm"],
          "note": "reads g~ (T m bytes, written just before and largely still in L2) and O~_A, writes dB"}
    db["frac"] = db["achieved_gbs"] / peaks["hbm"]
    if db_rides:
        t_own = sum(ms for name, ms in own_db_records if name == "gemm_db") / args.steps
        t_dx_own = sum(ms for name, ms in own_db_records if name == "gemm_dx") / args.steps
        own = {"kernel": "db_fused_kernel", "ms_per_step": t_own, "achieved_gbs": db_bytes / (t_own * 1e-3) / 1e9 if t_own > 0 else None,
               "frac": db_bytes / (t_own * 1e-3) / 1e9 / peaks["hbm"] if t_own > 0 else None,
               "gemm_dx_ms_per_step_without_rider": t_dx_own, "gemm_dx_ms_per_step_with_rider": breakdown.get("gemm_dx", 0.0)}
        db = {"bound": "hbm", "kernel": "gemm_fp8_pair_kernel (rider of the input-gradient product)", "bytes_per_step": db_bytes,
              "ms_per_step": None, "achieved_gbs": None, "peak_gbs": peaks["hbm"], "frac": None, "as_a_kernel_of_its_own": own,
              "note": "dB is computed inside the launch of the input-gradient product, on the SM pairs its last wave of tiles leaves "
                      "idle: it has no launch and no duration of its own (its flops are counted in that kernel's roofline entry); "
                      "--own-db runs and times it as a kernel of its own"}
    t_proxy = breakdown.get("sgd_score", 0.0) + breakdown.get("merge", 0.0)
    proxy_bytes = sum(12.0 * m * r + 4.0 * m + k * (2.0 * n + 8.0 * r) + r * n for _, n, m in linears)
    proxy = {"bound": "hbm for the optimizer pass, fp32 ALU for the merge at this rank", "bytes_per_step": proxy_bytes,
             "ms_per_step": t_proxy, "achieved_gbs": proxy_bytes / (t_proxy * 1e-3) / 1e9 if t_proxy > 0 else 0.0,
             "peak_gbs": peaks["hbm"], "merge_fma_per_step": sum(float(k) * n * r for _, n, m in linears),
             "merge_frac_of_fp32_fma_peak": (sum(float(k) * n * r for _, n, m in linears) / (breakdown.get("merge", 0.0) * 1e-3) /
                                             (148 * 128 * peaks_clock_ghz() * 1e9)) if breakdown.get("merge", 0.0) > 0 else None}
    proxy["frac"] = proxy["achieved_gbs"] / peaks["hbm"]

    # ---- end to end: inputs in pinned host memory, results read back, every step
    host = []
    for L in layers:
        host.append(dict(X=L["X"].cpu().pin_memory(), dY=L["dY"].cpu().pin_memory(),
                         dB=torch.empty(L["out_b"][1].shape, dtype=torch.float32).pin_memory(),
                         idx=torch.empty(k, dtype=torch.int32).pin_memory()))
    h2d = sum(H["X"].numel() * 2 + H["dY"].numel() * 2 for H in host)
    d2h = sum(H["dB"].numel() * 4 + H["idx"].numel() * 4 for H in host)
    e2e_steps = max(3, min(args.steps, 20))
    pipe = make_e2e_pipe(len(layers))
    for _ in range(2):
        run_step_e2e(fq, layers, host, lr, k, pipe, batch)
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        run_step_e2e(fq, layers, host, lr, k, pipe, batch)
    ev1.record()
    barrier()
    ms_e2e = max_over_ranks(ev0.elapsed_time(ev1)) / e2e_steps
    e2e_value = world * flops_step / (ms_e2e * 1e-3) / 1e12

    suffix = ":fused" if args.fused else ""
    bsuffix = suffix if args.fused else (":own_db" if args.own_db else "")
    table_launches = 2 if cfg.get("per_row", False) else 0      # per-row-scaled layers: one small table of scale factors per call
    launches_per_step = sum(fq.launch_count("falqon_melded_forward" + suffix) + fq.launch_count("falqon_melded_backward" + bsuffix) +
                            table_launches +
                            (fq.launch_count("falqon_proxy_update", k=k) if batch is None else 0) for L in layers)
    if batch is not None:
        launches_per_step += fq.launch_count("falqon_proxy_update_batched", k=k) * ((len(layers) + 7) // 8)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if not args.no_cpu_baseline:
        tf, secs, threads, desc = time_oracle_sample(args.oracle_tokens, r, k, lr)
        cpu_baseline = {"value": tf, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                        "seconds": secs, "host_cpus": os.cpu_count()}

    # ---- the FP8 tensor pipe alone (rank 0 at N = 1 only; at N > 1 the other ranks would be idle and the board power differs)
    if not args.no_tensor_ceiling and world == 1:
        tc = measure_tensor_ceiling(fq, 3.0, ["bell_shaped_codes"], local_rank)
        ceiling = tc["bell_shaped_codes"]["sustained"]
        roofline["mma_only_ceiling"] = {
            "sustained": ceiling, "burst": tc["bell_shaped_codes"]["burst"], "unit": "TFLOP/s",
            "clocks": tc["bell_shaped_codes"]["clocks"], "frac": achieved / ceiling if ceiling > 0 else None,
            "note": "this GPU's tensor pipe issuing the products' own MMA on shared-memory operands (bell-shaped E4M3 codes) "
                    "for 3 s under the power cap: no loads, no epilogue; python bench.py --tensor-ceiling 3 gives all fills"}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_step, "mcycles_per_step": with_cycles(ms_step, clocks), "per_step": per_step,
        "regime": "sustained: %.1f s of the same step loop ran right before the timed steps" % args.soak,
        "burst": {"ms_per_step": ms_burst, "value": world * flops_step / (ms_burst * 1e-3) / 1e12, "unit": UNIT, "steps": burst_steps,
                  "mcycles_per_step": with_cycles(ms_burst, clocks_burst), "clocks": clocks_burst,
                  "note": "the first steps after one idle second: clocks at their maximum, the board not yet at its power cap"},
        "fwd_bwd_only": {"ms_per_step": ms_fwd_bwd, "value": world * flops_step / (ms_fwd_bwd * 1e-3) / 1e12, "unit": UNIT,
                         "mcycles_per_step": with_cycles(ms_fwd_bwd, clocks_fwd_bwd), "clocks": clocks_fwd_bwd,
                         "note": "forward + backward of the seven projections with their input casts, without the proxy update, "
                                 "call by call after a soak of its own"},
        "instrumented_pass": {"ms_per_step": ms_step_instrumented, "mcycles_per_step": with_cycles(ms_step_instrumented, clocks_instrumented),
                              "clocks": clocks_instrumented,
                              "note": "the step call by call with every stage bracketed by CUDA events (no launch overlap across the "
                                      "brackets); source of roofline, stage_ms_per_step, quantize, db and proxy_update"},
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8",
        "data": "synthetic", "config": workload, "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e, "steps": e2e_steps,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "frac_of_fp8_peak": {"of_measured_sustained_x2": value / world / peak, "of_nominal_4500": value / world / 4500.0,
                             "burst_of_measured_burst_x2": world * flops_step / (ms_burst * 1e-3) / 1e12 / world / (peaks["bf16_burst"] * FP8_OVER_BF16),
                             "note": "whole step (casts, dB and proxy update inside the time, only product FLOP counted)"},
        "stage_ms_per_step": {k_: round(v, 4) for k_, v in sorted(breakdown.items())},
        "quantize": quantize, "db": db, "proxy_update": proxy,
        "proxy_update_effect": proxy_effect,
        "device_status": status,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
