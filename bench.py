#!/usr/bin/env python
"""Benchmark of the W2A4 decode hot path on B200.

A step is one decode pass over one LLaMA-shaped layer: for every linear of the layer,
rcp_quantize_act (block-Hadamard + int4) then rcp_gemv_w2a4 (LUT GEMV), on seeded synthetic
tensors already resident in HBM. Successive steps use different weight copies (more than twice
the L2 in total), so every step streams its weights from DRAM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload KEY] [--tokens M]
  python bench.py --impl reference ...     # the CPU oracle on a bounded sample, same metric

Prints ONE JSON line (rank 0).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from gen import configs as cfgs  # noqa: E402
from gen import synth  # noqa: E402

METRIC = "w2a4_decode_layer_hbm_gbs"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
GROUP = 128   # weight group size of the group-wise grid


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return json.load(open(path)), "measured"
    return {"hbm_gbs": 6650.0}, "fallback"


def source_sha():
    """Hash of the CUDA sources: counters taken from an older kernel are not reported."""
    import hashlib
    h = hashlib.sha1()
    d = os.path.join(ROOT, "paper_2502_15779_b200", "csrc")
    for name in sorted(os.listdir(d)):
        h.update(name.encode())
        h.update(open(os.path.join(d, name), "rb").read())
    return h.hexdigest()[:16]


def profiled_counters(key):
    """Per-launch counters of the streaming kernel for this workload, as the profiling helper
    (python -m paper_2502_15779_b200.ncu_counters) wrote them from an ncu capture: DRAM bytes and warp
    instructions per launch. None when there is no capture for the key or the kernel sources changed since."""
    path = os.path.join(ROOT, "profiles", "counters.txt")
    if not os.path.exists(path):
        return None
    for ln in open(path):
        f = ln.split()
        if len(f) >= 2 and f[0] == key:
            d = dict(zip(f[1::2], f[2::2]))
            if d.get("source_sha") != source_sha():
                return None
            return {"dram_bytes_per_launch": float(d["dram_bytes_per_launch"]),
                    "warp_instructions_per_launch": float(d["warp_instructions_per_launch"]),
                    "launches": int(d["launches"])}
    return None


def f16_bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read only)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100", "-i",
                 str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------- workload
class LayerSet:
    """Packed weights (several distinct copies), LUTs, activations and scratch for one decode layer."""

    def __init__(self, cfg, M, device, copies, rcp):
        self.cfg, self.M, self.dev, self.rcp = cfg, M, device, rcp
        self.layers = list(cfg.layers)
        self.words, self.luts, self.x, self.xq, self.scale, self.y, self.ws = [], [], [], [], [], [], []
        self.codes_first = []
        for li, L in enumerate(self.layers):
            wcopies, lcopies = [], []
            for c in range(copies):
                seed = cfgs.BASE_SEED + 101 * li + 7 * c
                codes, lut = synth.make_layer(L.N, L.K, L.had_block, cfg.codes, seed, device)
                wcopies.append(rcp.rcp_pack_weights(codes))
                lcopies.append(lut)
                if c == 0:
                    self.codes_first.append(None)  # codes regenerated on demand for the CPU sample
                del codes
            self.words.append(wcopies)
            self.luts.append(lcopies)
            self.x.append(synth.make_activations(M, L.K, cfgs.BASE_SEED + 13 * li, device))
            self.xq.append(torch.empty(M, L.K // 2, dtype=torch.uint8, device=device))
            self.scale.append(torch.empty(M, dtype=torch.float16, device=device))
            self.y.append(torch.empty(M, L.N, dtype=torch.float16, device=device))
            self.ws.append(rcp.make_workspace(M, L.N, L.K, device))
        self.copies = copies
        self.digits = self.unit = self.w3 = self.glut = None

    def step_w2a16(self, copy):
        """The same layer in the weight-only form (fp16 activations): split kernel + GEMV per linear."""
        if self.digits is None:
            self.digits = [torch.empty(self.M, 4, L.K, dtype=torch.int8, device=self.dev) for L in self.layers]
            self.unit = [torch.empty(self.M, 4, dtype=torch.float32, device=self.dev) for L in self.layers]
        for li, L in enumerate(self.layers):
            self.rcp.rcp_gemv_w2a16(self.words[li][copy], self.luts[li][copy], self.x[li], y=self.y[li],
                                    digits=self.digits[li], unit=self.unit[li], workspace=self.ws[li])

    def step_w3a4(self, copy):
        """The same layer with 3-bit weights (random codes: the timing does not depend on them): quantizer + GEMV."""
        if self.w3 is None:
            self.w3 = []
            for L in self.layers:
                per = []
                for _ in range(self.copies):
                    w2 = torch.randint(-2 ** 31, 2 ** 31 - 1, (L.N, L.K // 16), dtype=torch.int32, device=self.dev)
                    w1 = torch.randint(-2 ** 31, 2 ** 31 - 1, (L.N, L.K // 32), dtype=torch.int32, device=self.dev)
                    per.append((w2, w1))
                lut8 = torch.sort(torch.randn(L.N, 8, device=self.dev) * 0.02, dim=1).values.half()
                self.w3.append((per, lut8))
        for li, L in enumerate(self.layers):
            per, lut8 = self.w3[li]
            self.rcp.rcp_quantize_act(self.x[li], L.had_block, 1.0, xq=self.xq[li], scale=self.scale[li])
            self.rcp.rcp_gemv_w3a4(per[copy][0], per[copy][1], lut8, self.xq[li], self.scale[li], y=self.y[li])

    def step_grouped(self, copy):
        """The same layer with one grid per group of 128 weights (the paper's own granularity): the library's chain
        with group=128 (one kernel where the quantizer goes inside, else quantizer + GEMV)."""
        if self.glut is None:
            self.glut = [synth.make_lut_grouped(L.N, L.K // 128, cfgs.BASE_SEED + 31 * li, self.dev)
                         for li, L in enumerate(self.layers)]
        for li, L in enumerate(self.layers):
            self.rcp.rcp_linear_w2a4(self.x[li], L.had_block, 1.0, self.words[li][copy], self.glut[li], group=128,
                                     y=self.y[li], xq=self.xq[li], scale=self.scale[li], workspace=self.ws[li])

    def step(self, copy, variant="auto"):
        r = self.rcp
        if variant == "w2a16":
            return self.step_w2a16(copy)
        if variant == "grouped":
            return self.step_grouped(copy)
        if variant == "w3a4":
            return self.step_w3a4(copy)
        for li, L in enumerate(self.layers):
            if variant == "auto":
                # the library's own chain: one kernel where that is faster, else quantizer + GEMV
                r.rcp_linear_w2a4(self.x[li], L.had_block, 1.0, self.words[li][copy], self.luts[li][copy], y=self.y[li],
                                  xq=self.xq[li], scale=self.scale[li], workspace=self.ws[li])
            else:
                r.rcp_quantize_act(self.x[li], L.had_block, 1.0, xq=self.xq[li], scale=self.scale[li])
                r.rcp_gemv_w2a4(self.words[li][copy], self.luts[li][copy], self.xq[li], self.scale[li], y=self.y[li],
                                workspace=self.ws[li], variant=variant)

    def launches_per_step(self, variant="auto"):
        r = self.rcp
        if variant == "auto":
            return sum(r.rcp_linear_w2a4_launches(self.M, L.N, L.K, L.had_block) for L in self.layers)
        return sum(1 + -(-self.M // (8 if variant in ("mma", "mma_only") else 2)) for L in self.layers)

    def stream_kernels_only(self, copy, variant="auto"):
        """The launches of the streaming kernel a step makes, without the stand-alone quantizer launches."""
        r = self.rcp
        for li, L in enumerate(self.layers):
            if variant == "auto" and r.rcp_linear_w2a4_launches(self.M, L.N, L.K, L.had_block) == 1:
                r.rcp_linear_w2a4(self.x[li], L.had_block, 1.0, self.words[li][copy], self.luts[li][copy], y=self.y[li],
                                  xq=self.xq[li], scale=self.scale[li], workspace=self.ws[li])
            else:
                r.rcp_gemv_w2a4(self.words[li][copy], self.luts[li][copy], self.xq[li], self.scale[li], y=self.y[li],
                                workspace=self.ws[li], variant=variant)

    def gemv_bytes(self):
        return sum(cfgs.gemv_bytes(self.M, L.N, L.K) for L in self.layers)

    def quant_bytes(self):
        return sum(cfgs.quant_bytes(self.M, L.K) for L in self.layers)

    def weight_bytes(self):
        return sum(L.N * L.K // 4 for L in self.layers)


def replica_metrics(ms_local, step_bytes, steps, dist=None, device="cpu"):
    """Whole-job throughput of independent replicas (one per rank, no data-path collective): the
    timed region ends when the slowest rank does, so the time is the MAX over ranks and the value
    is the bytes ALL ranks processed over that time. Returns (ms_per_step, GB/s, world)."""
    world = 1
    ms = float(ms_local)
    if dist is not None:
        world = dist.get_world_size()
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_per_step = ms / steps
    return ms_per_step, world * step_bytes / (ms_per_step * 1e-3) / 1e9, world


def l2_bytes(device):
    return torch.cuda.get_device_properties(device).L2_cache_size


def time_graph_replays(graphs, order, stream):
    """Replays graphs[order[i]] back to back; returns total milliseconds by CUDA events on `stream`."""
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for i in order:
            graphs[i].replay()
        e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1)


def capture(fn, stream):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        fn()
    return g


def per_shape_table(cfg, Ms, device, rcp, stream, variant, reps=3):
    """us/call and GB/s for every GEMV shape of a config and every token count in Ms: graphs of
    back-to-back launches cycling through distinct weight copies (cold L2), timed with CUDA events."""
    rows = []
    L2 = l2_bytes(device)
    seen = set()
    for li, L in enumerate(cfg.layers):
        if (L.N, L.K) in seen:
            continue
        seen.add((L.N, L.K))
        wbytes = L.N * L.K // 4
        copies = max(2, -(-2 * L2 // wbytes) + 1)
        copies = min(copies, 1200)
        seed = cfgs.BASE_SEED + 101 * li
        codes, lut = synth.make_layer(L.N, L.K, L.had_block, cfg.codes, seed, device)
        base = rcp.rcp_pack_weights(codes)
        del codes
        # distinct copies: rows rotated so contents differ but the value distribution is the same
        words = [torch.roll(base, shifts=c, dims=0).contiguous() if c else base for c in range(copies)]
        luts = [torch.roll(lut, shifts=c, dims=0).contiguous() if c else lut for c in range(copies)]
        # the same shape with one grid per group of 128 weights (the paper's weight group size)
        lut_g = synth.make_lut_grouped(L.N, L.K // GROUP, seed, device) if L.K % GROUP == 0 else None
        luts_g = [torch.roll(lut_g, shifts=c, dims=0).contiguous() if c else lut_g for c in range(copies)] \
            if lut_g is not None else None
        launches = copies * max(1, 64 // copies)
        for M in Ms:
            x = synth.make_activations(M, L.K, cfgs.BASE_SEED + 13 * li, device)
            xq, scale = rcp.rcp_quantize_act(x, L.had_block, 1.0)
            y = torch.empty(M, L.N, dtype=torch.float16, device=device)
            ws = rcp.make_workspace(M, L.N, L.K, device)

            def body():
                for i in range(launches):
                    c = i % copies
                    rcp.rcp_gemv_w2a4(words[c], luts[c], xq, scale, y=y, workspace=ws, variant=variant)

            with torch.cuda.stream(stream):
                body()
            stream.synchronize()
            g = capture(body, stream)
            for _ in range(3):
                g.replay()
            stream.synchronize()
            best = min(time_graph_replays([g], [0], stream) for _ in range(reps))
            us = best * 1e3 / launches
            nbytes = cfgs.gemv_bytes(M, L.N, L.K)
            # isolated single launch: no neighbour to overlap with. Queued behind a spin of about 100 us, so that the
            # two event records and the launch are all waiting when the spin ends and no host latency is inside.
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            iso = []
            for c in range(min(copies, 5)):
                with torch.cuda.stream(stream):
                    if hasattr(torch.cuda, "_sleep"):
                        torch.cuda._sleep(200000)
                    e0.record(stream)
                    rcp.rcp_gemv_w2a4(words[c], luts[c], xq, scale, y=y, workspace=ws, variant=variant)
                    e1.record(stream)
                e1.synchronize()
                iso.append(e0.elapsed_time(e1) * 1e3)
            # the quantizer alone
            gq = capture(lambda: [rcp.rcp_quantize_act(x, L.had_block, 1.0, xq=xq, scale=scale) for _ in range(32)],
                         stream)
            gq.replay()
            stream.synchronize()
            q_us = min(time_graph_replays([gq], [0], stream) for _ in range(reps)) * 1e3 / 32
            row = {"layer": L.name, "N": L.N, "K": L.K, "M": M, "bytes": nbytes, "us_per_call": round(us, 3),
                   "gbs": round(nbytes / us / 1e3, 1),
                   "frac_of_8TBs": round(nbytes / us / 1e3 / NOMINAL_HBM_GBS, 4),
                   "isolated_us": round(min(iso), 2), "quantize_us": round(q_us, 2), "copies": copies}
            if luts_g is not None:
                def body_g():
                    for i in range(launches):
                        c = i % copies
                        rcp.rcp_gemv_w2a4_grouped(words[c], luts_g[c], xq, scale, group=GROUP, y=y, workspace=ws,
                                                  variant=variant if variant in ("auto", "simple", "dp4a", "mma_only")
                                                  else "auto")
                with torch.cuda.stream(stream):
                    body_g()
                stream.synchronize()
                gg = capture(body_g, stream)
                for _ in range(3):
                    gg.replay()
                stream.synchronize()
                us_g = min(time_graph_replays([gg], [0], stream) for _ in range(reps)) * 1e3 / launches
                nbytes_g = cfgs.gemv_grouped_bytes(M, L.N, L.K, GROUP)
                row.update({"grouped_bytes": nbytes_g, "grouped_us_per_call": round(us_g, 3),
                            "grouped_gbs": round(nbytes_g / us_g / 1e3, 1)})
                del gg
            if M <= 2 and L.K <= 32768:
                # the weight-only form on the same weights: fp16 activations, split kernel + GEMV per call
                dg = torch.empty(M, 4, L.K, dtype=torch.int8, device=device)
                un = torch.empty(M, 4, dtype=torch.float32, device=device)

                def body_a():
                    for i in range(launches):
                        c = i % copies
                        rcp.rcp_gemv_w2a16(words[c], luts[c], x, y=y, digits=dg, unit=un, workspace=ws)
                with torch.cuda.stream(stream):
                    body_a()
                stream.synchronize()
                ga = capture(body_a, stream)
                for _ in range(3):
                    ga.replay()
                stream.synchronize()
                us_a = min(time_graph_replays([ga], [0], stream) for _ in range(reps)) * 1e3 / launches
                nbytes_a = cfgs.gemv_w2a16_bytes(M, L.N, L.K)
                row.update({"w2a16_bytes": nbytes_a, "w2a16_us_per_call": round(us_a, 3),
                            "w2a16_gbs": round(nbytes_a / us_a / 1e3, 1)})
                del ga
            if M == 1:
                # the 3-bit variant on the same shape (random codes: the timing does not depend on them)
                w2 = [torch.randint(-2 ** 31, 2 ** 31 - 1, (L.N, L.K // 16), dtype=torch.int32, device=device)
                      for _ in range(copies)]
                w1 = [torch.randint(-2 ** 31, 2 ** 31 - 1, (L.N, L.K // 32), dtype=torch.int32, device=device)
                      for _ in range(copies)]
                lut8 = torch.sort(torch.randn(L.N, 8, device=device) * 0.02, dim=1).values.half()

                def body_3():
                    for i in range(launches):
                        rcp.rcp_gemv_w3a4(w2[i % copies], w1[i % copies], lut8, xq, scale, y=y)
                with torch.cuda.stream(stream):
                    body_3()
                stream.synchronize()
                g3 = capture(body_3, stream)
                g3.replay()
                stream.synchronize()
                us_3 = min(time_graph_replays([g3], [0], stream) for _ in range(reps)) * 1e3 / launches
                nbytes_3 = cfgs.gemv_w3a4_bytes(M, L.N, L.K)
                row.update({"w3a4_bytes": nbytes_3, "w3a4_us_per_call": round(us_3, 3),
                            "w3a4_gbs": round(nbytes_3 / us_3 / 1e3, 1)})
                del g3, w2, w1
            rows.append(row)
        del words, luts, base, luts_g, lut_g
        torch.cuda.empty_cache()
    return rows


# ------------------------------------------------------------------------------- CPU oracle leg
def workload_name(cfg, M):
    return (f"{cfg.key} ({cfg.title}), M={M}: " + ", ".join(f"{L.name} {L.N}x{L.K}" for L in cfg.layers))


class OracleSample:
    """A bounded sample of one step for the CPU oracle (as it stands, one thread): the full activation
    quantization of every linear of the layer plus the GEMV on the first `rows` output rows of each,
    `rows` chosen so that one pass takes about `target_seconds`. Inputs are generated once."""

    def __init__(self, cfg, M, target_seconds):
        import oracle
        self.oracle = oracle
        layers = list(cfg.layers)
        # calibration on a tiny slice
        L0 = layers[0]
        codes, lut = synth.make_layer(16, L0.K, L0.had_block, cfg.codes, 1)
        x = synth.make_activations(M, L0.K, 1)
        t = time.perf_counter()
        qa = oracle.quantize_act(f16_bits(x), L0.had_block, 1.0)
        oracle.gemv_w2a4(oracle.pack_weights(codes.numpy()), f16_bits(lut), qa["xq"], qa["scale"])
        per_code = (time.perf_counter() - t) / (16 * L0.K * M)
        total_codes = sum(L.N * L.K for L in layers) * M
        frac = min(1.0, target_seconds / max(1e-9, per_code * total_codes))
        self.items, self.nbytes, desc = [], 0, []
        for li, L in enumerate(layers):
            rows = min(L.N, max(16, int(L.N * frac)))
            seed = cfgs.BASE_SEED + 101 * li
            codes, lut = synth.make_layer(rows, L.K, L.had_block, cfg.codes, seed)
            x = synth.make_activations(M, L.K, cfgs.BASE_SEED + 13 * li)
            words = oracle.pack_weights(codes.numpy())  # offline step, not timed
            self.items.append((f16_bits(x), L.had_block, words, f16_bits(lut)))
            self.nbytes += cfgs.gemv_bytes(M, rows, L.K) + cfgs.quant_bytes(M, L.K)
            desc.append(f"{L.name}:{rows}/{L.N} rows")
        self.desc = "quantize_act + gemv on " + ", ".join(desc)

    def run(self):
        """One pass; returns (value in the benchmark's unit, seconds)."""
        t = time.perf_counter()
        for xb, had_block, words, lb in self.items:
            qa = self.oracle.quantize_act(xb, had_block, 1.0)
            self.oracle.gemv_w2a4(words, lb, qa["xq"], qa["scale"])
        secs = time.perf_counter() - t
        return self.nbytes / secs / 1e9, secs


def host_cpu():
    """Model name and logical core count of the host the oracle is timed on."""
    model = "unknown"
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.lower().startswith("model name"):
                model = ln.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    return {"cpu_model": model, "nproc": os.cpu_count()}


def run_reference(args, cfg, M):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    budget = min(args.sample_seconds, 60.0 / max(1, args.steps + args.warmup))
    sample = OracleSample(cfg, M, budget)
    vals, secs = [], []
    for i in range(args.warmup + args.steps):
        v, s = sample.run()
        if i >= args.warmup:
            vals.append(v)
            secs.append(s)
    value = statistics.mean(vals)
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(secs), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
           "config": {"workload": workload_name(cfg, M), "note": "CPU oracle on a bounded sample of each step"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample.desc,
                            **host_cpu()},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_70b", choices=list(cfgs.BY_KEY))
    ap.add_argument("--tokens", type=int, default=1)
    ap.add_argument("--variant", default="auto", choices=["auto", "simple", "dp4a", "mma", "mma_only", "mma_stream", "w2a16", "w3a4", "grouped"],
                    help="kernel variant of the W2A4 GEMV; w2a16, w3a4 and grouped (only with --profile) run the layer in "
                         "the weight-only form, with 3-bit weights and with one grid per group of 128 weights "
                         "instead, for the ncu summaries")
    ap.add_argument("--no-table", action="store_true", help="skip the per-shape table of the other configs")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle leg")
    ap.add_argument("--sample-seconds", type=float, default=12.0,
                    help="CPU seconds the oracle sample of one step aims for (reference arm and cpu_baseline)")
    ap.add_argument("--profile", action="store_true",
                    help="warm-up and timed steps only, then exit (the command line the ncu summaries in profiles/ use)")
    args = ap.parse_args()
    cfg = cfgs.BY_KEY[args.workload]
    M = args.tokens
    if args.warmup < 3:
        args.warmup = 3

    if args.variant in ("w2a16", "w3a4", "grouped") and (not args.profile or args.impl == "reference"):
        ap.error(f"--variant {args.variant} is a profiling aid: use it with --profile")
    if args.impl == "reference":
        run_reference(args, cfg, M)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain script: start the N replicas (one process per GPU) the same way a launcher would
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))

    import paper_2502_15779_b200 as rcp
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    device = torch.device(f"cuda:{local_rank}")
    rcp.lib()  # fail loudly if the CUDA library is missing

    L2 = l2_bytes(device)
    wbytes = sum(L.N * L.K // 4 for L in cfg.layers)
    copies = max(2, -(-2 * L2 // wbytes) + 1)
    layer = LayerSet(cfg, M, device, copies, rcp)
    stream = torch.cuda.Stream(device=device)

    # eager warm-up (sets kernel attributes), then one CUDA graph per weight copy
    with torch.cuda.stream(stream):
        for c in range(copies):
            layer.step(c, args.variant)
    stream.synchronize()
    graphs = [capture(lambda c=c: layer.step(c, args.variant), stream) for c in range(copies)]
    order = [i % copies for i in range(args.warmup)]
    time_graph_replays(graphs, order, stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    barrier()
    if sampler:
        sampler.start()
    order = [i % copies for i in range(args.steps)]
    ms = time_graph_replays(graphs, order, stream)
    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_run": True, "workload": cfg.key, "M": M, "steps": args.steps,
                              "ms_per_step": ms / args.steps}), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return
    # keep the GPU under the same load a little longer so that the clock sampler sees it
    t_end = time.time() + 0.6
    while time.time() < t_end:
        time_graph_replays(graphs, order[:max(1, len(order) // 4)], stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    step_bytes = layer.gemv_bytes() + layer.quant_bytes()
    ms_per_step, value, _ = replica_metrics(ms, step_bytes, args.steps, dist, device)
    launches = args.steps * layer.launches_per_step(args.variant)

    # ---- dominant kernel alone: the streaming-kernel launches of a step (the GEMV, with the quantizer
    # inside where the step uses the single kernel), back to back, cold L2
    ggraphs = [capture(lambda c=c: layer.stream_kernels_only(c, args.variant), stream) for c in range(copies)]
    time_graph_replays(ggraphs, order[:8], stream)
    gms = min(time_graph_replays(ggraphs, order, stream) for _ in range(3))
    g_launches = args.steps * (layer.launches_per_step(args.variant) -
                               sum(1 for L in layer.layers
                                   if args.variant != "auto" or rcp.rcp_linear_w2a4_launches(M, L.N, L.K, L.had_block) > 1))
    g_bytes_per_launch = layer.gemv_bytes() * args.steps / g_launches
    g_us = gms * 1e3 / g_launches
    achieved = g_bytes_per_launch / g_us / 1e3
    peaks, peak_kind = measured_peaks()
    roofline = {"bound": "hbm", "kernel": "gemv_stream_kernel (with the activation quantizer inside where the step "
                                          "uses the single kernel)", "achieved": round(achieved, 1),
                "peak": peaks["hbm_gbs"], "peak_kind": peak_kind, "unit": "GB/s",
                "frac": round(achieved / peaks["hbm_gbs"], 4), "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                "avg_launch_us": round(g_us, 3), "bytes_per_launch": int(g_bytes_per_launch), "traffic": None}
    # for comparison: the plain GEMV launches alone (activations already quantized), same protocol
    def plain_gemv(c):
        for li, L in enumerate(layer.layers):
            rcp.rcp_gemv_w2a4(layer.words[li][c], layer.luts[li][c], layer.xq[li], layer.scale[li], y=layer.y[li],
                              workspace=layer.ws[li], variant=args.variant)
    pgraphs = [capture(lambda c=c: plain_gemv(c), stream) for c in range(copies)]
    time_graph_replays(pgraphs, order[:8], stream)
    pms = min(time_graph_replays(pgraphs, order, stream) for _ in range(3))
    # had_block 1 never takes the single kernel: the count is the quantizer plus the GEMV launches
    p_launches = args.steps * sum(rcp.rcp_linear_w2a4_launches(M, L.N, L.K, 1) - 1 if args.variant == "auto"
                                  else -(-M // (8 if args.variant in ("mma", "mma_only") else 2))
                                  for L in layer.layers)
    p_us = pms * 1e3 / p_launches
    p_ach = layer.gemv_bytes() * args.steps / p_launches / p_us / 1e3
    roofline["plain_gemv"] = {"avg_launch_us": round(p_us, 3), "achieved": round(p_ach, 1),
                              "frac": round(p_ach / peaks["hbm_gbs"], 4),
                              "note": "rcp_gemv_w2a4 launches alone, activations quantized beforehand"}
    del pgraphs
    # Second bound: instruction issue. An SM issues at most four warp instructions per clock; the count per KB of
    # packed weights comes from the ncu capture of this workload (none, or taken from older sources: not reported).
    counters = profiled_counters(f"{cfg.key}_M{M}_{args.variant}")
    if counters and clocks and clocks.get("sm_mhz"):
        sms = torch.cuda.get_device_properties(device).multi_processor_count
        per_kb = counters["warp_instructions_per_launch"] / (layer.weight_bytes() * args.steps / g_launches / 1024.0)
        issue_gbs = 4.0 * sms * clocks["sm_mhz"] * 1e6 / per_kb * 1024.0 / 1e9
        roofline["issue_bound"] = {"warp_instructions_per_kb": round(per_kb, 1), "peak": round(issue_gbs, 1), "unit": "GB/s",
                                   "frac": round(achieved / issue_gbs, 4),
                                   "note": "4 warp instructions per clock per SM at the sampled SM clock; count from ncu"}
    if counters:
        roofline["traffic"] = int(counters["dram_bytes_per_launch"])

    # ---- end to end through the C ABI with host buffers
    xh = [layer.x[li].cpu().pin_memory() for li in range(len(layer.layers))]
    yh = [torch.empty(M, L.N, dtype=torch.float16).pin_memory() for L in layer.layers]

    def e2e_step(c):
        for li, L in enumerate(layer.layers):
            rcp.rcp_linear_w2a4_host(xh[li], L.had_block, 1.0, layer.words[li][c], layer.luts[li][c], yh[li],
                                     layer.x[li], layer.xq[li], layer.scale[li], layer.y[li], layer.ws[li])
    e2e_steps = min(args.steps, 100)
    with torch.cuda.stream(stream):
        for i in range(3):
            e2e_step(i % copies)
            stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for i in range(e2e_steps):
            e2e_step(i % copies)
            stream.synchronize()  # the host reads y before the next decode step
        e1.record(stream)
    e1.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms_per_step, e2e_value, _ = replica_metrics(e2e_ms, step_bytes, e2e_steps, dist, device)
    e2e = {"value": round(e2e_value, 2), "unit": UNIT,
           "ms_per_step": round(e2e_ms_per_step, 4),
           "transfer": "rcp_linear_w2a4_host on pinned buffers: the quantizer reads x from host memory and the GEMV "
                       "stores y into it directly (no staging copy); the host waits for the stream after every step",
           "h2d_bytes_per_step": sum(2 * M * L.K for L in layer.layers),
           "d2h_bytes_per_step": sum(2 * M * L.N for L in layer.layers)}
    # The same step from a C++ host program through the C ABI (no interpreter in the loop), one token: what the
    # binding and the interpreter add to the figure above. Rank 0 of a single-GPU run only; reported beside it.
    if rank == 0 and world == 1 and M == 1:
        try:
            from paper_2502_15779_b200 import build as _b
            drv = _b.build_driver()
            cmd = [drv, str(e2e_steps), "5"] + [str(v) for L in layer.layers for v in (L.N, L.K, L.had_block)]
            env = dict(os.environ, CUDA_VISIBLE_DEVICES=os.environ.get("CUDA_VISIBLE_DEVICES", str(local_rank)))
            out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
            d = json.loads(out.stdout.strip().splitlines()[-1])
            e2e["c_driver"] = {"value": round(d["gbs"], 2), "unit": UNIT, "ms_per_step": round(d["us_per_step"] / 1e3, 4),
                               "note": "e2e_driver.cu: rcp_linear_w2a4_host per linear on pinned buffers, "
                                       "cudaStreamSynchronize after every step, host wall clock"}
        except Exception as ex:   # noqa: BLE001  (the driver is an extra: never fail the benchmark for it)
            e2e["c_driver"] = {"unavailable": repr(ex)[:200]}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    shapes = []
    if not args.no_table:
        del graphs, ggraphs
        for c in cfgs.CONFIGS:
            Ms = tuple(sorted(set(c.Ms) | ({M} if c.key == cfg.key else set())))
            shapes.append({"config": c.key, "rows": per_shape_table(c, Ms, device, rcp, stream, args.variant)})

    # offline step: weight packing throughput (not part of the decode step)
    Lp = cfg.layers[0]
    codes = synth.make_codes_uniform(Lp.N, Lp.K, 1, device)
    outw = torch.empty(Lp.N, Lp.K // 16, dtype=torch.int32, device=device)
    rcp.rcp_pack_weights(codes, out=outw)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    rcp.rcp_pack_weights(codes, out=outw)
    e1.record()
    e1.synchronize()
    pack_ms = e0.elapsed_time(e1)
    pack = {"N": Lp.N, "K": Lp.K, "ms": round(pack_ms, 4),
            "gbs": round((Lp.N * Lp.K * 1.25) / pack_ms / 1e6, 1), "note": "offline step, includes the status read-back"}

    cpu = None
    if not args.no_cpu:
        sample = OracleSample(cfg, M, args.sample_seconds)
        v, secs = sample.run()
        cpu = {"value": round(v, 4), "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample.desc,
               "seconds": round(secs, 2), **host_cpu()}

    out = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "int32", "data": "synthetic",
           "config": {"workload": workload_name(cfg, M),
                      "step": "per linear: rcp_linear_w2a4 (activation quantization + LUT GEMV: one kernel for one "
                              "token of 4096 or 8192 under one rotation block, else rcp_quantize_act then "
                              "rcp_gemv_w2a4), replayed from a CUDA graph",
                      "cold_l2": f"{copies} distinct weight copies in rotation ({copies * wbytes / 1e6:.0f} MB > 2x L2 "
                                 f"of {L2 / 1e6:.0f} MB)",
                      "variant": args.variant, "parallelism": "replicas only" if world > 1 else "single GPU",
                      "bytes_per_step": step_bytes},
           "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
           "us_per_gemv_call": round(g_us, 3), "pack": pack, "shapes": shapes}
    print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
