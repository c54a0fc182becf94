#!/usr/bin/env python
"""Benchmark of the TAQ cross-attention hot path on B200.

``python bench.py [--gpus N] [--steps K] [--warmup W]`` times K passes of one cross-attention layer
(to_q with Q~ = Q_a(Q), fused attention with Eq. 3, to_out; K~/V~ of Eq. 2 projected once per prompt outside
the step, as they do not depend on the image tokens) on the SD-1.5 highest-resolution configuration
(B=2, N=4096, C=320, 8 heads, T=77, W4 group 128, trigger tokens {4,5}) and prints one JSON line.
Every step uses a different set of input/output/weight buffers out of a ring larger than twice the L2, so
each pass streams its activations from HBM.  ``--impl reference`` times the CPU oracle instead.
Under torchrun each rank runs an independent replica (the path has no exchange step).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "TAQ cross-attn queries/s per layer"
UNIT = "queries/s"


def measured_traffic(kernel: str):
    """DRAM bytes per launch (read + write) of `kernel` from the last ncu capture, as recorded by
    `python -m paper_2603_22943_b200.profile_traffic`; None when there is no record or the kernel's source has changed
    since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    rec = json.load(open(path)).get(kernel)
    if not rec:
        return None
    src = os.path.join(ROOT, rec["source"])
    if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != rec["source_sha256"]:
        return None
    return int(rec["dram_bytes_per_launch"])
WORKLOAD = "config2: SD-1.5 64x64 cross-attn layer, B=2 N=4096 C=320 H=8 d=40 T=77 Dc=768, W4 g128, int8 Q/K/V rows, uint8 probs, fp16 trigger rows {4,5}"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20", "-i", str(self.gpu)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of per-rank timings over all ranks (the job is as slow as its slowest replica)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(units_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling: every rank processes its own units)."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def _oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle(shape, data, sample_rows: int, repeats: int = 1):
    """Contract-mode oracle on `sample_rows` query rows of every sequence; returns (seconds, rows)."""
    from oracle import taq_oracle as orc
    rows = np.arange(min(sample_rows, shape.n_query))
    cfg = orc.TaqConfig(heads=shape.heads, w_bits=shape.w_bits, w_group=shape.w_group, q_bits=shape.q_bits, contract=True)
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.taq_layer(data["X"][:, rows], data["ctx"], data["Wq"], data["Wk"], data["Wv"], data["Wout"], data["bout"], data["mask"], cfg)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best, shape.batch * len(rows)


def run_reference(args, shape, data):
    """The base contract's reference arm: the CPU oracle, as it stands, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = min(shape.n_query, args.ref_rows)
    for _ in range(args.warmup):
        time_oracle(shape, data, sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(shape, data, sample)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = shape.batch * sample / dt
    cores = _oracle_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": f"first {sample} query rows of each of the {shape.batch} sequences per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": f"{shape.batch}x{sample} query rows per step (whole layer incl. K/V projection)"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def time_replays(torch, g, min_total_ms=400.0, min_replays=5, max_replays=20000):
    """Replays a captured graph until at least `min_total_ms` of device time have been timed; every replay has its own
    pair of CUDA events on the launching stream.  Returns the per-replay milliseconds: median, min, max, and the count."""
    g.replay()
    torch.cuda.synchronize()
    times = []
    total = 0.0
    while (total < min_total_ms or len(times) < min_replays) and len(times) < max_replays:
        n = 16 if times else 4
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in evs:
            a.record()
            g.replay()
            b.record()
        torch.cuda.synchronize()
        for a, b in evs:
            t = a.elapsed_time(b)
            times.append(t)
            total += t
    return {"median": statistics.median(times), "min": min(times), "max": max(times), "replays": len(times)}


def _graph_time(torch, fn, count, replays):
    """Captures `count` calls of fn(i) into one CUDA graph and returns the milliseconds of one replay (device time)."""
    for i in range(min(count, 8)):
        fn(i)
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for i in range(count):
            fn(i)
    g.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(replays):
        g.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / replays


def _layer_flops_bytes(tb, l):
    """Algorithmic FLOPs and bytes of one layer pass (a3..a9): X in, Y out, the two packed weight matrices and the K~/V~
    operand images once."""
    rows = l.batch * l.n_query
    flops = 4 * rows * l.channels * l.channels + 4 * rows * l.n_ctx * l.channels
    desc = tb.layer_desc(l.batch, l.n_query, l.channels, l.heads, l.n_ctx, l.ctx_dim, l.w_bits, l.w_group, q_bits=l.q_bits, max_trigger=len(l.trigger))
    wbytes = tb.taq_packed_weight_bytes(tb.weight_desc(l.channels, l.channels, l.w_bits, l.w_group))
    nbytes = 2 * rows * l.channels * 2 + 2 * wbytes + tb.taq_kv_layout_of(desc).operand_head_bytes * l.heads * l.batch
    return flops, nbytes


def _bench_layers(torch, tb, synth, dev, layers, n_sets, steps):
    """One step = taq_layer_forward on every layer of `layers`; every step uses another of `n_sets` buffer sets.  Returns
    the replay statistics (ms per step), launches per step by kernel family, and the per-step bytes of a buffer set."""
    sets = []
    for k in range(n_sets):
        L = []
        for shp in layers:
            data = synth.make_layer(shp)
            desc = tb.layer_desc(shp.batch, shp.n_query, shp.channels, shp.heads, shp.n_ctx, shp.ctx_dim, shp.w_bits, shp.w_group,
                                 q_bits=shp.q_bits, max_trigger=len(shp.trigger))
            wd_cc = tb.weight_desc(shp.channels, shp.channels, shp.w_bits, shp.w_group)
            wd_cd = tb.weight_desc(shp.channels, shp.ctx_dim, shp.w_bits, shp.w_group)
            mask = dev(data["mask"])
            kv = tb.taq_kv_project(desc, dev(data["ctx"]), tb.taq_pack_weights(wd_cd, dev(data["Wk"])), tb.taq_pack_weights(wd_cd, dev(data["Wv"])), mask)
            L.append((desc, dev(np.roll(data["X"], k, axis=1)), tb.taq_pack_weights(wd_cc, dev(data["Wq"])),
                      tb.taq_pack_weights(wd_cc, dev(data["Wout"]), dev(data["bout"])), kv, mask,
                      torch.empty((shp.batch, shp.n_query, shp.channels), dtype=torch.float16, device="cuda"),
                      torch.empty(tb.taq_workspace_bytes(desc, 1), dtype=torch.uint8, device="cuda")))
        sets.append(L)
    tb.taq_poll_device_status()

    def step(i):
        for (desc, x, Wq, Wo, kv, mask, y, ws) in sets[i % n_sets]:
            tb.taq_layer_forward(desc, x, Wq, Wo, kv, mask, y, ws)

    for i in range(min(steps, 8)):
        step(i)
    torch.cuda.synchronize()
    tb.taq_dispatch_reset()
    step(0)
    per_step = tb.taq_dispatch_counts()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream()):
        for i in range(steps):
            step(i)
    rep = time_replays(torch, g)
    tb.taq_poll_device_status()
    return {k: v / steps for k, v in rep.items() if k != "replays"} | {"replays": rep["replays"]}, per_step


def _workload_line(metric, workload, layers, ms, rep, per_step, steps, n_sets, peaks, clocks, tb, bound):
    rows = sum(l.batch * l.n_query for l in layers)
    fb = [_layer_flops_bytes(tb, l) for l in layers]
    flops, nbytes = sum(f for f, _ in fb), sum(b for _, b in fb)
    tf, gbs = flops / (ms * 1e-3) / 1e12, nbytes / (ms * 1e-3) / 1e9
    launches = sum(per_step.values())
    roof = {"bound": bound, "traffic": None, "flops_per_step": flops, "bytes_per_step": nbytes,
            "tensor": {"achieved_TFLOPs": tf, "peak_TFLOPs": peaks["bf16_tflops"], "frac": tf / peaks["bf16_tflops"]},
            "hbm": {"achieved_GBps": gbs, "peak_GBps": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"]},
            "peak_source": peaks["source"]}
    if bound == "tensor":
        roof.update({"achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"]})
    else:
        roof.update({"achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]})
    return {"metric": metric, "value": rows / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": 8, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": workload, "launch": "one CUDA graph of the steps, replayed until 0.4 s are timed; value = median replay",
                       "l2_policy": f"ring of {n_sets} buffer sets ({n_sets * nbytes / 1e6:.0f} MB of activations and weights)"},
            "timing": {"replays": rep["replays"], "ms_per_step_min": rep["min"], "ms_per_step_max": rep["max"]},
            "kernel_launches_per_step": per_step, "generic_kernel_launches": per_step["linear_generic"] + per_step["attention_generic"],
            "clocks": clocks, "gpu_launches": launches * steps, "roofline": roof}


def run_other_workload(args):
    """The other measured configurations (not the headline line): `config1`, the SD-1.5 lowest-resolution layer (W8);
    `config3`, one SD-1.5 UNet step of all 16 cross-attention layers; `config4`, the two SDXL-shaped layers (one line
    each); `config5`, the multi-checkpoint serving sweep on the 64x64 layer; `attention`, taq_cross_attention alone at
    three launches of many CTAs (one line each, HBM roofline).  One GPU."""
    import torch
    from paper_2603_22943_b200 import binding as tb
    from paper_2603_22943_b200 import synth
    torch.cuda.set_device(0)
    tb.lib()
    peaks = _peaks()
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    sampler = ClockSampler(0)
    sampler.start()
    if args.workload == "attention":
        # taq_cross_attention alone at launches of many CTAs: Q~ codes and scales in, O out (the HBM-bound stage)
        lines = []
        for B, N, C_, H, Dc in ((64, 256, 1280, 8, 768), (16, 1024, 640, 8, 768), (32, 4096, 320, 8, 768)):
            T = 77
            desc = tb.layer_desc(B, N, C_, H, T, Dc, 4, 128, q_bits=8, max_trigger=2)
            r = np.random.default_rng(7)
            wd = tb.weight_desc(C_, Dc, 4, 128)
            Wk = tb.taq_pack_weights(wd, dev((r.standard_normal((C_, Dc)) / np.sqrt(Dc)).astype(np.float32)))
            Wv = tb.taq_pack_weights(wd, dev((r.standard_normal((C_, Dc)) / np.sqrt(Dc)).astype(np.float32)))
            m = np.zeros((B, T), np.uint8)
            m[:, 4:6] = 1
            mask = dev(m)
            kv = tb.taq_kv_project(desc, dev(r.standard_normal((B, T, Dc)).astype(np.float16)), Wk, Wv, mask)
            img = tb.taq_kv_layout_of(desc).operand_head_bytes * H * B
            nbytes = B * N * (C_ + 4 * H) + B * N * C_ * 2 + img          # Q~ codes + scales, O, operand images
            n_sets = max(3, int(np.ceil(2.2 * l2 / nbytes)))
            sets = [(torch.randint(-127, 128, (B * N, C_), dtype=torch.int8, device="cuda"), torch.rand((B * N, H), device="cuda") * 0.05,
                     torch.empty((B, N, C_), dtype=torch.float16, device="cuda")) for _ in range(n_sets)]

            def step(i, sets=sets, desc=desc, kv=kv, mask=mask, n_sets=n_sets):
                q, qs, o = sets[i % n_sets]
                tb.taq_cross_attention(desc, q, qs, kv, mask, o)

            steps = max(n_sets, 12)
            for i in range(8):
                step(i)
            torch.cuda.synchronize()
            tb.taq_dispatch_reset()
            step(0)
            torch.cuda.synchronize()
            counts = tb.taq_dispatch_counts()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=torch.cuda.Stream()):
                for i in range(steps):
                    step(i)
            rep = time_replays(torch, g, min_total_ms=200.0)
            ms = rep["median"] / steps
            gbs = nbytes / (ms * 1e-3) / 1e9
            lines.append({"metric": "TAQ attention queries/s (taq_cross_attention alone)", "value": B * N / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps,
                          "warmup": 8, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
                          "config": {"workload": f"attention: B={B} N={N} C={C_} H={H} d={C_ // H} T=77, int8 Q~ per (row, head), trigger {{4,5}}",
                                     "l2_policy": f"ring of {n_sets} buffer sets ({n_sets * nbytes / 1e6:.0f} MB)"},
                          "timing": {"replays": rep["replays"], "ms_per_step_min": rep["min"] / steps, "ms_per_step_max": rep["max"] / steps},
                          "kernel_launches_per_step": counts, "gpu_launches": steps,
                          "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                       "traffic": measured_traffic(f"attention_sm100_kernel_d{C_ // H}_b{B}"), "bytes_per_launch": nbytes,
                                       "peak_source": peaks["source"]}})
            del sets
        tb.taq_poll_device_status()
        clocks = sampler.stop()
        for line in lines:
            line["clocks"] = clocks
            print(json.dumps(line), flush=True)
        return
    if args.workload in ("config1", "config3", "config4"):
        if args.workload == "config1":
            cases = [("TAQ cross-attn queries/s per layer", "config1: SD-1.5 8x8 cross-attn layer, B=1 N=64 C=1280 H=8 d=160 T=77 Dc=768, W8 per-channel, trigger {5}",
                      [synth.config1()], "hbm")]
        elif args.workload == "config4":
            cases = [("TAQ cross-attn queries/s per layer", f"config4: SDXL-shaped cross-attn layer, B=2 N={l.n_query} C={l.channels} H={l.heads} d=64 T=77 Dc=2048, W4 g128, trigger {{3,4,5}}",
                      [l], "tensor") for l in synth.config4_layers()]
        else:
            cases = [("TAQ cross-attn queries/s over one SD-1.5 UNet step (16 layers)",
                      "config3: all 16 SD-1.5 cross-attn layers (5x(N=4096,C=320), 5x(1024,640), 5x(256,1280), 1x(64,1280)), B=2, T=77, W4 g128, trigger {4,5}",
                      synth.config3_layers(), "tensor")]
        lines = []
        for metric, workload, layers, bound in cases:
            set_bytes = sum(_layer_flops_bytes(tb, l)[1] for l in layers)
            n_sets = max(3, int(np.ceil(2.2 * l2 / set_bytes)))
            steps = max(n_sets, min(args.steps, 96 if set_bytes < 20e6 else 12))
            rep, per_step = _bench_layers(torch, tb, synth, dev, layers, n_sets, steps)
            lines.append((metric, workload, layers, rep, per_step, steps, n_sets, bound))
        clocks = sampler.stop()
        for metric, workload, layers, rep, per_step, steps, n_sets, bound in lines:
            print(json.dumps(_workload_line(metric, workload, layers, rep["median"], rep, per_step, steps, n_sets, peaks, clocks, tb, bound)), flush=True)
        return
    # config5: 64 checkpoints resident, requests routed to random checkpoints, the N=4096 x C=320 layer
    n_ckpt, N, C_, H, T, Dc = 64, 4096, 320, 8, 77, 768
    wd_cc, wd_cd = tb.weight_desc(C_, C_, 4, 128), tb.weight_desc(C_, Dc, 4, 128)
    desc1 = tb.layer_desc(1, N, C_, H, T, Dc, 4, 128, q_bits=8, max_trigger=3)
    ck = []
    for c in range(n_ckpt):
        cp = synth.make_checkpoint(c, C_, Dc, T)
        w = cp.weights
        ck.append((cp, tb.taq_pack_weights(wd_cc, dev(w["Wq"])), tb.taq_pack_weights(wd_cc, dev(w["Wout"]), dev(w["bout"])),
                   tb.taq_pack_weights(wd_cd, dev(w["Wk"])), tb.taq_pack_weights(wd_cd, dev(w["Wv"]))))
    n_slots = 64
    route = synth.make_request_batch(n_slots, n_ckpt, 0)
    slot = []
    for r in range(n_slots):
        cp, Wq, Wo, Wk, Wv = ck[int(route[r])]
        act = synth.make_request_activations(cp, N, C_, Dc, T, r)
        mask = dev(act["mask"])
        kv = tb.taq_kv_project(desc1, dev(act["ctx"]), Wk, Wv, mask)
        slot.append((Wq, Wo, kv, mask, act["X"]))
    x_all = dev(np.concatenate([s_[4] for s_ in slot], axis=0))              # [64][N][C]
    y_all = torch.empty_like(x_all)
    per_ckpt_all_layers = sum(2 * tb.taq_packed_weight_bytes(tb.weight_desc(l.channels, l.channels, 4, 128)) +
                              2 * tb.taq_packed_weight_bytes(tb.weight_desc(l.channels, l.ctx_dim, 4, 128)) for l in synth.config3_layers())
    results = []
    for nb in (1, 8, 32, 64):
        groups = n_slots // nb
        tables = [tb.make_request_table([slot[g * nb + j][:4] for j in range(nb)], "cuda") for g in range(groups)]
        ws = torch.empty(tb.taq_workspace_bytes(desc1, nb), dtype=torch.uint8, device="cuda")

        def step(i, nb=nb, groups=groups, tables=tables, ws=ws):
            g = i % groups
            tb.taq_layer_forward_batched(desc1, tables[g], nb, x_all[g * nb:(g + 1) * nb], y_all[g * nb:(g + 1) * nb], ws)

        count = max(groups, 16)
        for i in range(min(count, 8)):
            step(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=torch.cuda.Stream()):
            for i in range(count):
                step(i)
        rep = time_replays(torch, g, min_total_ms=200.0)
        ms = rep["median"] / count
        flops = nb * (4 * N * C_ * C_ + 4 * N * T * C_)
        results.append({"requests_per_batch": nb, "ms_per_batch": round(ms, 5), "ms_per_batch_min": round(rep["min"] / count, 5), "ms_per_batch_max": round(rep["max"] / count, 5),
                        "requests_per_s": nb / (ms * 1e-3), "queries_per_s": nb * N / (ms * 1e-3),
                        "TFLOP/s": flops / (ms * 1e-3) / 1e12, "frac_of_tensor_peak": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]})
    tb.taq_poll_device_status()
    best = results[-1]
    kvl = tb.taq_kv_layout_of(desc1)
    line = {"metric": "TAQ multi-checkpoint serving, requests/s on the N=4096 x C=320 layer", "value": best["requests_per_s"], "unit": "requests/s", "n_gpus": 1,
            "steps": 16, "warmup": 8, "ms_per_step": best["ms_per_batch"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
            "data": "synthetic",
            "config": {"workload": "config5: 64 synthetic checkpoints resident (packed W4 g128), each request routed to a random checkpoint with its own weights, K~/V~ and trigger span (1-3 tokens)",
                       "launch": "one kernel per batch (grid.z = request), batches rotate over 64 resident request slots (168 MB of activations)",
                       "packed_bytes_per_checkpoint_all_16_layers": per_ckpt_all_layers, "fp16_bytes_per_checkpoint_all_16_layers": int(per_ckpt_all_layers / 4.25 * 16),
                       "kv_bytes_per_prompt_this_layer": kvl.block_bytes,
                       "kv_bytes_per_prompt_this_layer_without_operand_images": kvl.block_bytes - kvl.operand_head_bytes * H},
            "sweep": results, "clocks": sampler.stop(), "gpu_launches": 16,
            "roofline": {"bound": "tensor", "achieved": best["TFLOP/s"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": best["frac_of_tensor_peak"],
                         "traffic": None, "peak_source": peaks["source"]}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="taq", choices=["taq", "reference"])
    ap.add_argument("--ref-rows", type=int, default=1024, help="query rows per sequence in one reference-arm step")
    ap.add_argument("--cpu-rows", type=int, default=4096, help="query rows per sequence of the cpu_baseline sample")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU time to spend on the cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--n-query", type=int, default=0, help="override N (profiling on a smaller case)")
    ap.add_argument("--workload", default="config2", choices=["config1", "config2", "config3", "config4", "config5", "attention"],
                    help="config2 (default) is the headline line; the others print the other measured configurations (config4: one line per SDXL layer; attention: one line per shape)")
    args = ap.parse_args()
    if args.workload != "config2":
        run_other_workload(args)
        return
    if args.warmup < 3 and args.impl == "taq":
        args.warmup = 3

    from paper_2603_22943_b200 import synth
    shape = synth.config2()
    if args.n_query:
        shape = synth.shrink(shape, args.n_query)
    data = synth.make_layer(shape)

    if args.impl == "reference":
        run_reference(args, shape, data)
        return

    import torch
    from paper_2603_22943_b200 import binding as tb
    from paper_2603_22943_b200 import build as tbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the TAQ path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if not os.path.exists(tb.LIB_PATH):
        tbuild.build_library()
    tb.lib()

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    B, N, C_, H, T, Dc = shape.batch, shape.n_query, shape.channels, shape.heads, shape.n_ctx, shape.ctx_dim
    M = B * N
    desc = tb.layer_desc(B, N, C_, H, T, Dc, shape.w_bits, shape.w_group, q_bits=shape.q_bits, max_trigger=len(shape.trigger))
    wd_cc = tb.weight_desc(C_, C_, shape.w_bits, shape.w_group)
    wd_cd = tb.weight_desc(C_, Dc, shape.w_bits, shape.w_group)
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    set_bytes = 2 * M * C_ * 2
    n_sets = max(4, int(np.ceil(2.2 * l2 / set_bytes)))

    Wk = tb.taq_pack_weights(wd_cd, dev(data["Wk"]))
    Wv = tb.taq_pack_weights(wd_cd, dev(data["Wv"]))
    mask = dev(data["mask"])
    ctx = dev(data["ctx"])
    x_host = data["X"]
    sets = []
    for i in range(n_sets):     # every set: its own activations, weights, K~/V~ and workspace
        s = {"x": dev(np.roll(x_host, i, axis=1)), "y": torch.empty((B, N, C_), dtype=torch.float16, device="cuda"),
             "Wq": tb.taq_pack_weights(wd_cc, dev(data["Wq"])), "Wout": tb.taq_pack_weights(wd_cc, dev(data["Wout"]), dev(data["bout"])),
             "ws": torch.empty(tb.taq_workspace_bytes(desc, 1), dtype=torch.uint8, device="cuda")}
        s["kv"] = tb.taq_kv_project(desc, ctx, Wk, Wv, mask)
        sets.append(s)
    tb.taq_poll_device_status()

    def step(i):
        s = sets[i % n_sets]
        tb.taq_layer_forward(desc, s["x"], s["Wq"], s["Wout"], s["kv"], mask, s["y"], s["ws"])

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # The timed region is one CUDA graph holding the K steps (3 launches each): the step is a few microseconds of
    # GPU work, so launching it call by call from Python would time the interpreter, not the kernels.
    for i in range(args.warmup):
        step(i)
    barrier()
    cap_stream = torch.cuda.Stream()

    def capture(fn, count):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap_stream):
            for i in range(count):
                fn(i)
        return g

    def time_graph(g, replays=1):
        g.replay()                       # untimed: uploads the graph
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / replays

    g_steps = capture(step, args.steps)
    g_steps.replay()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    # The graph of exactly K steps is replayed until about 0.4 s of device time have been timed, every replay between its
    # own pair of CUDA events; the reported step time is the median replay divided by K (minimum and maximum beside it).
    rep = time_replays(torch, g_steps)
    barrier()
    ms_total = rep["median"]

    # A step is one launch (the whole layer pass in one kernel), so the step time is that kernel's launch duration.  For
    # comparison the stand-alone entry points (fused to_q + attention, and to_q / attention / to_out as separate kernels)
    # are timed the same way: one graph of n_sets back-to-back launches over the buffer ring, CUDA events around it.
    q_c = torch.empty((M, C_), dtype=torch.int8 if shape.q_bits == 8 else torch.float16, device="cuda")
    q_s = torch.empty((M, H), dtype=torch.float32, device="cuda")
    o_sets = [torch.empty((B, N, C_), dtype=torch.float16, device="cuda") for _ in range(n_sets)]
    q_sets = [(torch.empty_like(q_c), torch.empty_like(q_s)) for _ in range(n_sets)]

    def stage_qattn(i):
        s = sets[i % n_sets]
        tb.taq_query_attention(desc, s["x"], s["Wq"], s["kv"], mask, o_sets[i % n_sets], s["ws"])

    def stage_q(i):
        s = sets[i % n_sets]
        qc, qs = q_sets[i % n_sets]
        if shape.q_bits == 8:
            tb.taq_quantized_linear(wd_cc, s["x"], s["Wq"], tb.TAQ_OUT_INT8_HEAD_ROWS, heads=H, y=qc, scales=qs)
        else:
            tb.taq_quantized_linear(wd_cc, s["x"], s["Wq"], tb.TAQ_OUT_F16, y=qc)

    def stage_attn(i):
        s = sets[i % n_sets]
        qc, qs = q_sets[i % n_sets]
        tb.taq_cross_attention(desc, qc, qs if shape.q_bits == 8 else None, s["kv"], mask, o_sets[i % n_sets])

    def stage_out(i):
        s = sets[i % n_sets]
        tb.taq_quantized_linear(wd_cc, o_sets[i % n_sets], s["Wout"], tb.TAQ_OUT_F16, y=s["y"])

    # the integer-activation reading (int8 X and O, tcgen05 kind::i8): the layer pass, and its to_out GEMM alone on codes
    # quantized beforehand
    ws_a8 = torch.empty(tb.taq_workspace_bytes_a8(desc), dtype=torch.uint8, device="cuda")
    oq_sets = [tb.taq_quantize_rows_f16(sets[i]["x"].view(M, C_)) for i in range(n_sets)]

    def stage_layer_a8(i):
        s = sets[i % n_sets]
        tb.taq_layer_forward_a8(desc, s["x"], s["Wq"], s["Wout"], s["kv"], mask, s["y"], ws_a8)

    def stage_out_i8(i):
        s = sets[i % n_sets]
        oc, os_ = oq_sets[i % n_sets]
        tb.taq_quantized_linear_i8(wd_cc, oc, os_, s["Wout"], tb.TAQ_OUT_F16, y=s["y"])

    stage_ms = {}
    for name, fn in (("qattn", stage_qattn), ("to_q", stage_q), ("attn", stage_attn), ("to_out", stage_out),
                     ("layer_a8", stage_layer_a8), ("to_out_i8", stage_out_i8)):
        for i in range(n_sets):
            fn(i)
        torch.cuda.synchronize()
        g = capture(fn, n_sets)
        stage_ms[name] = time_graph(g, replays=max(1, min(args.steps, 200) // n_sets)) / n_sets
    clocks = sampler.stop()

    # End to end through the same call with host buffers: H2D of X and D2H of Y inside the timed region.
    xh = [torch.from_numpy(np.ascontiguousarray(np.roll(x_host, i, axis=1))).pin_memory() for i in range(4)]
    yh = [torch.empty((B, N, C_), dtype=torch.float16).pin_memory() for _ in range(4)]
    e_steps = max(10, min(args.steps, 100))

    # Three streams: the upload of step i + 1 and the download of step i - 1 run under the kernel of step i (PCIe is full
    # duplex), every copy is inside the timed region, and a buffer set is reused only after its previous user is done.
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in, ev_cmp, ev_out = {}, {}, {}

    def e2e_step(i):
        s = sets[i % n_sets]
        with torch.cuda.stream(s_in):
            if i - n_sets in ev_cmp:
                s_in.wait_event(ev_cmp[i - n_sets])          # the set's X is no longer being read
            s["x"].copy_(xh[i % 4], non_blocking=True)
            ev_in[i] = torch.cuda.Event()
            ev_in[i].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(ev_in[i])
            if i - n_sets in ev_out:
                s_cmp.wait_event(ev_out[i - n_sets])         # the set's Y has been downloaded
            tb.taq_layer_forward(desc, s["x"], s["Wq"], s["Wout"], s["kv"], mask, s["y"], s["ws"])
            ev_cmp[i] = torch.cuda.Event()
            ev_cmp[i].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[i])
            yh[i % 4].copy_(s["y"], non_blocking=True)
            ev_out[i] = torch.cuda.Event()
            ev_out[i].record(s_out)

    for i in range(3):
        e2e_step(i)
    barrier()
    ev_in.clear(); ev_cmp.clear(); ev_out.clear()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(s_in)
    for i in range(e_steps):
        e2e_step(i)
    f1.record(s_out)
    barrier()
    e2e_ms = f0.elapsed_time(f1)
    tb.taq_poll_device_status()

    ms_total, e2e_ms, ms_min, ms_max = max_over_ranks([ms_total, e2e_ms, rep["min"], rep["max"]], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = _peaks()
    ms_per_step = ms_total / args.steps
    value = aggregate_throughput(M, world, ms_per_step)
    e2e_value = aggregate_throughput(M, world, e2e_ms / e_steps)
    kv_block = tb.taq_kv_layout_of(desc).block_bytes * B
    wbytes = tb.taq_packed_weight_bytes(wd_cc)
    qbytes = M * C_ * (1 if shape.q_bits == 8 else 2) + (M * H * 4 if shape.q_bits == 8 else 0)
    img_bytes = tb.taq_kv_layout_of(desc).operand_head_bytes * H * B
    kernels = [
        {"name": "layer_c320_kernel<.,true>: the whole layer pass in one kernel (taq_layer_forward)", "ms": ms_per_step, "in_step": True,
         "bytes": 2 * M * C_ * 2 + 2 * wbytes + img_bytes, "flops": 4 * M * C_ * C_ + 4 * M * T * C_, "traffic": measured_traffic("layer_c320_kernel")},
        {"name": "layer_c320_kernel<.,false>: to_q + Q_a + attention, stand-alone (taq_query_attention)", "ms": stage_ms["qattn"], "in_step": False,
         "bytes": 2 * M * C_ * 2 + wbytes + img_bytes, "flops": 2 * M * C_ * C_ + 4 * M * T * C_, "traffic": None},
        {"name": "linear_sm100_kernel<160>: to_out dequant-GEMM, stand-alone (taq_quantized_linear)", "ms": stage_ms["to_out"], "in_step": False,
         "bytes": 2 * M * C_ * 2 + wbytes, "flops": 2 * M * C_ * C_, "traffic": None},
        {"name": "linear_sm100_kernel<160>: to_q dequant-GEMM + Q_a epilogue, stand-alone (taq_quantized_linear)", "ms": stage_ms["to_q"], "in_step": False,
         "bytes": M * C_ * 2 + qbytes + wbytes, "flops": 2 * M * C_ * C_, "traffic": None},
        {"name": "layer_c320_kernel<.,false,Q given>: attention, stand-alone (taq_cross_attention)", "ms": stage_ms["attn"], "in_step": False,
         "bytes": qbytes + M * C_ * 2 + img_bytes, "flops": 4 * M * T * C_, "traffic": None},
        {"name": "qattn_c320_kernel<.,true,int8>: integer-activation layer pass in one kernel, Q_a(X) and Q_a(O) inside the CTA (taq_layer_forward_a8)", "ms": stage_ms["layer_a8"],
         "in_step": False, "bytes": 2 * M * C_ * 2 + 2 * wbytes + img_bytes, "flops": 4 * M * C_ * C_ + 4 * M * T * C_, "traffic": None},
        {"name": "linear_sm100_kernel<160,int8>: to_out as int8 x int8 -> int32 GEMM, stand-alone (taq_quantized_linear_i8)", "ms": stage_ms["to_out_i8"],
         "in_step": False, "bytes": M * C_ + M * 4 + M * C_ * 2 + wbytes, "flops": 2 * M * C_ * C_, "traffic": None},
    ]
    for k in kernels:
        k["GB/s"] = k["bytes"] / (k["ms"] * 1e-3) / 1e9
        k["TFLOP/s"] = k["flops"] / (k["ms"] * 1e-3) / 1e12
    dom = kernels[0]
    # 378 FLOP per algorithmic byte against a ridge of about 250: the fused layer is bounded by the tensor cores, not HBM
    roofline = {"kernel": dom["name"], "bound": "tensor", "achieved": dom["TFLOP/s"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": dom["TFLOP/s"] / peaks["bf16_tflops"],
                "peak_source": peaks["source"] + ": burst bf16 figure of measured (fp16 operands run at the same rate)", "traffic": dom["traffic"],
                "flops_per_launch": dom["flops"], "bytes_per_launch": dom["bytes"], "ms_per_launch": dom["ms"],
                "hbm": {"achieved_GBps": dom["GB/s"], "peak_GBps": peaks["hbm_gbs"], "frac": dom["GB/s"] / peaks["hbm_gbs"]},
                "stages": [{"name": k["name"], "in_step": k["in_step"], "ms": round(k["ms"], 5), "GB/s": round(k["GB/s"], 1), "TFLOP/s": round(k["TFLOP/s"], 2)} for k in kernels]}
    sm_mhz = clocks.get("sm_mhz") or 0.0
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
            "data": "synthetic",
            "timing": {"replays": rep["replays"], "ms_per_step_median": ms_per_step, "ms_per_step_min": ms_min / args.steps, "ms_per_step_max": ms_max / args.steps,
                       "us_x_sm_mhz": ms_per_step * 1e3 * sm_mhz,
                       "note": "each replay is one CUDA graph of exactly `steps` steps between its own pair of CUDA events; value = median replay"},
            "config": {"workload": WORKLOAD if not args.n_query else WORKLOAD + f" (N overridden to {N})", "kv_projection": "once per prompt, outside the step",
                       "launch": "the K timed steps are one CUDA graph (one kernel launch per step: the whole layer pass), replayed until 0.4 s are timed",
                       "l2_policy": f"inputs larger than L2: ring of {n_sets} buffer sets ({n_sets * set_bytes / 1e6:.0f} MB of activations, L2 {l2 / 1e6:.0f} MB)",
                       "replicas": world},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": M * C_ * 2, "d2h_bytes_per_step": M * C_ * 2, "steps": e_steps},
            "gpu_launches": args.steps,
            "roofline": roofline}
    if not args.no_cpu_baseline:
        t_cpu, n_pass, rows = 0.0, 0, 0
        while t_cpu < args.cpu_seconds and n_pass < 200:      # a bounded sample: whole-layer passes until about 10 s of CPU work
            secs, rows = time_oracle(shape, data, args.cpu_rows)
            t_cpu += secs
            n_pass += 1
        line["cpu_baseline"] = {"value": rows * n_pass / t_cpu, "unit": UNIT, "cores": _oracle_threads(), "kind": "oracle",
                                "sample": f"{n_pass} passes over {rows} query rows ({B} sequences x {rows // B}) of the same layer incl. K/V projection, {t_cpu:.1f} s in total"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
