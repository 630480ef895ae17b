#!/usr/bin/env python
"""Benchmark of the LineAR hot path on B200: image tokens/s of compressed-KV decode attention.

One "step" = one whole image generation of the batch through the hot path: reset, prefill append,
then for every visual token and every layer one fused append+decode-attention launch, and at every
line end the score/evict/compact launch of every layer.  Inputs are synthetic (seeded generator of
paper_2512_04857_b200.workloads) and resident in HBM before the timed region; the per-line launch
sequences are captured once into CUDA graphs and replayed.  All layers are cycled every token, so
the working set (GBs) is far larger than L2.

Prints ONE JSON line.  `--impl reference` times the CPU oracle
on a bounded sample instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "image tokens/s of compressed-KV decode attention"
UNIT = "image_tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one decode launch (bytes), from an ncu capture of a 4-layer case of
# the same shape and launch configuration (one launch = one layer, so the capture gives the per-launch figure of the
# full workload); null for shapes that have no capture
NCU_TRAFFIC_PER_LAUNCH = {"janus_pro_7b": 78.0e6, "gqa_1024": 42.4e6, "llamagen_xl": 26.8e6}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_value(images_per_rank, n_visual, world, ms_per_step_max):
    """Image tokens/s of all ranks together: every rank is a replica doing the same work (weak scaling)."""
    return world * images_per_rank * n_visual / (ms_per_step_max * 1e-3)


def _replica_entry(index, n, port, target, args):
    os.environ.update({"RANK": str(index), "LOCAL_RANK": str(index), "WORLD_SIZE": str(n),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    target(args)


def spawn_replicas(n, target, args):
    """`--gpus N` without a launcher: start N processes on this node, one replica per GPU, each with the
    environment torchrun would give it (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR, MASTER_PORT)."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    mp.spawn(_replica_entry, args=(n, port, target, args), nprocs=n, join=True)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        load = [x for x in sm if x >= 0.5 * max(sm)] or sm
        return {"sm_mhz": statistics.median(load), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
def cpu_baseline(w, budget_s: float = 12.0, sample_units: int = 256):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload's independent units.

    The sample is `sample_units` whole (layer, sequence, kv-head) units (every token of the generation, line-end
    evictions included); the same sample is run repeatedly until about `budget_s` seconds of oracle time have
    passed (the oracle's cost does not depend on the values)."""
    import numpy as np
    from oracle import lar_oracle as O
    from paper_2512_04857_b200 import workloads as W
    cfg = O.cfg_from_workload(w)
    total_units = w.n_layers * w.n_units
    out_bytes_per_unit = w.n_visual * w.group * w.head_dim * 8      # the oracle returns fp64 outputs
    n_units = max(1, min(sample_units, total_units, (512 << 20) // out_bytes_per_unit))
    us = []
    for j in range(n_units):
        layer = j % w.n_layers
        s = (j // w.n_layers) % w.batch
        h = (j // (w.n_layers * w.batch)) % w.n_kv_heads
        us.append(W.gen_unit(w, layer, s, h))
    st = lambda key: np.stack([u[key].numpy() for u in us])
    ins = (st("q"), st("k"), st("v"), st("kc"), st("vc"))
    O.run_units(cfg, *[x[:8] for x in ins], want_out=False, want_kept=False)   # page the library in
    passes, dt, thr = 0, 0.0, 1
    while dt < budget_s and passes < 1000:
        t0 = time.perf_counter()
        _, _, thr = O.run_units(cfg, *ins, want_out=True, want_kept=True)
        dt += time.perf_counter() - t0
        passes += 1
    units_per_image = total_units / w.images
    value = (n_units * passes / units_per_image) * w.n_visual / dt
    return {"value": value, "unit": UNIT, "cores": int(thr), "kind": "oracle",
            "sample": f"{n_units} of {total_units} independent (layer, sequence, kv-head) units of '{w.name}', whole "
                      f"generation ({w.n_visual} tokens, line-end evictions), {passes} passes, {dt:.1f} s of oracle time",
            "seconds": dt, "units": n_units * passes}


def run_reference(args):
    from paper_2512_04857_b200 import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = W.WORKLOADS[args.workload]
    if args.score_norm != "mid":
        w = w.scaled(score_norm=args.score_norm)
    vals = []
    cb = None
    for i in range(args.warmup + args.steps):
        cb = cpu_baseline(w, budget_s=max(2.0, min(20.0, 90.0 / max(1, args.warmup + args.steps))))
        if i >= args.warmup:
            vals.append(cb)
    value = sum(c["units"] for c in vals) / sum(c["seconds"] for c in vals) * vals[0]["value"] * vals[0]["seconds"] / vals[0]["units"]
    ms = 1e3 * sum(c["seconds"] for c in vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "score_norm": w.score_norm, "sampled_units_per_step": vals[0]["units"]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cb["cores"], "kind": "oracle",
                             "sample": cb["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
class Runner:
    """Device-resident inputs + per-line CUDA graphs of one workload."""

    def __init__(self, w, dev, args, flags_extra=0, input_lines=0):
        import torch
        from paper_2512_04857_b200 import lar, workloads as W
        self.torch, self.lar, self.w, self.dev = torch, lar, w, dev
        self.per_layer_line_end = bool(getattr(args, "per_layer_line_end", False))
        flags = lar.LAR_FLAG_NO_HOST_CHECKS | flags_extra
        if not args.no_pdl:
            flags |= lar.LAR_FLAG_PDL
        if args.tile_ranges:
            flags |= lar.LAR_FLAG_TILE_RANGES
        if getattr(args, "slot_reuse", False):
            flags |= lar.LAR_FLAG_SLOT_REUSE
        self.cfg = lar.config_from_workload(w, flags=flags, kv_splits=args.kv_splits, warps_per_cta=args.warps,
                                            stages=args.stages, page_tokens=args.page_tokens, decode_ctas=args.ctas)
        self.cache = lar.Cache(self.cfg, device=str(dev))
        L, S, Hq, Hkv, d, n, h = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.line_width, w.n_lines
        dt = w.torch_dtype
        # distinct lines of inputs kept resident (all of them by default); throughput does not depend on the
        # values, so the batch sweep reuses a few lines to bound memory
        hl = self.input_lines = h if input_lines <= 0 else min(h, input_lines)
        self.q = torch.empty((hl, n, L, S, Hq, d), dtype=dt, device=dev)
        self.k = torch.empty((hl, n, L, S, Hkv, d), dtype=dt, device=dev)
        self.v = torch.empty((hl, n, L, S, Hkv, d), dtype=dt, device=dev)
        self.kc = torch.empty((L, S, Hkv, max(w.cond_len, 1), d), dtype=dt, device=dev)
        self.vc = torch.empty_like(self.kc)
        self.out = torch.empty((n, L, S, Hq, d), dtype=dt, device=dev)
        for layer in range(L):
            if w.cond_len:
                a, b = W.gen_prefix(w, layer, dev)
                self.kc[layer], self.vc[layer] = a, b
            for line in range(hl):
                q, k, v = W.gen_tokens(w, layer, line * n, (line + 1) * n, dev)
                self.q[line, :, layer], self.k[line, :, layer], self.v[line, :, layer] = q, k, v
        torch.cuda.synchronize(dev)
        self.graphs = None
        self.launches_per_generation = 0

    def _enqueue_decode(self, line):
        w, c = self.w, self.cache
        line = line % self.input_lines
        for t in range(w.line_width):
            for layer in range(w.n_layers):
                c.decode_step(layer, self.q[line, t, layer], self.k[line, t, layer], self.v[line, t, layer],
                              self.out[t, layer])
        return w.line_width * w.n_layers

    def _enqueue_line_end(self, line):
        w, c = self.w, self.cache
        if line == w.n_lines - 1:
            return 0
        if self.per_layer_line_end:
            for layer in range(w.n_layers):
                c.line_end_score_evict(layer)
            return w.n_layers
        c.line_end_score_evict_all()
        return 1

    def capture(self):
        """Two graphs per line: A = (reset + prefill on line 0) + n x L fused decode steps, B = L line ends."""
        torch = self.torch
        self.graphs = []
        s = torch.cuda.Stream(device=self.dev)
        n0 = self.cache.launch_count()
        with torch.cuda.stream(s):
            for line in range(self.w.n_lines):
                ga = torch.cuda.CUDAGraph()
                with torch.cuda.graph(ga, stream=s):
                    if line == 0:
                        self.cache.reset()
                        if self.w.cond_len:
                            for layer in range(self.w.n_layers):
                                self.cache.append_kv(layer, self.kc[layer], self.vc[layer], self.w.cond_len)
                    self._enqueue_decode(line)
                gb = None
                if line < self.w.n_lines - 1 and not self.w.is_full_cache:
                    gb = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gb, stream=s):
                        self._enqueue_line_end(line)
                self.graphs.append((ga, gb))
        torch.cuda.synchronize(self.dev)
        self.launches_per_generation = self.cache.launch_count() - n0

    def generation(self, events=None):
        """Replay one whole image generation on the current stream; optionally record (start, end) events
        around the decode part of every line."""
        torch = self.torch
        if self.graphs is None:            # eager mode
            for line in range(self.w.n_lines):
                if line == 0:
                    self.cache.reset()
                    if self.w.cond_len:
                        for layer in range(self.w.n_layers):
                            self.cache.append_kv(layer, self.kc[layer], self.vc[layer], self.w.cond_len)
                if events is not None:
                    events[line][0].record()
                self._enqueue_decode(line)
                if events is not None:
                    events[line][1].record()
                self._enqueue_line_end(line)
            return
        for line, (ga, gb) in enumerate(self.graphs):
            if events is not None:
                e0, e1 = events[line]
                e0.record()
                ga.replay()
                e1.record()
            else:
                ga.replay()
            if gb is not None:
                gb.replay()

    def close(self):
        self.graphs = None
        self.cache.close()
        self.q = self.k = self.v = self.out = None


def time_generations(r: Runner, steps: int, warmup: int, dist=None, sampler=None):
    torch = r.torch
    dev = r.dev
    for _ in range(warmup):
        r.generation()
    torch.cuda.synchronize(dev)
    evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            for _ in range(r.w.n_lines)] for _ in range(steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(dev)
    if sampler:
        sampler.start()
    start.record()
    for s in range(steps):
        r.generation(evs[s])
    stop.record()
    torch.cuda.synchronize(dev)
    clocks = sampler.stop() if sampler else None
    if dist is not None:
        dist.barrier()
    total_ms = start.elapsed_time(stop)
    decode_ms = sum(e0.elapsed_time(e1) for step in evs for (e0, e1) in step)
    n = r.w.line_width
    half = r.w.n_lines // 2
    first_ms = sum(e0.elapsed_time(e1) for step in evs for (e0, e1) in step[:half]) / (steps * half * n)
    last_ms = sum(e0.elapsed_time(e1) for step in evs for (e0, e1) in step[half:]) / (steps * (r.w.n_lines - half) * n)
    return total_ms, decode_ms, clocks, (first_ms, last_ms)


def measure_e2e(w, dev, args, steps=3):
    """Same metric through the host-buffer entry point: every layer-step copies q, k, v from pinned host
    memory, runs the fused kernel and copies the output back (all inside the timed region)."""
    import torch
    from paper_2512_04857_b200 import lar, workloads as W
    flags = lar.LAR_FLAG_NO_HOST_CHECKS | lar.LAR_FLAG_HOST_DEFER_OUT
    if not args.no_pdl:
        flags |= lar.LAR_FLAG_PDL
    cfg = lar.config_from_workload(w, flags=flags, kv_splits=args.kv_splits, warps_per_cta=args.warps,
                                   stages=args.stages, page_tokens=args.page_tokens, decode_ctas=args.ctas)
    cache = lar.Cache(cfg, device=str(dev))
    L, S, Hq, Hkv, d, n, h = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.line_width, w.n_lines
    dt = w.torch_dtype
    # one line of pinned host inputs, reused for every line (throughput does not depend on the values); q | k | v of a
    # layer-step are adjacent, as they leave a fused QKV projection: the entry point then moves them in one copy
    nq, nk = S * Hq * d, S * Hkv * d
    hqkv = torch.empty((n, L, nq + 2 * nk), dtype=dt).pin_memory()
    hq = hqkv[..., :nq].unflatten(-1, (S, Hq, d))
    hk = hqkv[..., nq:nq + nk].unflatten(-1, (S, Hkv, d))
    hv = hqkv[..., nq + nk:].unflatten(-1, (S, Hkv, d))
    ho = torch.empty((n, L, S, Hq, d), dtype=dt).pin_memory()
    for layer in range(L):
        q, k, v = W.gen_tokens(w, layer, 0, n, dev)
        hq[:, layer], hk[:, layer], hv[:, layer] = q.cpu(), k.cpu(), v.cpu()
    kc = torch.zeros((L, S, Hkv, max(w.cond_len, 1), d), dtype=dt, device=dev)
    s = torch.cuda.Stream(device=dev)
    graphs = []
    with torch.cuda.stream(s):
        # one graph per line, captured in order (a graph holds the cache lengths of the steps it was captured at)
        for line in range(h):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                if line == 0:
                    cache.reset()
                    if w.cond_len:
                        for layer in range(L):
                            cache.append_kv(layer, kc[layer], kc[layer], w.cond_len)
                for t in range(n):
                    for layer in range(L):
                        cache.decode_step_host(layer, hq[t, layer], None, None, ho[t, layer])   # q | k | v packed
                cache.host_join()                             # the line's last copy-outs re-join the stream
                if line < h - 1 and not w.is_full_cache:
                    if args.per_layer_line_end:
                        for layer in range(L):
                            cache.line_end_score_evict(layer)
                    else:
                        cache.line_end_score_evict_all()      # one launch for every layer, as in the headline
            graphs.append(g)

        def gen():
            for g in graphs:
                g.replay()
        for _ in range(2):
            gen()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            gen()
        e1.record()
        torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / steps
    bits = cache.poll_device_status()
    cache.close()
    qb = S * Hq * d * w.elt_bytes
    kb = S * Hkv * d * w.elt_bytes
    return {"ms": ms, "steps": steps, "h2d": w.n_visual * L * (qb + 2 * kb), "d2h": w.n_visual * L * qb, "status_bits": bits}


def run_ours(args):
    import torch
    from paper_2512_04857_b200 import lar, workloads as W
    lar.lib()  # fail loudly if the CUDA library is missing
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group(backend="nccl", device_id=torch.device(f"cuda:{local}"))
        dist = dist_mod
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    peak, peak_kind = load_peaks()
    w = W.WORKLOADS[args.workload]
    if args.layers:
        w = w.scaled(n_layers=args.layers)
    if args.score_norm != "mid":
        w = w.scaled(score_norm=args.score_norm)

    def bench_workload(wl, steps, warmup, sample_clocks, input_lines=0):
        r = Runner(wl, dev, args, input_lines=input_lines)
        if args.eager:
            r.launches_per_generation = (wl.n_layers * (wl.n_visual + (1 if wl.cond_len else 0))
                                         + (0 if wl.is_full_cache else
                                            (wl.n_layers if r.per_layer_line_end else 1) * (wl.n_lines - 1)))
        else:
            r.capture()
        sampler = ClockSampler(local) if sample_clocks else None
        total_ms, decode_ms, clocks, halves = time_generations(r, steps, warmup, dist, sampler)
        bits = r.cache.poll_device_status()
        plan = r.cache.plan
        res = {"ms_per_step": total_ms / steps, "decode_ms_per_step": decode_ms / steps, "clocks": clocks,
               "launches": r.launches_per_generation, "status_bits": bits,
               "plan": {"kv_splits": plan.kv_splits, "warps_per_cta": plan.warps_per_cta, "stages": plan.stages,
                        "page_tokens": plan.page_tokens, "decode_smem_bytes": plan.decode_smem_bytes,
                        "decode_ctas": plan.decode_ctas},
               "per_token_ms_first_half": halves[0], "per_token_ms_last_half": halves[1]}
        r.close()
        torch.cuda.empty_cache()
        return res

    def roofline_of(wl, decode_ms_per_step):
        kvb = wl.kv_bytes_per_generation()
        nd = wl.n_visual * wl.n_layers
        ach = kvb / (decode_ms_per_step * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": "decode_stream_kernel (fused append + decode attention)",
                "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_kind": f"of {peak_kind} copy bandwidth", "frac_of_8TBs": ach / 8000.0,
                "algorithmic_bytes_per_launch": kvb / nd, "avg_launch_us": decode_ms_per_step * 1e3 / nd,
                "traffic": NCU_TRAFFIC_PER_LAUNCH.get(wl.name)}

    main = bench_workload(w, args.steps, args.warmup, True)
    ms_step, ms_decode = max_over_ranks([main["ms_per_step"], main["decode_ms_per_step"]], dist, dev)
    value = whole_job_value(w.images, w.n_visual, world, ms_step)
    kv_bytes = w.kv_bytes_per_generation()
    n_decode = w.n_visual * w.n_layers

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "layers": w.n_layers, "sequences": w.batch, "images": w.images,
                       "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                       "storage": w.dtype, "prefix": w.cond_len, "grid": f"{w.n_lines}x{w.line_width}",
                       "budget_lines": w.budget_lines, "anchor": w.anchor_len, "recent_lines": w.recent_lines,
                       "score_norm": w.score_norm,
                       "launch": ("cuda-graph per line, fused append+decode" + (", PDL" if not args.no_pdl else "") +
                                  (", line end per layer" if args.per_layer_line_end else ", one line-end launch for all layers") +
                                  (", slot reuse instead of compaction" if args.slot_reuse else "")),
                       "l2": "inputs larger than L2: all layers cycled every token "
                             f"({kv_bytes / n_decode / 1e6:.0f} MB per launch x {w.n_layers} layers)",
                       "plan": main["plan"], "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
            "clocks": main["clocks"],
            "gpu_launches": main["launches"] * args.steps,
            "roofline": roofline_of(w, ms_decode),
            "sequence_tokens_per_s": world * w.batch * w.n_visual / (ms_step * 1e-3),
            "line_end_ms_per_step": ms_step - ms_decode,
            "per_token_ms": {"first_half": main["per_token_ms_first_half"], "last_half": main["per_token_ms_last_half"]},
            "device_status_bits": main["status_bits"]}

    # ---- speedup over the library's own full-cache path on the same inputs
    if not args.no_full:
        full = bench_workload(w.full_cache(), max(1, min(args.steps, 2)), 1, False)
        fm = torch.tensor([full["ms_per_step"]], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(fm, op=dist.ReduceOp.MAX)
        line["full_cache"] = {"ms_per_step": float(fm[0]), "value": world * w.images * w.n_visual / (float(fm[0]) * 1e-3),
                              "per_token_ms": {"first_half": full["per_token_ms_first_half"],
                                               "last_half": full["per_token_ms_last_half"]}}
        line["speedup_vs_full_cache"] = float(fm[0]) / ms_step
    # ---- end to end through host buffers
    if not args.no_e2e:
        e = measure_e2e(w, dev, args)
        em = torch.tensor([e["ms"]], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(em, op=dist.ReduceOp.MAX)
        line["e2e"] = {"value": world * w.images * w.n_visual / (float(em[0]) * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": e["h2d"], "d2h_bytes_per_step": e["d2h"], "ms_per_step": float(em[0]),
                       "steps": e["steps"], "warmup": 2, "device_status_bits": e["status_bits"],
                       "api": "lar_decode_step_host (pinned host q|k|v -> device, kernel, out -> host) per layer-step; "
                              "copies on the library's own streams overlap the neighbouring calls' kernels (deferred copy-out, "
                              "joined once per line), one CUDA graph per line, same launch configuration as the headline "
                              "(programmatic dependent launch, one line-end launch for all layers)"}
    # ---- other benchmark shapes (not the headline line)
    if args.also:
        line["also"] = {}
        for name in args.also.split(","):
            w2 = W.WORKLOADS[name]
            if name == w.name:
                continue
            n2 = max(1, min(args.steps, 3))
            r2 = bench_workload(w2, n2, 3, True)
            ms2, dec2 = max_over_ranks([r2["ms_per_step"], r2["decode_ms_per_step"]], dist, dev)
            line["also"][name] = {"value": whole_job_value(w2.images, w2.n_visual, world, ms2), "unit": UNIT,
                                  "ms_per_step": ms2, "steps": n2, "warmup": 3, "roofline": roofline_of(w2, dec2),
                                  "line_end_ms_per_step": ms2 - dec2, "plan": r2["plan"], "clocks": r2["clocks"],
                                  "device_status_bits": r2["status_bits"]}
    # ---- batch sweep of one shape, compressed and full-cache (not the headline line)
    if args.batch_sweep:
        wb = W.WORKLOADS[args.sweep_workload]
        line["batch_sweep"] = {"workload": wb.name, "inputs": "2 lines of inputs reused for every line", "points": []}
        for b in [int(x) for x in args.batch_sweep.split(",")]:
            w2 = wb.scaled(batch=2 * b, images=b)
            rc = bench_workload(w2, 1, 1, False, input_lines=2)
            ach = w2.kv_bytes_per_generation() / (rc["decode_ms_per_step"] * 1e-3) / 1e9
            pt = {"images": b, "sequences": 2 * b, "value": world * b * w2.n_visual / (rc["ms_per_step"] * 1e-3),
                  "ms_per_step": rc["ms_per_step"], "decode_launch_us": rc["decode_ms_per_step"] * 1e3 / (w2.n_visual * w2.n_layers),
                  "roofline_achieved_gbs": ach, "roofline_frac": ach / peak, "frac_of_8TBs": ach / 8000.0, "plan": rc["plan"]}
            if not args.no_full:
                rf = bench_workload(w2.full_cache(), 1, 1, False, input_lines=2)
                pt["full_cache_ms_per_step"] = rf["ms_per_step"]
                pt["speedup_vs_full_cache"] = rf["ms_per_step"] / rc["ms_per_step"]
            line["batch_sweep"]["points"].append(pt)
    # ---- budget-ratio sweep at a given batch (the layout of the paper's efficiency table; not the headline line)
    if args.ratio_sweep:
        wr = W.WORKLOADS[args.sweep_workload]
        if args.sweep_images:
            wr = wr.scaled(batch=2 * args.sweep_images, images=args.sweep_images)
        rf = bench_workload(wr.full_cache(), 1, 1, False, input_lines=2)
        full_slab = lar.lar_cache_slab_bytes(lar.config_from_workload(wr.full_cache()))
        line["ratio_sweep"] = {"workload": wr.name, "images": wr.images, "sequences": wr.batch,
                               "full_cache": {"ms_per_step": rf["ms_per_step"], "kv_slab_gb": full_slab / 1e9,
                                              "value": world * wr.images * wr.n_visual / (rf["ms_per_step"] * 1e-3)},
                               "points": []}
        for b in [int(x) for x in args.ratio_sweep.split(",")]:
            w2 = wr.scaled(budget_lines=b, recent_lines=max(1, (b - 2) // 2), anchor_len=wr.line_width)
            rc = bench_workload(w2, 1, 1, False, input_lines=2)
            slab = lar.lar_cache_slab_bytes(lar.config_from_workload(w2))
            ach = w2.kv_bytes_per_generation() / (rc["decode_ms_per_step"] * 1e-3) / 1e9
            line["ratio_sweep"]["points"].append(
                {"budget_lines": b, "budget_tokens": w2.budget_tokens, "ratio": f"{b}/{w2.n_lines}",
                 "recent_lines": w2.recent_lines, "mid_len": w2.mid_len,
                 "value": world * w2.images * w2.n_visual / (rc["ms_per_step"] * 1e-3), "ms_per_step": rc["ms_per_step"],
                 "speedup_vs_full_cache": rf["ms_per_step"] / rc["ms_per_step"], "kv_slab_gb": slab / 1e9,
                 "memory_saving": 1.0 - slab / full_slab, "roofline_achieved_gbs": ach, "roofline_frac": ach / peak})
    # ---- CPU oracle on the host cores (rank 0, N = 1 only)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = {k: v for k, v in cpu_baseline(w).items() if k not in ("seconds", "units")}
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="janus_pro_7b")
    ap.add_argument("--also", default="gqa_1024",
                    help="comma-separated extra workloads reported under 'also' with the headline's roofline fields "
                         "(default: the 1024-px GQA shape, the other shape the target is stated on; '' for none)")
    ap.add_argument("--batch-sweep", default="", help="comma-separated image counts: sweep the batch of --sweep-workload")
    ap.add_argument("--sweep-workload", default="gqa_1024")
    ap.add_argument("--ratio-sweep", default="", help="comma-separated line budgets: sweep the budget of --sweep-workload")
    ap.add_argument("--sweep-images", type=int, default=0, help="images per batch in --ratio-sweep (0: the workload's own)")
    ap.add_argument("--kv-splits", type=int, default=0)
    ap.add_argument("--warps", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--page-tokens", type=int, default=0)
    ap.add_argument("--ctas", type=int, default=0, help="CTAs of the persistent decode grid (0: one per SM)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling / small cases)")
    ap.add_argument("--eager", action="store_true", help="plain stream launches instead of CUDA graphs (profiling)")
    ap.add_argument("--no-pdl", action="store_true")
    ap.add_argument("--per-layer-line-end", action="store_true", help="one line-end launch per layer instead of one for all layers")
    ap.add_argument("--tile-ranges", action="store_true", help="deal 32-row tiles, not whole units, to the decode CTAs")
    ap.add_argument("--score-norm", default="mid", choices=["mid", "cache", "accum"],
                    help="line-end scoring: Eq. 9 over the mid keys (as written), over the whole live cache (variant), or "
                         "attention accumulated over all decode steps (the paper's 'w. AttAcc' ablation)")
    ap.add_argument("--slot-reuse", action="store_true",
                    help="line end without compaction: the evicted slots take the newest line's rows (LAR_FLAG_SLOT_REUSE)")
    ap.add_argument("--no-full", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_replicas(args.gpus, run_ours, args)   # plain `python bench.py --gpus N`: start the N replicas here
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
