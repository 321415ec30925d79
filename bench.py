#!/usr/bin/env python
"""Benchmark of the PVQ hot path on B200: group-wise encode + decode throughput.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl reference]

A step is one pass of the whole hot path over one batch: encode of the
workload's matrices and decode back to bf16 (decode only for c4, the fused
round trip for c5).  Inputs are seeded and synthetic (paper_2410_16926_b200.inputs)
and sit in HBM before the timed region; the step rotates through enough buffer
sets that the working set exceeds the L2 cache.  Rank 0 prints ONE JSON line.

With N > 1 (torchrun) every rank runs its own replica of the workload on its
own GPU (rows of a weight set are independent, so there is no collective on the
data path); the value is the sum over ranks divided by the slowest rank's time.

--impl reference times the CPU oracle (the only reference there is: the paper
ships no code) on a bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0

# Per-launch counters of the kernels from the ncu captures summarised under profiles/ (same
# workload and launch configuration as this bench): DRAM bytes read + written, and warp
# instructions executed.  Set an entry to None when its kernel changes until it is re-captured.
NCU_COUNTERS = {
    ("c2_bf16_q_proj", "encode"): {"dram_bytes": 33_969_920 + 1_792, "warp_inst": 32_479_472},
    ("c2_bf16_q_proj", "decode"): {"dram_bytes": 6_658_816 + 473_600, "warp_inst": 37_778_508},
    ("c5_bf16_activations", "roundtrip"): {"dram_bytes": 134_471_936 + 88_764_672, "warp_inst": 214_752_520},
    ("c6_bf16_q_proj_group128", "encode"): {"dram_bytes": 34_222_592 + 5_632, "warp_inst": 89_047_985},
    ("c6_bf16_q_proj_group128", "decode"): {"dram_bytes": 7_047_936 + 222_720, "warp_inst": 81_724_198},
}
SMS, SCHEDULERS_PER_SM = 148, 4      # issue slots per cycle on the part = SMS * SCHEDULERS_PER_SM


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ byte accounting

def compressed_bytes(rows, cols, N, index_bits, scale_bits):
    """Direction codes + amplitude indices + row norms of one matrix, as stored bits."""
    G = cols // N
    return rows * G * index_bits // 8 + rows * G * scale_bits // 8 + rows * 4


def algorithmic_bytes(wl, direction):
    """HBM bytes one launch has to move: encode reads the matrix and writes the compressed
    form; decode reads the compressed form and writes bf16; the fused round trip reads the
    matrix and writes bf16."""
    total = 0
    for m in wl.matrices:
        comp = compressed_bytes(m.rows, m.cols, wl.N, wl.index_bits, wl.scale_bits)
        in_b = m.rows * m.cols * (4 if m.dtype == "f32" else 2)
        out_b = m.rows * m.cols * 2
        if direction == "encode":
            total += in_b + comp
        elif direction == "decode":
            total += comp + out_b
        else:
            total += in_b + out_b
    return total


def make_workload(name):
    from paper_2410_16926_b200 import inputs
    return {"c1": inputs.config1, "c2": inputs.config2, "c3": inputs.config3, "c4": inputs.config4,
            "c5": inputs.config5, "c5r": inputs.config5_unrotated, "c6": inputs.config6, "c7": inputs.config7,
            "c8": inputs.config8, "c9": inputs.config9, "c10": inputs.config10,
            "c10r": inputs.config10_unrotated}[name]()


# ------------------------------------------------------------------------ clocks

class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [s.strip() for s in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------- GPU runner

class DeviceRun:
    """Device state of one workload: tables, codebooks, S rotating buffer sets."""

    def __init__(self, wl, device):
        import torch
        from paper_2410_16926_b200 import pvq
        self.torch, self.pvq, self.wl, self.dev = torch, pvq, wl, device
        N, b = wl.N, wl.scale_bits
        self.K = pvq.max_pulses(N, wl.index_bits)
        self.W = pvq.code_words(N, self.K)
        self.table = pvq.build_count_table(N, self.K, device)
        self.signs = torch.from_numpy(wl.signs).to(device) if wl.signs is not None else None
        self.books = {}
        for m in wl.matrices:
            G = m.cols // N
            if G not in self.books:      # 16-bit amplitudes use no codebook
                self.books[G] = pvq.build_scale_codebook(N, G, b, device) if b <= 8 else (None, None)
        per_set = algorithmic_bytes(wl, "encode") + algorithmic_bytes(wl, "decode")
        self.nsets = max(1, min(16, -(-3 * L2_BYTES // per_set)))
        self.host = [self._host_tensor(m) for m in wl.matrices]
        self.sets = []
        for _ in range(self.nsets):
            items = []
            for m, h in zip(wl.matrices, self.host):
                G = m.cols // N
                codes, sidx, rnorm = pvq.alloc_encoded(m.rows, G, self.W, b, device)
                edges, levels = self.books[G]
                items.append(dict(x=h.to(device), codes=codes, scale_idx=sidx, row_norm=rnorm, edges=edges,
                                  levels=levels, cols=m.cols,
                                  out=torch.empty((m.rows, m.cols), dtype=torch.bfloat16, device=device)))
            self.sets.append(items)
        self.dtype = torch.float32 if wl.matrices[0].dtype == "f32" else torch.bfloat16
        if wl.mode == "decode":          # codes resident in HBM before the timed region
            for items in self.sets:
                pvq.encode_batched(items, self.dtype, N, self.K, b, self.table)
        torch.cuda.synchronize()

    def _host_tensor(self, m):
        t = self.torch.from_numpy(m.data.view(np.int16) if m.dtype == "bf16" else m.data)
        t = t.view(self.torch.bfloat16) if m.dtype == "bf16" else t
        return t.pin_memory()

    # the launches of one step; returns the number of kernels launched
    def encode(self, items):
        self.pvq.encode_batched(items, self.dtype, self.wl.N, self.K, self.wl.scale_bits, self.table)

    def decode(self, items):
        self.pvq.decode_batched(items, self.wl.N, self.K, self.wl.scale_bits, self.table)

    def fused(self, items):
        it = items[0]
        self.pvq.roundtrip(it["x"], self.wl.N, self.K, self.wl.scale_bits, self.table, it["edges"],
                           it["levels"], out=it["out"])

    def fused_rotate(self, items):
        it = items[0]
        self.pvq.rotate_roundtrip(it["x"], self.wl.rot_block, self.signs, self.wl.N, self.K, self.wl.scale_bits,
                                  self.table, it["edges"], it["levels"], out=it["out"])

    def phases(self):
        return {"encode+decode": [("encode", self.encode), ("decode", self.decode)],
                "decode": [("decode", self.decode)],
                "roundtrip": [("roundtrip", self.fused)],
                "rotate_roundtrip": [("rotate_roundtrip", self.fused_rotate)]}[self.wl.mode]

    def run(self, steps, warmup):
        """Returns (total_ms, {phase: [ms per launch]}) timed with CUDA events on the launch stream."""
        torch = self.torch
        phases = self.phases()
        for i in range(warmup):
            for _, fn in phases:
                fn(self.sets[i % self.nsets])
        torch.cuda.synchronize()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(phases) + 1)] for _ in range(steps)]
        for i in range(steps):
            items = self.sets[i % self.nsets]
            ev[i][0].record()
            for j, (_, fn) in enumerate(phases):
                fn(items)
                ev[i][j + 1].record()
        torch.cuda.synchronize()
        total_ms = ev[0][0].elapsed_time(ev[-1][-1])
        per = {name: [ev[i][j].elapsed_time(ev[i][j + 1]) for i in range(steps)]
               for j, (name, _) in enumerate(phases)}
        return total_ms, per

    def run_graph(self, steps, warmup):
        """The same steps replayed from a CUDA graph (one step per buffer set captured through the
        library's calls): the device time of a step without the host's launch work, which is what
        a launch-bound workload otherwise measures.  Returns ms per step."""
        torch = self.torch
        phases = self.phases()
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            for items in self.sets:                    # kernel attributes are set on first use
                for _, fn in phases:
                    fn(items)
            stream.synchronize()
            with torch.cuda.graph(graph, stream=stream):
                for items in self.sets:
                    for _, fn in phases:
                        fn(items)
            replays = max(1, (steps + self.nsets - 1) // self.nsets)
            for _ in range(max(1, warmup // self.nsets)):
                graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(replays):
                graph.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) / (replays * self.nsets)

    def _new_set(self):
        """One more device buffer set (the end-to-end leg wants at least two to overlap steps)."""
        torch, pvq, wl = self.torch, self.pvq, self.wl
        items = []
        for m, h in zip(wl.matrices, self.host):
            G = m.cols // wl.N
            codes, sidx, rnorm = pvq.alloc_encoded(m.rows, G, self.W, wl.scale_bits, self.dev)
            edges, levels = self.books[G]
            items.append(dict(x=torch.empty_like(h, device=self.dev), codes=codes, scale_idx=sidx, row_norm=rnorm,
                              edges=edges, levels=levels, cols=m.cols,
                              out=torch.empty((m.rows, m.cols), dtype=torch.bfloat16, device=self.dev)))
        return items

    def run_e2e(self, steps, warmup):
        """The same step from pinned HOST buffers, through the public API: every step copies its
        inputs host -> device and its results device -> host inside the timed region.  Steps are
        pipelined as a user streaming matrices through the codec would: copies in, kernels and
        copies out run on three streams over two or three device buffer sets, so the transfer of
        one step overlaps the kernels and the opposite transfer of its neighbours.
        Returns (ms per step, h2d bytes, d2h bytes)."""
        torch = self.torch
        wl = self.wl
        while len(self.sets) < 2:
            self.sets.append(self._new_set())
        sets = self.sets[:3]
        S = len(sets)
        host_out = [torch.empty((m.rows, m.cols), dtype=torch.bfloat16).pin_memory() for m in wl.matrices]
        host_codes = [torch.empty_like(it["codes"], device="cpu").pin_memory() for it in sets[0]]
        host_sidx = [torch.empty_like(it["scale_idx"], device="cpu").pin_memory() for it in sets[0]]
        host_rn = [torch.empty_like(it["row_norm"], device="cpu").pin_memory() for it in sets[0]]
        s_main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(S)]
        ev_comp = [torch.cuda.Event() for _ in range(S)]
        ev_free = [torch.cuda.Event() for _ in range(S)]
        used = [False] * S
        h2d = d2h = 0

        def step(i):
            nonlocal h2d, d2h
            h2d = d2h = 0
            k = i % S
            items = sets[k]
            with torch.cuda.stream(s_in):
                if used[k]:
                    s_in.wait_event(ev_free[k])       # the set's previous results have left the device
                if wl.mode in ("encode+decode", "roundtrip", "rotate_roundtrip"):
                    for it, h in zip(items, self.host):
                        it["x"].copy_(h, non_blocking=True)
                        h2d += h.numel() * h.element_size()
                if wl.mode == "decode":            # the compressed form comes from the host
                    for it, hc, hs, hr in zip(items, host_codes, host_sidx, host_rn):
                        it["codes"].copy_(hc, non_blocking=True)
                        it["scale_idx"].copy_(hs, non_blocking=True)
                        it["row_norm"].copy_(hr, non_blocking=True)
                        h2d += hc.numel() * 4 + hs.numel() + hr.numel() * 4
                ev_in[k].record(s_in)
            s_main.wait_event(ev_in[k])
            for _, fn in self.phases():
                fn(items)
            ev_comp[k].record(s_main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[k])
                if wl.mode == "encode+decode":
                    for it, hc, hs, hr in zip(items, host_codes, host_sidx, host_rn):
                        hc.copy_(it["codes"], non_blocking=True)
                        hs.copy_(it["scale_idx"], non_blocking=True)
                        hr.copy_(it["row_norm"], non_blocking=True)
                        d2h += hc.numel() * 4 + hs.numel() + hr.numel() * 4
                for it, ho in zip(items, host_out):
                    ho.copy_(it["out"], non_blocking=True)
                    d2h += ho.numel() * 2
                ev_free[k].record(s_out)
            used[k] = True

        if wl.mode == "decode":
            for it, hc, hs, hr in zip(sets[0], host_codes, host_sidx, host_rn):
                hc.copy_(it["codes"])
                hs.copy_(it["scale_idx"])
                hr.copy_(it["row_norm"])
        for i in range(warmup):
            step(i)
        torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record(s_main)
        s_in.wait_event(t0)
        for i in range(steps):
            step(warmup + i)
        s_main.wait_stream(s_in)
        s_main.wait_stream(s_out)
        t1.record(s_main)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / steps, h2d, d2h


# -------------------------------------------------------------------- CPU oracle

def oracle_sample(wl, target_seconds=12.0):
    """Times the oracle, as it stands, on a bounded sample (leading rows of every matrix) of the
    workload.  Returns (GB/s by the same byte accounting, threads, description)."""
    from oracle import beta_codebook as bc
    from oracle import pvq_oracle as po
    N, b = wl.N, wl.scale_bits
    K = po.max_pulses(N, wl.index_bits)
    W = po.words_for_bits(wl.index_bits)
    books = {}
    for m in wl.matrices:
        G = m.cols // N
        if G not in books:
            books[G] = (bc.edges_f32(N, G, b), bc.levels_amp_f32(N, G, b)) if b <= 8 else (None, None)

    def run(frac_rows, nthreads=0):
        nbytes, t = 0, 0.0
        for m in wl.matrices:
            rows = max(1, min(m.rows, int(round(m.rows * frac_rows))))
            x = np.ascontiguousarray(m.data[:rows])
            e_np, l_np = books[m.cols // N]
            comp = compressed_bytes(rows, m.cols, N, wl.index_bits, b)
            t0 = time.perf_counter()
            if wl.mode == "rotate_roundtrip":
                x = po.rotate(x, wl.rot_block, wl.signs)
            enc = po.encode(x, N, K, b, e_np, W=W, nthreads=nthreads)
            if wl.mode != "decode":
                nbytes += rows * m.cols * (4 if m.dtype == "f32" else 2) + (comp if wl.mode == "encode+decode" else 0)
            t1 = time.perf_counter()
            po.decode(*enc, N, K, b, l_np, nthreads=nthreads)
            t2 = time.perf_counter()
            nbytes += rows * m.cols * 2 + (comp if wl.mode in ("encode+decode", "decode") else 0)
            t += (t2 - t1) if wl.mode == "decode" else (t2 - t0)
        return nbytes, t

    probe = 16.0 / max(m.rows for m in wl.matrices)
    nb, t = run(probe)
    frac = min(1.0, probe * target_seconds / max(t, 1e-4))
    nb, t = run(frac)
    reps = 1
    if frac >= 1.0 and t < target_seconds / 4:       # the whole workload is quick: repeat it for a steadier figure
        reps = int(min(20, max(1, target_seconds / 4 / max(t, 1e-4))))
        for _ in range(reps - 1):
            nb2, t2 = run(frac)
            nb, t = nb + nb2, t + t2
    rows = [max(1, min(m.rows, int(round(m.rows * frac)))) for m in wl.matrices]
    threads = po.threads()
    nb1, t1 = run(max(probe, frac / (2 * threads)), nthreads=1)      # one thread, a sample 2 x threads smaller
    run(probe, nthreads=threads)                                      # (the thread count set by a call stays: put it back)
    return (nb / t / 1e9, threads, "first %s rows of each matrix, %d pass(es), %.1f s" % (rows, reps, t), nb, t,
            nb1 / t1 / 1e9)


# ----------------------------------------------------------------- over the ranks

def max_over_ranks(value, world, device=None):
    """The slowest rank's time: what every multi-GPU number is divided by."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(step_bytes, steps, world, total_ms):
    """GB/s of the whole job: every rank runs its own replica of the workload (rows shard with no
    exchange), so the bytes add up over the ranks and the time is the slowest rank's."""
    return step_bytes * steps * world / (total_ms * 1e-3) / 1e9


# --------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="c2", choices=["c1", "c2", "c3", "c4", "c5", "c5r", "c6", "c7", "c8", "c9", "c10", "c10r"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph", action="store_true",
                    help="also time the steps replayed from a CUDA graph (for launch-bound workloads)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    wl = make_workload(args.config)
    metric = "pvq_%s_throughput" % wl.mode.replace("+", "_")
    dirs = {"encode+decode": ["encode", "decode"], "decode": ["decode"], "roundtrip": ["roundtrip"],
            "rotate_roundtrip": ["rotate_roundtrip"]}[wl.mode]
    step_bytes = sum(algorithmic_bytes(wl, d) for d in dirs)
    config = {"workload": wl.name, "matrices": [[m.name, m.rows, m.cols, m.dtype] for m in wl.matrices],
              "N": wl.N, "index_bits": wl.index_bits, "scale_bits": wl.scale_bits, "mode": wl.mode,
              "weights": wl.weights, "algorithmic_bytes_per_step": step_bytes}

    if args.impl == "reference":
        if rank != 0:
            return
        gbs, threads, sample, nb, t, gbs1 = oracle_sample(wl, target_seconds=max(2.0, min(20.0, 0.05 * args.steps)))
        line = {"impl": "reference", "metric": metric, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
                "steps": args.steps, "warmup": warmup, "ms_per_step": step_bytes / (gbs * 1e9) * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32",
                "data": "synthetic", "config": config,
                "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                 "sample": sample, "single_thread_value": gbs1},
                "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    run = DeviceRun(wl, device)
    config["buffer_sets"] = run.nsets
    config["l2"] = "rotating %d buffer sets, %.0f MB in total, larger than the 126 MB L2" % (
        run.nsets, run.nsets * step_bytes / 1e6)
    config["K"], config["W"] = run.K, run.W

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    total_ms, per = run.run(args.steps, warmup)
    barrier()
    clocks = sampler.stop()
    total_ms = max_over_ranks(total_ms, world, device)
    value = whole_job_value(step_bytes, args.steps, world, total_ms)

    graph_ms = run.run_graph(args.steps, warmup) if args.graph else None

    e2e = None
    if not args.no_e2e:
        e_steps = max(3, min(args.steps, 20))
        ms, h2d, d2h = run.run_e2e(e_steps, 3)
        ms = max_over_ranks(ms, world, device)
        e2e = {"value": whole_job_value(step_bytes, 1, world, ms), "unit": "GB/s", "ms_per_step": ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    kernels = {}
    for name, ms_list in per.items():
        avg = sum(ms_list) / len(ms_list)
        nbytes = algorithmic_bytes(wl, name)
        kernels[name] = {"avg_ms": avg, "median_ms": sorted(ms_list)[len(ms_list) // 2], "min_ms": min(ms_list),
                         "algorithmic_bytes": nbytes,
                         "GBps": nbytes / (avg * 1e-3) / 1e9, "Gweights_per_s": wl.weights / (avg * 1e-3) / 1e9,
                         "frac_of_%s_hbm" % peak_kind: nbytes / (avg * 1e-3) / 1e9 / peak,
                         "frac_of_nominal_8TBps": nbytes / (avg * 1e-3) / 1e9 / 8000.0}
    dom = max(kernels, key=lambda k: kernels[k]["avg_ms"])
    ncu = NCU_COUNTERS.get((wl.name, dom))
    roofline = {"kernel": "pvq %s_kernel" % dom, "bound": "hbm", "achieved": kernels[dom]["GBps"], "peak": peak,
                "peak_source": "%s (MEASURED_PEAKS.json hbm_gbs)" % peak_kind if peak_kind == "measured"
                else "fallback", "unit": "GB/s", "frac": kernels[dom]["GBps"] / peak,
                "traffic": ncu["dram_bytes"] if ncu else None}
    # The limit that binds in practice: instruction issue (every kernel here is integer work
    # on a table walk).  achieved = ncu's warp instructions per launch / measured time,
    # peak = issue slots per second at the SM clock sampled during the run.
    issue = {}
    for name in kernels:
        c = NCU_COUNTERS.get((wl.name, name))
        mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz")
        if c and mhz:
            ach = c["warp_inst"] / (kernels[name]["avg_ms"] * 1e-3)
            pk = SMS * SCHEDULERS_PER_SM * mhz * 1e6
            issue[name] = {"bound": "alu", "achieved": ach / 1e9, "peak": pk / 1e9, "unit": "Gwarp-inst/s",
                           "frac": ach / pk, "warp_inst_per_weight": c["warp_inst"] / wl.weights}

    cpu = None
    if not args.no_cpu_baseline:
        gbs, threads, sample, nb, t, gbs1 = oracle_sample(wl)
        cpu = {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample,
               "single_thread_value": gbs1}

    line = {"metric": metric, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32", "data": "synthetic",
            "config": config, "Gweights_per_s": wl.weights * args.steps * world / (total_ms * 1e-3) / 1e9,
            "kernels": kernels, "roofline": roofline, "issue": issue, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
            "gpu_launches": len(per) * args.steps}
    if graph_ms is not None:
        line["graph_replay"] = {"ms_per_step": graph_ms, "GBps": step_bytes / (graph_ms * 1e-3) / 1e9}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
