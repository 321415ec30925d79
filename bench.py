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
# instructions executed.  They hold for the CUDA sources they were captured from, whose hash
# is recorded with them; with any other sources the line reports them as null.
NCU_SOURCES = "348419117bfdfb77"
NCU_COUNTERS = {
    ("c3_llama3_8b_layer", "encode"): {"dram_bytes": 436_685_056 + 75_231_744, "warp_inst": 415_329_152,
                                       "kernel": "encode_fast_kernel<32,3,bf16>", "profile": "profiles/encode_fast_kernel_c3.md"},
    ("c3_llama3_8b_layer", "decode"): {"dram_bytes": 88_923_904 + 377_352_448, "warp_inst": 255_617_296,
                                       "kernel": "decode_search_kernel<32,3>", "profile": "profiles/decode_search_kernel_c3.md"},
    ("c2_bf16_q_proj", "encode"): {"dram_bytes": 33_675_520 + 0, "warp_inst": 31_428_752,
                                   "kernel": "encode_fast_kernel<32,3,bf16>", "profile": "profiles/encode_fast_kernel_c2.md"},
    ("c2_bf16_q_proj", "decode"): {"dram_bytes": 6_712_064 + 9_216, "warp_inst": 19_980_032,
                                   "kernel": "decode_search_kernel<32,3>", "profile": "profiles/decode_search_kernel_c2.md"},
    ("c4_bf16_down_proj_70b", "decode"): {"dram_bytes": 91_192_832 + 424_887_552, "warp_inst": 648_495_454,
                                          "kernel": "decode_kernel<64,6,int8>", "profile": "profiles/decode_kernel_c4.md"},
    ("c5_bf16_activations", "roundtrip"): {"dram_bytes": 134_330_368 + 91_422_976, "warp_inst": 210_351_000,
                                           "kernel": "encode_fast_kernel<32,2,bf16,FUSED>",
                                           "profile": "profiles/roundtrip_kernel_c5.md"},
}
for _c in NCU_COUNTERS.values():
    _c["kernel_sha"] = NCU_SOURCES
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
    """SM clock and throttle reasons of one GPU, polled through NVML from a thread while the
    bench runs (a few hundred samples per second, each with its host time), so that even a
    timed region of some milliseconds holds samples of its own.  `nvidia-smi -lms` serves
    when NVML cannot be loaded."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, index):
        self.index, self.samples, self.thread, self.proc = index, [], None, None
        self.stop_flag = threading.Event()
        self.sm_max = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))

            def poll():
                while not self.stop_flag.is_set():
                    try:
                        mhz = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
                        why = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                        self.samples.append((time.perf_counter(), float(mhz), int(why)))
                    except Exception:
                        pass
                    time.sleep(0.002)
            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
        except Exception:
            self._start_smi()

    def _physical_index(self):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            ids = [v for v in vis.split(",") if v.strip() != ""]
            if self.index < len(ids) and ids[self.index].strip().isdigit():
                return int(ids[self.index])
        return self.index

    def _start_smi(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self._physical_index()), "--query-gpu=" + q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)

            def read():
                for line in self.proc.stdout:
                    f = [x.strip() for x in line.split(",")]
                    try:
                        why = sum(bit for (_, bit), v in zip(self.REASONS, f[2:6]) if v.lower().startswith("active"))
                        self.samples.append((time.perf_counter(), float(f[0]), why))
                        self.sm_max = float(f[1])
                    except (ValueError, IndexError):
                        pass
            self.thread = threading.Thread(target=read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def stop(self):
        self.stop_flag.set()
        if self.proc:
            self.proc.terminate()
        if self.thread:
            self.thread.join(timeout=5)

    def summary(self, t0, t1):
        """Median SM clock and the throttle reasons seen between host times t0 and t1 (the timed
        region); `samples_under_load` counts everything from warm-up on, whose median is given
        too, since a short region may hold few samples of its own."""
        inside = [x for x in self.samples if t0 <= x[0] <= t1]
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "samples": 0, "reasons": ["no clock samples"]}
        use = inside if inside else self.samples
        why = 0
        for x in use:
            why |= x[2]
        return {"sm_mhz": statistics.median(x[1] for x in use), "sm_max_mhz": self.sm_max,
                "samples": len(inside), "samples_under_load": len(self.samples),
                "sm_mhz_under_load": statistics.median(x[1] for x in self.samples),
                "reasons": sorted(n for n, bit in self.REASONS if why & bit)}


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
    if frac < 1.0 and t < target_seconds / 2:        # the probe overestimated the cost per row: scale once more
        frac = min(1.0, frac * target_seconds / max(t, 1e-4))
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

CONFIGS = ["c1", "c2", "c3", "c4", "c5", "c5r", "c6", "c7", "c8", "c9", "c10", "c10r"]
MODE_DIRS = {"encode+decode": ["encode", "decode"], "decode": ["decode"], "roundtrip": ["roundtrip"],
             "rotate_roundtrip": ["rotate_roundtrip"]}


def kernel_source_sha():
    """Hash of the CUDA sources: the ncu counters typed in above hold only for the sources they
    were captured from."""
    import hashlib
    d = os.path.join(ROOT, "paper_2410_16926_b200", "csrc")
    h = hashlib.sha256()
    for f in sorted(os.listdir(d)):
        if f.endswith((".cu", ".cuh")):
            h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def config_of(wl, K, W):
    step_bytes = sum(algorithmic_bytes(wl, d) for d in MODE_DIRS[wl.mode])
    per_set = algorithmic_bytes(wl, "encode") + algorithmic_bytes(wl, "decode")
    nsets = max(1, min(16, -(-3 * L2_BYTES // per_set)))
    return {"workload": wl.name, "matrices": [[m.name, m.rows, m.cols, m.dtype] for m in wl.matrices],
            "N": wl.N, "index_bits": wl.index_bits, "scale_bits": wl.scale_bits, "mode": wl.mode,
            "weights": wl.weights, "algorithmic_bytes_per_step": step_bytes, "buffer_sets": nsets,
            "l2": ("%d buffer set(s), %.0f MB in total, larger than the 126 MB L2" % (nsets, nsets * step_bytes / 1e6)
                   if nsets * step_bytes > L2_BYTES else
                   "%d buffer sets, %.1f MB: fits the L2 (launch-bound workload)" % (nsets, nsets * step_bytes / 1e6)),
            "K": K, "W": W}


def kernel_table(wl, per, peak, peak_kind):
    kernels = {}
    for name, ms_list in per.items():
        avg = sum(ms_list) / len(ms_list)
        nbytes = algorithmic_bytes(wl, name)
        kernels[name] = {"avg_ms": avg, "median_ms": sorted(ms_list)[len(ms_list) // 2], "min_ms": min(ms_list),
                         "algorithmic_bytes": nbytes,
                         "GBps": nbytes / (avg * 1e-3) / 1e9, "Gweights_per_s": wl.weights / (avg * 1e-3) / 1e9,
                         "frac_of_%s_hbm" % peak_kind: nbytes / (avg * 1e-3) / 1e9 / peak,
                         "frac_of_nominal_8TBps": nbytes / (avg * 1e-3) / 1e9 / 8000.0}
    return kernels


def issue_table(wl, kernels, clocks, sha):
    """The limit that binds in practice: instruction issue (every kernel here is integer work on
    a table walk or a sorting network).  achieved = warp instructions per launch (from the ncu
    capture under profiles/, valid while the sources are unchanged) / the time measured in this
    run; peak = issue slots per second at the SM clock sampled during the run."""
    issue = {}
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz")
    for name in kernels:
        c = NCU_COUNTERS.get((wl.name, name))
        pk = SMS * SCHEDULERS_PER_SM * mhz * 1e6 if mhz else None
        entry = {"bound": "alu", "peak": pk / 1e9 if pk else None, "unit": "Gwarp-inst/s",
                 "peak_source": "148 SMs x 4 schedulers x sampled SM clock"}
        if c and c.get("kernel_sha") == sha and pk:
            ach = c["warp_inst"] / (kernels[name]["avg_ms"] * 1e-3)
            entry.update({"achieved": ach / 1e9, "frac": ach / pk, "warp_inst_per_weight": c["warp_inst"] / wl.weights,
                          "warp_inst_source": "ncu capture %s (not this run)" % c["profile"]})
        else:
            entry.update({"achieved": None, "frac": None, "warp_inst_per_weight": None,
                          "warp_inst_source": "no capture of the current sources"})
        issue[name] = entry
    return issue


def timed_run(run, steps, warmup, sampler, barrier, min_warm_seconds=0.3):
    """W warm-up steps (repeated until the GPU has been busy for min_warm_seconds, so that its
    clocks have settled and the sampler has something to show), then exactly `steps` steps
    between two barriers.  Returns (total_ms, per-kernel ms lists, clock summary)."""
    import torch
    t_w = time.perf_counter()
    run.run(1, warmup)
    while time.perf_counter() - t_w < min_warm_seconds:
        run.run(1, warmup)
    barrier()
    t0 = time.perf_counter()
    total_ms, per = run.run(steps, 0)
    barrier()
    t1 = time.perf_counter()
    return total_ms, per, sampler.summary(t0, t1)


def spawn_ranks(n, argv):
    """`bench.py --gpus N` started without a launcher: start the N ranks, one per GPU."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="c3", choices=CONFIGS,
                    help="the workload of the JSON line; c3 (the full decoder layer) is the largest that "
                         "runs both directions")
    ap.add_argument("--others", default=None,
                    help="comma list of further workloads timed briefly and reported under `other_workloads` "
                         "(default: c2,c4,c5 beside c3 on one GPU; `none` to skip)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph", action="store_true",
                    help="also time the steps replayed from a CUDA graph (for launch-bound workloads)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    warmup = max(args.warmup, 3)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    wl = make_workload(args.config)
    metric = "pvq_%s_throughput" % wl.mode.replace("+", "_")
    step_bytes = sum(algorithmic_bytes(wl, d) for d in MODE_DIRS[wl.mode])

    if args.impl == "reference":
        if rank != 0:
            return
        from oracle import pvq_oracle as po
        K = po.max_pulses(wl.N, wl.index_bits)
        config = config_of(wl, K, po.words_for_bits(wl.index_bits))
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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    run = DeviceRun(wl, device)
    config = config_of(wl, run.K, run.W)
    assert config["buffer_sets"] == run.nsets

    barrier()
    total_ms, per, clocks = timed_run(run, args.steps, warmup, sampler, barrier)
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

    peak, peak_kind = measured_peak()
    sha = kernel_source_sha()

    # the other workloads of the metric, each timed briefly on its own (one GPU only)
    others = args.others if args.others is not None else ("c2,c4,c5" if args.config == "c3" and world == 1 else "none")
    other_lines = {}
    if others != "none":
        del run
        torch.cuda.empty_cache()
        for name in [o for o in others.split(",") if o and o != args.config]:
            wl2 = make_workload(name)
            run2 = DeviceRun(wl2, device)
            o_steps = max(10, min(args.steps, 50))
            ms2, per2, clk2 = timed_run(run2, o_steps, warmup, sampler, barrier)
            sb2 = sum(algorithmic_bytes(wl2, d) for d in MODE_DIRS[wl2.mode])
            other_lines[wl2.name] = {"steps": o_steps, "ms_per_step": ms2 / o_steps,
                                     "value": sb2 * o_steps / (ms2 * 1e-3) / 1e9, "unit": "GB/s",
                                     "config": config_of(wl2, run2.K, run2.W),
                                     "kernels": kernel_table(wl2, per2, peak, peak_kind), "clocks": clk2}
            other_lines[wl2.name]["issue"] = issue_table(wl2, other_lines[wl2.name]["kernels"], clk2, sha)
            del run2
            torch.cuda.empty_cache()
    sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    kernels = kernel_table(wl, per, peak, peak_kind)
    dom = max(kernels, key=lambda k: kernels[k]["avg_ms"])
    ncu = NCU_COUNTERS.get((wl.name, dom))
    if ncu and ncu.get("kernel_sha") != sha:
        ncu = None                      # the kernels have changed since the counters were taken
    roofline = {"kernel": ncu["kernel"] if ncu else "pvq %s kernel" % dom, "bound": "hbm", "achieved": kernels[dom]["GBps"], "peak": peak,
                "peak_source": "%s (MEASURED_PEAKS.json hbm_gbs)" % peak_kind if peak_kind == "measured"
                else "fallback", "unit": "GB/s", "frac": kernels[dom]["GBps"] / peak,
                "traffic": ncu["dram_bytes"] if ncu else None,
                "traffic_source": "ncu capture %s (not this run)" % ncu["profile"] if ncu else None}
    issue = issue_table(wl, kernels, clocks, sha)

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
            "gpu_launches": len(per) * args.steps, "kernel_source_sha": sha}
    if other_lines:
        line["other_workloads"] = other_lines
    if graph_ms is not None:
        line["graph_replay"] = {"ms_per_step": graph_ms, "GBps": step_bytes / (graph_ms * 1e-3) / 1e9}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
