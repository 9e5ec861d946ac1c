#!/usr/bin/env python
"""Benchmark of the block-rotated MXFP4 W4A4 linear layer on B200.

One *step* = one pass of the whole hot path — fused block-Hadamard rotation + MXFP4 quantisation
of the activations, then the block-scaled MXFP4 GEMM against pre-packed weights — over every
shape of the workload.  Default workload: cfg5, the 70B-shaped layer K = 8192, N = 28672 with
M in {1, 16, 128, 1024, 8192, 32768} tokens (the largest single-GPU workload of the five).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg1|cfg2|cfg3|cfg4] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is device-timed throughput with inputs resident in HBM;
`e2e` is the same metric through the host-buffer entry point (H2D of x and D2H of y inside the
timed region); `roofline` describes the dominant kernel (the GEMM on the tensor-bound shapes,
M >= 1024) timed per launch with CUDA events — its `operand_data_effect` times one of those launches
on the real operands and on all-zero codes, which separates the kernel from the chip's power
management —, `decode` the weight-streaming shapes (M <= 128) against the HBM copy bandwidth; `per_config` repeats the per-kernel figures for the other
workloads (cfg2, cfg3 and the block-size sweep cfg4) in the same process; `cpu_baseline` is the
CPU oracle on a bounded sample.  With --gpus N > 1 every rank runs an independent replica — the
path has no cross-GPU exchange; when no launcher has set WORLD_SIZE the script starts its N ranks
itself.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "MXFP4 W4A4 linear TFLOPS (rotate+quantize+GEMM)"
UNIT = "TFLOP/s"
L2_BYTES = 126 * 1024 * 1024
FP4_OVER_BF16 = 4.0          # nominal dense fp4 : bf16 tensor throughput ratio on B200 (9 : 2.25)
NOMINAL_FP4_TFLOPS = 9000.0  # dense FP4 tensor peak of one B200 (vendor figure)
NOMINAL_HBM_GBS = 8000.0     # vendor HBM3e figure


def workload_shapes(name):
    from paper_2511_04214_b200 import synth
    cfg = synth.CONFIGS[name]
    shapes = [s for s in cfg["shapes"] if s[2] > 0]
    return cfg, shapes


def select_shapes(args):
    """The workload's shapes, or the single one picked with --shape-index (seed offsets kept)."""
    cfg, shapes = workload_shapes(args.workload)
    idx = list(range(len(shapes)))
    if args.shape_index >= 0:
        idx = [args.shape_index]
    return cfg, [shapes[i] for i in idx], idx


# DRAM traffic of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum per launch) from ncu:
#   ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum,\
#       sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed --clock-control none -k regex:gemm_mxfp4 -s 3 -c 2 \
#       python bench.py --workload cfg5 --shape-index 4 --steps 4 --warmup 3 --no-graph --no-e2e --no-cpu-baseline --no-per-config
# i.e. ONE shape of the default workload, M = 8192 (K = 8192, N = 28672: 1.6 GB on the device, and a 470 MB
# output that does not fit the 126 MB L2, so written bytes do reach DRAM).  The traffic of this kernel grows
# in proportion to M for a fixed weight matrix (the packed weights are re-read once per raster band of 8
# tile rows of 256, the output is written once), so the figure for the whole record is the captured one scaled by
# the rows processed.  "cfg3" holds the one shape captured with `--set full -k regex:gemm_mxfp4 -s 3 -c 2`
# under `--workload cfg3 --shape-index 1`, "cfg4" the block-32 kernel captured with `-k
# regex:rotate_quantize_direct -s 6 -c 2` under `--workload cfg4 --only-block --block 32`.
# The figures belong to one exact version of the kernels: every entry names the kernel source files it was
# captured on and their SHA-256 at capture time, and the benchmark reports null once they have changed.
# (Which GEMM kernel runs for a shape is decided in bro.cu; gemm_kernel_name() below restates that rule
# and the launch list under profiles/ shows it in effect at capture time.)
GEMM_SOURCES = ("bro_common.cuh", "gemm_mxfp4.cuh", "gemm_mxfp4_2cta.cuh")
RQ_SOURCES = ("bro_common.cuh", "rotate_quantize.cuh", "rotate_quantize_direct.cuh")
NCU_TRAFFIC = {
    "cfg5": {"sources": GEMM_SOURCES, "digest": "096c61cb1b9865ca985e775b0d340c5efb1060c2d39547c30f96dd9d3d65fab1",
             "per_row_of": (8192, 8192, 28672), "bytes": 535339776 + 441953536},
    "cfg3": {"sources": GEMM_SOURCES, "digest": "096c61cb1b9865ca985e775b0d340c5efb1060c2d39547c30f96dd9d3d65fab1",
             "shapes": {(4096, 4096, 14336): 68345088 + 69353728}},
    "cfg4": {"sources": RQ_SOURCES, "digest": "aa6e030cc76b05e3c4883ecbdfdbfc516261469c9425d0325a4fb2e97853c75c",
             "shapes": {(16384, 4096, 32): 134233600 + 19132928}},
}


def kernel_sources_digest(files=None):
    """SHA-256 over the named files of csrc/ (all of them if none are named)."""
    import glob
    import hashlib
    csrc = os.path.join(ROOT, "paper_2511_04214_b200", "csrc")
    paths = sorted(glob.glob(os.path.join(csrc, "*"))) if files is None else [os.path.join(csrc, f) for f in files]
    h = hashlib.sha256()
    for f in paths:
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(workload, shapes):
    """Bytes per step for the dominant kernel from the recorded ncu capture, or None if the capture
    does not cover this workload or the kernels have changed since it was taken."""
    table = NCU_TRAFFIC.get(workload)
    if table is None or kernel_sources_digest(table["sources"]) != table["digest"]:
        return None
    if "per_row_of" in table:
        # one captured shape; the others share its K and N, and traffic grows in proportion to the rows
        M0, K0, N0 = table["per_row_of"]
        if any((K, N) != (K0, N0) for (M, K, N) in shapes):
            return None
        return float(table["bytes"]) * sum(M for (M, K, N) in shapes) / M0
    try:
        return float(sum(table["shapes"][tuple(s)] for s in shapes))
    except KeyError:
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(value, dist, device):
    """The largest `value` over all ranks of the job (the job's time is its slowest rank's)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank_per_step, steps, world, ms_max):
    """Whole-job throughput: every rank runs an independent replica of the workload (weak scaling,
    no exchange on the data path), so the job processed world * steps * units in the time of the
    slowest rank."""
    return units_per_rank_per_step * steps * world / (ms_max * 1e-3)


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the GPU works."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.marks = {}
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def mark(self, name):
        self.marks[name] = time.time()

    def window(self, t0, t1):
        """Median SM clock, highest power reading and throttle reasons of the samples taken in [t0, t1]."""
        sm, power, reasons = [], [], set()
        for (t, line) in list(self.rows):
            f = [v.strip() for v in line.split(",")]
            if len(f) < 9 or not (t0 <= t <= t1):
                continue
            try:
                sm.append(float(f[1]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "power_w_max": max(power) if power else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        t0, t1 = self.marks.get("t0", 0), self.marks.get("t1", float("inf"))
        inside, allc, smax, reasons, power = [], [], None, set(), []
        for (t, line) in self.rows:
            f = [v.strip() for v in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm, mx = float(f[1]), float(f[2])
            except ValueError:
                continue
            smax = mx
            allc.append(sm)
            if t0 <= t <= t1 + 0.1:
                inside.append(sm)
                try:
                    power.append(float(f[3]))
                except ValueError:
                    pass
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        use = inside if inside else allc
        return {"sm_mhz": statistics.median(use) if use else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples_in_timed_region": len(inside),
                "power_w_max": max(power) if power else None}


# ------------------------------------------------------------------------------------------------
def oracle_prepare(shapes, cfg, rows_per_shape, block, idx=None):
    """Inputs for the CPU oracle: the first `rows_per_shape` rows of every shape, weights packed by
    the oracle (offline, untimed)."""
    import oracle
    from paper_2511_04214_b200 import synth
    prepared = []
    for j, (M, K, N) in enumerate(shapes):
        i = idx[j] if idx is not None else j
        m = min(M, rows_per_shape)
        x = synth.activations(m, K, seed=cfg["seed"] + i, recipe=cfg["recipe"])
        key = (N, K, cfg["seed"] + i, block)
        if key not in _PACKED_BY_ORACLE:
            w = synth.weights(N, K, seed=cfg["seed"] + i)
            _PACKED_BY_ORACLE[key] = oracle.pack_weights(synth.bf16_bits(w), block)
        wc, ws = _PACKED_BY_ORACLE[key]
        prepared.append((synth.bf16_bits(x), wc, ws, m, K, N))
    return prepared


_PACKED_BY_ORACLE = {}      # offline weight packing by the oracle, done once per weight matrix


def oracle_step(prepared, block):
    """One pass of the oracle's whole layer over the prepared sample.  Returns (seconds, flops)."""
    import oracle
    t0 = time.perf_counter()
    flops = 0.0
    for (xb, wc, ws, m, K, N) in prepared:
        oracle.linear(xb, block, wc, ws)
        flops += 2.0 * m * K * N
    return time.perf_counter() - t0, flops


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload,
    sized so that warmup + steps finish in about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfg, shapes, idx = select_shapes(args)
    rows = args.ref_rows
    if rows <= 0:
        t1, _ = oracle_step(oracle_prepare(shapes, cfg, 1, args.block, idx), args.block)
        t1, _ = oracle_step(oracle_prepare(shapes, cfg, 1, args.block, idx), args.block)
        rows = int(max(1, min(64, 120.0 / (max(args.steps + args.warmup, 1) * max(t1, 1e-4)))))
    prepared = oracle_prepare(shapes, cfg, rows, args.block, idx)
    for _ in range(max(args.warmup, 0)):
        oracle_step(prepared, args.block)
    total_t, total_f = 0.0, 0.0
    for _ in range(args.steps):
        t, f = oracle_step(prepared, args.block)
        total_t += t
        total_f += f
    value = total_f / total_t / 1e12
    sample = f"first {rows} rows of each of {len(shapes)} shapes per step (weights packed offline, untimed)"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_t / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": args.workload, "shapes_MKN": shapes, "block": args.block,
                                         "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------------
class Layers:
    """Device-resident inputs of one workload: per shape a ring of independent activation / weight /
    output / workspace sets, so that consecutive launches never find their operands in L2 (126 MB)."""

    def __init__(self, bro, synth, cfg, shapes, idx, block, dev, randomised=False, max_ring=8):
        import torch
        self.bro, self.shapes, self.block, self.dev = bro, shapes, block, dev
        self.per_step_bytes = sum(M * K * 2 + N * K // 2 + M * N * 2 for (M, K, N) in shapes)
        self.ring = max(2, min(max_ring, -(-3 * L2_BYTES // self.per_step_bytes)))
        # --randomised: R_i = diag(s) H / sqrt(block) with a seeded +-1 vector per layer (Sec. 5.1)
        self.signs = [synth.rotation_signs(K, seed=cfg["seed"] + idx[j]).to(dev) if randomised else None
                      for j, (M, K, N) in enumerate(shapes)]
        self.sets = []
        wcache = {}
        for j, (M, K, N) in enumerate(shapes):
            i = idx[j]
            wkey = (N, K, cfg["seed"] + i)
            if wkey not in wcache:
                wcache.clear()                  # (one bf16 weight matrix on the device at a time)
                wcache[wkey] = synth.weights(N, K, seed=cfg["seed"] + i).to(dev)
            w = wcache[wkey]
            x0 = synth.activations(M, K, seed=cfg["seed"] + i, recipe=cfg["recipe"]).to(dev)
            ws_bytes = bro.linear_workspace_bytes(M, N, K)
            per_ring = []
            for r in range(self.ring):
                wcodes = bro.alloc_codes(N, K, dev)
                wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM, dev)
                if self.signs[j] is not None:
                    bro.pack_weights_rs(w, block, self.signs[j], wcodes, wscales)   # offline, untimed
                else:
                    bro.pack_weights(w, block, wcodes, wscales)                     # offline, untimed
                x = x0 if r == 0 else x0.roll(r * 7, 0).contiguous()   # same statistics, separate memory
                per_ring.append({"x": x, "wcodes": wcodes, "wscales": wscales,
                                 "y": torch.empty((M, N), dtype=torch.bfloat16, device=dev),
                                 "ws": bro.alloc_workspace(ws_bytes, dev)})
            self.sets.append(per_ring)
        wcache.clear()
        torch.cuda.synchronize()

    def step(self, r):
        bro = self.bro
        for i, (M, K, N) in enumerate(self.shapes):
            s = self.sets[i][r % self.ring]
            if self.signs[i] is not None:
                bro.linear_rs(s["x"], self.block, self.signs[i], s["wcodes"], s["wscales"], N, s["y"], s["ws"])
            else:
                bro.linear(s["x"], self.block, s["wcodes"], s["wscales"], N, s["y"], s["ws"])

    def views(self, i, r):
        M, K, N = self.shapes[i]
        s = self.sets[i][r]
        nc = self.bro.codes_bytes(M, K)
        off = (nc + 1023) // 1024 * 1024
        sc = self.bro.scales_bytes(M, K, self.bro.LAYOUT_GEMM)
        off2 = (off + sc + 1023) // 1024 * 1024
        return s, s["ws"][:nc], s["ws"][off:off + sc], s["ws"][off2:]

    def flops_per_step(self):
        return sum(2.0 * M * K * N for (M, K, N) in self.shapes)


def time_steps(layers, steps, warmup, use_graph, barrier, sampler=None):
    """Device time of `steps` whole-layer steps (rounded up to a multiple of the ring when replaying a
    CUDA graph of one ring of steps).  Returns (milliseconds on this rank, steps actually run)."""
    import torch
    for i in range(max(warmup, 3)):            # also sets kernel attributes before any graph capture
        layers.step(i)
    torch.cuda.synchronize()
    graph = None
    ring = layers.ring
    if use_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for r in range(ring):
                layers.step(r)
        graph.replay()
        torch.cuda.synchronize()
        replays = max(1, -(-steps // ring))
        steps = replays * ring
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler is not None:
        sampler.mark("t0")
    e0.record()
    if graph is not None:
        for _ in range(replays):
            graph.replay()
    else:
        for i in range(steps):
            layers.step(i)
    e1.record()
    barrier()
    if sampler is not None:
        sampler.mark("t1")
    return e0.elapsed_time(e1), steps


def time_kernels(layers, groups):
    """Per-kernel device times: the two C-ABI calls bro_linear makes, each timed with CUDA events
    around a group of `ring` back-to-back launches (one per ring set, so no launch finds its operands
    in L2); per-launch time = group time / ring.  Timing every launch with its own pair of events adds
    microseconds of event latency to kernels that only run for ten.  Returns (rq_ms, gemm_ms) per shape."""
    import torch
    bro, shapes, ring, block = layers.bro, layers.shapes, layers.ring, layers.block
    rq_ev = [[] for _ in shapes]
    gemm_ev = [[] for _ in shapes]
    torch.cuda._sleep(int(4e7))        # hold the stream (~20 ms) while the launches below queue up
    for it in range(groups + 2):
        for i, (M, K, N) in enumerate(shapes):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            ev[0].record()
            for r in range(ring):
                s, acodes, ascales, _ = layers.views(i, r)
                if layers.signs[i] is not None:
                    bro.rotate_quantize_mxfp4_rs(s["x"], block, layers.signs[i], acodes, ascales, bro.LAYOUT_GEMM)
                else:
                    bro.rotate_quantize_mxfp4(s["x"], block, acodes, ascales, bro.LAYOUT_GEMM)
            ev[1].record()
            for r in range(ring):
                s, acodes, ascales, gws = layers.views(i, r)
                bro.gemm_mxfp4(acodes, ascales, s["wcodes"], s["wscales"], M, N, K, s["y"], workspace=gws)
            ev[2].record()
            if it >= 2:
                rq_ev[i].append((ev[0], ev[1]))
                gemm_ev[i].append((ev[1], ev[2]))
    torch.cuda.synchronize()
    rq_t = [statistics.mean(a.elapsed_time(b) for a, b in lst) / ring for lst in rq_ev]
    gemm_t = [statistics.mean(a.elapsed_time(b) for a, b in lst) / ring for lst in gemm_ev]
    return rq_t, gemm_t


def operand_data_effect(layers, i, groups=6, sampler=None):
    """The same GEMM launch timed on the real quantised operands and on operands whose codes are all
    zero (scales, shapes, kernel and launch unchanged).  The instruction stream is identical; what
    differs is how much the tensor pipe's inputs toggle, and with that the power the chip draws and the
    SM clock its power management allows.  A diagnostic beside the roofline record, not a throughput."""
    import torch
    bro, ring = layers.bro, layers.ring
    M, K, N = layers.shapes[i]
    real, zero = [], []
    for r in range(ring):
        s, acodes, ascales, gws = layers.views(i, r)
        bro.rotate_quantize_mxfp4(s["x"], layers.block, acodes, ascales, bro.LAYOUT_GEMM)
        real.append((acodes, ascales, s["wcodes"], s["wscales"], s["y"], gws))
    za, zw = torch.zeros_like(real[0][0]), torch.zeros_like(real[0][2])
    for (_, ascales, _, wscales, y, gws) in real:
        zero.append((za, ascales, zw, wscales, y, gws))          # (the output still sweeps L2 between launches)

    def run(sets):
        # the chip's power management reacts over ~100 ms: settle on this operand data first
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for (ac, asc, wc, wsc, y, gws) in sets:
            bro.gemm_mxfp4(ac, asc, wc, wsc, M, N, K, y, workspace=gws)
        e1.record()
        torch.cuda.synchronize()
        settle = int(min(2000, max(4, 0.3 / max(e0.elapsed_time(e1) * 1e-3 / len(sets), 1e-6))))
        t_begin = time.time()
        for n in range(settle):
            ac, asc, wc, wsc, y, gws = sets[n % len(sets)]
            bro.gemm_mxfp4(ac, asc, wc, wsc, M, N, K, y, workspace=gws)
        times = []
        for it in range(groups):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for (ac, asc, wc, wsc, y, gws) in sets:
                bro.gemm_mxfp4(ac, asc, wc, wsc, M, N, K, y, workspace=gws)
            e1.record()
            times.append((e0, e1))
        torch.cuda.synchronize()
        t_end = time.time()
        # what nvidia-smi saw during the run (its first 0.1 s, the transition, left out)
        seen = sampler.window(t_begin + 0.1, t_end) if sampler is not None and sampler.proc is not None else None
        return statistics.mean(a.elapsed_time(b) for a, b in times) / len(sets) * 1e3, seen

    (us_zero, seen_zero), (us_real, seen_real) = run(zero), run(real)
    return {"MKN": [M, K, N], "gemm_kernel": gemm_kernel_name(M, K, N), "us_real_operands": round(us_real, 2),
            "us_zero_codes": round(us_zero, 2), "ratio": round(us_real / us_zero, 4),
            "tflops_zero_codes": round(2.0 * M * K * N / us_zero / 1e6, 1),
            "nvidia_smi_real_operands": seen_real, "nvidia_smi_zero_codes": seen_zero,
            "timing": "each after 0.3 s of back-to-back launches on the same operands",
            "note": "same kernel, launch and instruction stream; all-zero codes draw less power and keep the SM clock "
                    "up, so the ratio is what the chip's power management adds to a sustained run on real operands"}


def gemm_kernel_name(M, K, N, sm_count=148):
    """Which GEMM kernel the library picks for this problem (the rule of bro.cu, restated for the record's
    label; the ncu launch list under profiles/ shows the kernels that actually ran)."""
    pair = K >= 4096 and (-(-M // 256)) * (-(-N // 256)) >= 2 * (sm_count // 2)
    return "gemm_mxfp4_pair_kernel" if pair else "gemm_mxfp4_kernel"


def gemm_bytes(M, K, N):
    """Algorithmic bytes of one GEMM launch: packed codes and scales of both operands, bf16 output."""
    return (M + N) * K * (0.5 + 1 / 32) + 2 * M * N


def kernel_records(shapes, rq_t, gemm_t, peaks, ring, groups):
    """The roofline records of one workload from its per-shape kernel times.  The GEMM record covers
    the tensor-bound shapes (M >= 1024; all shapes if there is none); shapes with M <= 128 stream the
    packed weights once and are reported against the HBM copy bandwidth."""
    fp4_peak = peaks["bf16_tflops"] * FP4_OVER_BF16
    fp4_sustained = peaks["bf16_tflops_sustained"] * FP4_OVER_BF16
    big = [i for i, (M, K, N) in enumerate(shapes) if M >= 1024] or list(range(len(shapes)))
    small = [i for i, (M, K, N) in enumerate(shapes) if M <= 128 and i not in big]
    flops = sum(2.0 * shapes[i][0] * shapes[i][1] * shapes[i][2] for i in big)
    t = sum(gemm_t[i] for i in big) * 1e-3
    tflops = flops / t / 1e12
    per_shape = []
    for i, (M, K, N) in enumerate(shapes):
        tf = 2.0 * M * K * N / (gemm_t[i] * 1e-3) / 1e12
        gb = gemm_bytes(M, K, N) / (gemm_t[i] * 1e-3) / 1e9
        per_shape.append({"MKN": [M, K, N], "gemm_kernel": gemm_kernel_name(M, K, N),
                          "gemm_us": round(gemm_t[i] * 1e3, 2), "rq_us": round(rq_t[i] * 1e3, 2),
                          "gemm_tflops": round(tf, 1), "gemm_frac_of_4x_bf16_burst": round(tf / fp4_peak, 4),
                          "gemm_gbs": round(gb, 1), "gemm_frac_of_hbm_copy": round(gb / peaks["hbm_gbs"], 4)})
    roofline = {"bound": "tensor", "kernel": "/".join(sorted({gemm_kernel_name(*shapes[i]) for i in big})),
                "achieved": tflops, "peak": fp4_peak,
                "unit": "TFLOP/s", "frac": tflops / fp4_peak,
                "peak_source": f"{FP4_OVER_BF16:.0f} x {peaks['source']} bf16 burst ({peaks['bf16_tflops']} TFLOP/s)",
                "frac_of_sustained": tflops / fp4_sustained,
                "frac_of_nominal_fp4": tflops / NOMINAL_FP4_TFLOPS, "nominal_fp4_tflops": NOMINAL_FP4_TFLOPS,
                "shapes": [list(shapes[i]) for i in big],
                "algorithmic_bytes": sum(gemm_bytes(*shapes[i]) for i in big),
                "timing": f"CUDA events around groups of {ring} back-to-back launches, {groups} groups per shape",
                "per_shape_us": [round(gemm_t[i] * 1e3, 2) for i in big]}
    decode = None
    if small:
        b = sum(gemm_bytes(*shapes[i]) for i in small)
        ts = sum(gemm_t[i] for i in small) * 1e-3
        decode = {"bound": "hbm", "kernel": "gemm_mxfp4_kernel", "achieved": b / ts / 1e9, "peak": peaks["hbm_gbs"],
                  "unit": "GB/s", "frac": b / ts / 1e9 / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                  "frac_of_nominal_hbm": b / ts / 1e9 / NOMINAL_HBM_GBS,
                  "shapes": [list(shapes[i]) for i in small], "algorithmic_bytes": b,
                  "per_shape_us": [round(gemm_t[i] * 1e3, 2) for i in small]}
    rq_bytes = sum(M * K * 2.53125 for (M, K, N) in shapes)
    rq_gbs = rq_bytes / (sum(rq_t) * 1e-3) / 1e9
    rq = {"bound": "hbm", "kernel": "rotate_quantize_direct_kernel", "achieved": rq_gbs, "peak": peaks["hbm_gbs"],
          "unit": "GB/s", "frac": rq_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
          "frac_of_nominal_hbm": rq_gbs / NOMINAL_HBM_GBS,
          "per_shape_us": [round(t * 1e3, 2) for t in rq_t]}
    return roofline, decode, rq, per_shape


def block_sweep(bro, synth, peaks, blocks, groups):
    """cfg4: rotate+quantize of the [16384, 4096] tensor for each rotation size.  Per-size times come
    from CUDA events around groups of back-to-back launches that cycle through a ring of three inputs
    (3 x 134 MB > L2), so every launch reads from HBM.  2.53125 algorithmic bytes per element."""
    import torch
    cfg = synth.CONFIGS["cfg4"]
    M, K, _ = cfg["shapes"][0]
    x0 = synth.activations(M, K, seed=cfg["seed"], recipe=cfg["recipe"]).cuda()
    ring = 3
    xs = [x0.roll(7 * r, 0).contiguous() for r in range(ring)]
    codes = [bro.alloc_codes(M, K) for _ in range(ring)]
    scales = [bro.alloc_scales(M, K, bro.LAYOUT_GEMM) for _ in range(ring)]
    for _ in range(3):
        for b in blocks:
            bro.rotate_quantize_mxfp4(xs[0], b, codes[0], scales[0], bro.LAYOUT_GEMM)
    torch.cuda.synchronize()
    group = 2 * ring
    evs = {b: [] for b in blocks}
    torch.cuda._sleep(int(2e7))
    for gi in range(groups):
        for b in blocks:
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(group):
                bro.rotate_quantize_mxfp4(xs[i % ring], b, codes[i % ring], scales[i % ring], bro.LAYOUT_GEMM)
            c.record()
            evs[b].append((a, c))
    torch.cuda.synchronize()
    bytes_per_launch = M * K * 2.53125
    per_block = {}
    for b in blocks:
        ms = statistics.mean(a.elapsed_time(c) / group for a, c in evs[b])
        gbs = bytes_per_launch / (ms * 1e-3) / 1e9
        per_block[str(b if b else K)] = {"us": round(ms * 1e3, 2), "gbs": round(gbs, 1),
                                         "frac_of_measured_copy": round(gbs / peaks["hbm_gbs"], 4),
                                         "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    # The rotation fused into its producer (Sec. 4.3: the online rotation sits before down_proj, whose
    # input is silu(gate) * up): one launch that reads gate and up and writes codes and scales (4.53125 B
    # per element) against the two-step path, producer kernel then rotate+quantize (8.53125 B per element).
    gates = [(x * 0.5).to(torch.bfloat16) for x in xs]
    ups = [torch.randn((M, K), dtype=torch.float32, device="cuda", generator=torch.Generator(device="cuda").manual_seed(r)).to(torch.bfloat16)
           for r in range(ring)]
    h = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")

    def fused(i):
        bro.swiglu_rotate_quantize_mxfp4(gates[i % ring], ups[i % ring], 32, codes[i % ring], scales[i % ring], bro.LAYOUT_GEMM)

    def two_step(i):
        bro.swiglu_bf16(gates[i % ring], ups[i % ring], h)
        bro.rotate_quantize_mxfp4(h, 32, codes[i % ring], scales[i % ring], bro.LAYOUT_GEMM)

    producer = {}
    for name, fn, nbytes in (("fused", fused, 4.53125), ("two_step", two_step, 8.53125)):
        for i in range(3):
            fn(i)
        ts = []
        for gi in range(groups):
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(group):
                fn(i)
            c.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(c) / group)
        ms = statistics.mean(ts)
        producer[name] = {"us": round(ms * 1e3, 2), "algorithmic_bytes": M * K * nbytes,
                          "gbs": round(M * K * nbytes / (ms * 1e-3) / 1e9, 1)}
    producer["speedup"] = round(producer["two_step"]["us"] / producer["fused"]["us"], 3)
    del gates, ups, h
    # Simulated quantisation (Sec. 3.1: how the paper evaluates the formats): rotate, quantise, dequantise
    # to fp32 in one launch — 2 B read and 4 B written per element (2 + 2 read for the per-row formats).
    deq = torch.empty((M, K), dtype=torch.float32, device="cuda")
    fws = torch.empty(bro.fake_quantize_workspace_bytes(M, "int4_row_asym"), dtype=torch.uint8, device="cuda")
    fake = {}
    for fmt in ("mxfp4", "bfp4", "mxint4", "bint4", "int4_row_sym", "int4_row_asym"):     # (the last two: two passes over x)
        for i in range(2):
            bro.rotate_fake_quantize(xs[i % ring], 32, deq, fmt, workspace=fws)
        ts = []
        for gi in range(max(2, groups // 2)):
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(ring):
                bro.rotate_fake_quantize(xs[i % ring], 32, deq, fmt, workspace=fws)
            c.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(c) / ring)
        ms = statistics.mean(ts)
        nbytes = 8.0 if fmt.startswith("int4_row") else 6.0      # (the per-row formats read x twice)
        fake[fmt] = {"us": round(ms * 1e3, 2), "gbs": round(M * K * nbytes / (ms * 1e-3) / 1e9, 1),
                     "frac_of_measured_copy": round(M * K * nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}
    del deq, fws
    return {"shape_MK": [M, K], "algorithmic_bytes": bytes_per_launch, "per_block": per_block,
            "swiglu_producer_block32": producer, "fake_quantize_block32": fake,
            "timing": f"CUDA events around groups of {group} back-to-back launches, {groups} groups per size"}, (xs, codes, scales)


def run_ours(args):
    import torch
    from paper_2511_04214_b200 import build
    build.build()
    from paper_2511_04214_b200 import binding as bro, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod
    dev = torch.device("cuda", local_rank)
    cfg, shapes, idx = select_shapes(args)
    block = args.block
    peaks = measured_peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    layers = Layers(bro, synth, cfg, shapes, idx, block, dev, randomised=args.randomised)
    ring = layers.ring
    flops_per_step = layers.flops_per_step()

    ms_local, steps = time_steps(layers, args.steps, args.warmup, not args.no_graph, barrier, sampler)
    ms_total = max_over_ranks(ms_local, dist, dev)
    status = bro.last_device_status()
    if status != 0:
        raise SystemExit(f"device status {bro.status_string(status)} after the timed region")
    value = aggregate_throughput(flops_per_step, steps, world, ms_total) / 1e12

    groups = max(3, min(steps // ring, 16))
    rq_t, gemm_t = time_kernels(layers, groups)
    roofline, decode, rq_rec, per_shape = kernel_records(shapes, rq_t, gemm_t, peaks, ring, groups)
    roofline["traffic"] = ncu_traffic(args.workload, [tuple(s) for s in roofline["shapes"]])
    if roofline["traffic"] is not None and "per_row_of" in NCU_TRAFFIC.get(args.workload, {}):
        roofline["traffic_note"] = ("ncu capture of the M = %d shape (%d bytes per launch), scaled by the rows processed"
                                    % (NCU_TRAFFIC[args.workload]["per_row_of"][0], NCU_TRAFFIC[args.workload]["bytes"]))

    # ---- end-to-end through the host-buffer entry point
    notes = {}

    def guarded(name, fn):
        """A secondary measurement that cannot run (pinned-memory or device-memory limits, a missing
        compiler for the oracle) must not cost the run its main line: on a single-GPU run the reason goes
        to `notes` and the key stays null.  (With several ranks an exception has to propagate: the other
        ranks would wait at the next barrier.)"""
        if world > 1:
            return fn()
        try:
            return fn()
        except (RuntimeError, MemoryError, OSError, ValueError, subprocess.CalledProcessError) as exc:
            notes[name] = repr(exc)[:300]
            torch.cuda.synchronize()
            return None

    if world == 1 and not args.randomised and not args.no_operand_effect:
        tensor_bound = [i for i, sh in enumerate(shapes) if list(sh) in roofline["shapes"]]
        mid = [i for i in tensor_bound if shapes[i][0] <= 8192] or tensor_bound
        pick = max(mid, key=lambda i: shapes[i][0] * shapes[i][1] * shapes[i][2])
        roofline["operand_data_effect"] = guarded("operand_data_effect",
                                                  lambda: operand_data_effect(layers, pick, sampler=sampler))

    def measure_e2e():
        host = []
        for i, (M, K, N) in enumerate(shapes):
            s = layers.sets[i][0]
            host.append({"xh": s["x"].cpu().pin_memory(),
                         "yh": torch.empty((M, N), dtype=torch.bfloat16).pin_memory(),
                         "xs": torch.empty((M, K), dtype=torch.bfloat16, device=dev)})

        # One stream per layer: the layers of a step are independent here, so the upload of one layer's
        # activations overlaps the compute and the download of another's (PCIe is full duplex).  Within a
        # layer everything — H2D, rotate+quantize, GEMM, D2H — is ordered on its stream, step after step
        # (the staging buffers are reused), and the layer streams are joined only at the ends of the
        # timed region, so the downloads of one step overlap the uploads of the next.
        main = torch.cuda.current_stream()
        lay = [torch.cuda.Stream(device=dev) for _ in shapes]

        def e2e_steps(n):
            start = torch.cuda.Event()
            start.record(main)
            for st in lay:
                st.wait_event(start)
            for _ in range(n):
                for i, (M, K, N) in enumerate(shapes):
                    s, h = layers.sets[i][0], host[i]
                    bro.linear_host(h["xh"], block, s["wcodes"], s["wscales"], N, h["yh"], h["xs"], s["y"], s["ws"],
                                    stream=lay[i])
            for st in lay:
                done = torch.cuda.Event()
                done.record(st)
                main.wait_event(done)
        h2d = sum(M * K * 2 for (M, K, N) in shapes)
        d2h = sum(M * N * 2 for (M, K, N) in shapes)
        e2e_steps(3 if h2d + d2h < (1 << 30) else 1)
        barrier()
        # about a second of PCIe traffic at 25 GB/s, at least 3 steps
        n_e2e = int(max(3, min(steps, 30, 25e9 / max(h2d + d2h, 1))))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        e2e_steps(n_e2e)
        b.record()
        barrier()
        ms = max_over_ranks(a.elapsed_time(b), dist, dev)
        return {"value": aggregate_throughput(flops_per_step, n_e2e, world, ms) / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": ms / n_e2e,
                "streams": len(shapes)}

    e2e = None
    if not args.no_e2e and not args.randomised:     # (the host-buffer entry point has no randomised form)
        e2e = guarded("e2e", measure_e2e)
    clocks = sampler.stop() if rank == 0 else None
    status = bro.last_device_status()
    if status != 0:
        raise SystemExit(f"device status {bro.status_string(status)} after the end-to-end region")

    # ---- the other workloads, per kernel, in the same process (rank 0 of a single-GPU run)
    def measure_per_config():
        per_config = {}
        for name in ("cfg2", "cfg3"):
            if name == args.workload:
                continue
            c2 = synth.CONFIGS[name]
            sh = [s for s in c2["shapes"] if s[2] > 0]
            lay2 = Layers(bro, synth, c2, sh, list(range(len(sh))), 32, dev)
            ms2, st2 = time_steps(lay2, 4 * lay2.ring, 3, True, barrier)
            g2 = 8
            rq2, gm2 = time_kernels(lay2, g2)
            roof2, dec2, rqrec2, ps2 = kernel_records(sh, rq2, gm2, peaks, lay2.ring, g2)
            per_config[name] = {"value": lay2.flops_per_step() * st2 / (ms2 * 1e-3) / 1e12, "unit": UNIT,
                                "ms_per_step": ms2 / st2, "steps": st2, "block": 32,
                                "gemm": {k: roof2[k] for k in ("achieved", "peak", "frac", "frac_of_nominal_fp4", "unit")},
                                "rotate_quantize": {k: rqrec2[k] for k in ("achieved", "peak", "frac", "frac_of_nominal_hbm", "unit")},
                                "per_shape": ps2}
            del lay2
            torch.cuda.empty_cache()
        sweep, keep = block_sweep(bro, synth, peaks, synth.CONFIGS["cfg4"]["blocks"], 8)
        per_config["cfg4"] = sweep
        del keep
        torch.cuda.empty_cache()
        return per_config

    per_config = None
    layers = None                      # (frees the device buffers of the main workload)
    if rank == 0 and world == 1 and not args.no_per_config and args.shape_index < 0:
        torch.cuda.empty_cache()
        per_config = guarded("per_config", measure_per_config)
        status = bro.last_device_status()
        if status != 0:
            raise SystemExit(f"device status {bro.status_string(status)} after the per-config pass")

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, single-GPU runs only)
    def measure_cpu_baseline():
        import oracle
        rows = 128
        prepared = oracle_prepare(shapes, cfg, rows, block, idx)
        t, f, passes = 0.0, 0.0, 0
        while t < 10.0 and passes < 200:          # about 10 s of CPU work
            dt, df = oracle_step(prepared, block)
            t, f, passes = t + dt, f + df, passes + 1
        return {"value": f / t / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                "sample": f"first {rows} rows of each of the {len(shapes)} shapes, {passes} passes, {t:.1f} s "
                          "(weights packed offline, untimed)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = guarded("cpu_baseline", measure_cpu_baseline)

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "mxfp4 (e2m1 x e8m0) operands, f32 accumulate, bf16 out", "data": "synthetic",
            "config": {"workload": args.workload, "shapes_MKN": shapes, "block": block,
                       "l2": f"ring of {ring} independent input/output sets ({layers_bytes(shapes) * ring / 1e6:.0f} MB) > 126 MB L2",
                       "launch": "direct" if args.no_graph else "cuda_graph", "parallelism": "replicas only",
                       "rotation": "randomised block Hadamard (diag(s) H)" if args.randomised else "block Hadamard"},
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": steps * len(shapes) * 2,
            "roofline": roofline,
            "decode": decode,
            "rotate_quantize": rq_rec,
            "per_shape": per_shape,
            "per_config": per_config,
            "cpu_baseline": cpu,
        }
        if notes:
            out["notes"] = notes
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def layers_bytes(shapes):
    return sum(M * K * 2 + N * K // 2 + M * N * 2 for (M, K, N) in shapes)


def run_rotate_quantize_only(args):
    """Workload cfg4: the block-size sweep on a rotate+quantize-only activation tensor
    [16384, 4096]; one step = one launch per rotation size.  Reports HBM GB/s per size
    (2.53125 algorithmic bytes per element: 2 read, 1/2 code, 1/32 scale)."""
    import torch
    from paper_2511_04214_b200 import build
    build.build()
    from paper_2511_04214_b200 import binding as bro, synth
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    cfg = synth.CONFIGS["cfg4"]
    M, K, _ = cfg["shapes"][0]
    blocks = [args.block] if args.only_block else cfg["blocks"]
    peaks = measured_peaks()
    x0 = synth.activations(M, K, seed=cfg["seed"], recipe=cfg["recipe"]).cuda()
    ring = 3                                                   # 3 x 128 MiB inputs > 126 MB L2
    xs = [x0.roll(7 * r, 0).contiguous() for r in range(ring)]
    codes = [bro.alloc_codes(M, K) for _ in range(ring)]
    scales = [bro.alloc_scales(M, K, bro.LAYOUT_GEMM) for _ in range(ring)]
    sampler = ClockSampler(0)
    sampler.start()
    per_block = {}
    steps = args.steps
    for _ in range(max(args.warmup, 3)):
        for b in blocks:
            bro.rotate_quantize_mxfp4(xs[0], b, codes[0], scales[0], bro.LAYOUT_GEMM, flags=args.flags)
    torch.cuda.synchronize()
    sampler.mark("t0")
    t_all0 = torch.cuda.Event(enable_timing=True); t_all1 = torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(int(2e7))
    t_all0.record()
    # One step = one launch per rotation size.  Per-size times come from CUDA events around groups
    # of `group` back-to-back launches of that size (cycling through the ring of inputs, so every
    # launch reads its 134 MB from HBM); an event pair around every single launch would add its own
    # latency to a 30 us kernel.
    group = 2 * ring
    n_groups = max(1, steps // group)
    steps = n_groups * group
    evs = {b: [] for b in blocks}
    for gi in range(n_groups):
        for b in blocks:
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(group):
                bro.rotate_quantize_mxfp4(xs[i % ring], b, codes[i % ring], scales[i % ring], bro.LAYOUT_GEMM, flags=args.flags)
            c.record()
            evs[b].append((a, c))
    t_all1.record()
    torch.cuda.synchronize()
    sampler.mark("t1")
    assert bro.last_device_status() == 0
    bytes_per_launch = M * K * 2.53125
    for b in blocks:
        ts = [a.elapsed_time(c) / group for a, c in evs[b]]
        per_block[str(b if b else K)] = {"us": statistics.mean(ts) * 1e3, "gbs": bytes_per_launch / (statistics.mean(ts) * 1e-3) / 1e9,
                                         "frac_of_measured_copy": bytes_per_launch / (statistics.mean(ts) * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    # The oracle's per-group quantisation error per rotation size (Sec. 4.1 / 4.2, Fig. 6-7) and its scale
    # statistics (App. A.3), on the first 512 rows: mean error over all MX groups and split into regular
    # and outlier groups (an outlier group holds one of the top 0.1 % |x| entries of the sample), and the
    # fraction of regular groups whose E8M0 scale byte rises under each rotation.
    oracle_mse = None
    if not args.no_cpu_baseline:
        import oracle
        rows = 512
        xs_cpu = synth.activations(M, K, seed=cfg["seed"], recipe=cfg["recipe"])[:rows]
        bits = synth.bf16_bits(xs_cpu)
        omask, othr = oracle.outlier_groups(bits, 1000)
        outlier = omask.astype(bool)
        obefore = oracle.group_scale_bytes(bits, 1)
        oracle_mse = {"rows": rows, "outlier_group_fraction": float(outlier.mean()), "threshold_bf16_bits": othr}
        for b in blocks:
            y = oracle.rotate(bits, b)
            c, sc = oracle.quantize(y)
            mse = oracle.group_mse(y, c, sc)
            infl = oracle.scale_inflation(obefore, sc, omask)
            oracle_mse[str(b if b else K)] = {"all": float(mse.mean()), "regular": float(mse[~outlier].mean()),
                                              "outlier": float(mse[outlier].mean()),
                                              "regular_scale_up_fraction": float(infl[0, 2]) / float(infl[0].sum()),
                                              "outlier_scale_down_fraction": float(infl[1, 0]) / max(float(infl[1].sum()), 1.0)}
    # The same statistics over the WHOLE tensor on the GPU, all through library calls: outlier groups
    # (bro_outlier_groups), per-group error (bro_group_quant_error: 2 bytes read per element, 4 bytes
    # written per group), scale bytes before / after each rotation and the inflation counts.
    gpu_mse = {}
    mse_buf = torch.empty((M, K // 32), dtype=torch.float32, device="cuda")
    gmask = torch.empty((M, K // 32), dtype=torch.uint8, device="cuda")
    ginfo = torch.zeros(4, dtype=torch.int32, device="cuda")
    gws = torch.empty(bro.outlier_workspace_bytes(), dtype=torch.uint8, device="cuda")
    bro.outlier_groups(xs[0], gmask, ginfo, gws, top_ppm=1000)
    outlier_gpu = gmask.bool()
    sb_before = torch.empty((M, K // 32), dtype=torch.uint8, device="cuda")
    sb_after = torch.empty((M, K // 32), dtype=torch.uint8, device="cuda")
    counts = torch.empty((2, 3), dtype=torch.int64, device="cuda")
    hist = torch.empty((2, 256), dtype=torch.int64, device="cuda")
    bro.group_scale_bytes(xs[0], 1, sb_before)
    for b in blocks:
        for i in range(3):
            bro.group_quant_error(xs[i % ring], b, mse_buf)
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(2 * ring):
            bro.group_quant_error(xs[i % ring], b, mse_buf)
        c.record()
        bro.group_quant_error(xs[0], b, mse_buf)
        bro.group_scale_bytes(xs[0], b, sb_after)
        bro.scale_inflation(sb_before, sb_after, gmask, counts)
        bro.scale_histogram(sb_after, gmask, hist)
        torch.cuda.synchronize()
        cn = counts.cpu().numpy().astype(float)
        hn = hist.cpu().numpy().astype(float)
        us = a.elapsed_time(c) * 1e3 / (2 * ring)
        gpu_mse[str(b if b else K)] = {"us": us, "gbs": M * K * 2.125 / us / 1e3, "all": float(mse_buf.mean()),
                                       "regular": float(mse_buf[~outlier_gpu].mean()),
                                       "outlier": float(mse_buf[outlier_gpu].mean()),
                                       "regular_scale_up_fraction": cn[0, 2] / cn[0].sum(),
                                       "outlier_scale_down_fraction": cn[1, 0] / max(cn[1].sum(), 1.0),
                                       "mean_scale_byte_regular": float((hn[0] * range(256)).sum() / hn[0].sum()),
                                       "mean_scale_byte_outlier": float((hn[1] * range(256)).sum() / max(hn[1].sum(), 1.0))}
    gpu_mse["outlier_group_fraction"] = float(outlier_gpu.float().mean())
    gpu_mse["threshold_bf16_bits"] = int(ginfo[0])
    # Format study (Sec. 3.2 / Fig. 2-3) on the same tensor: mean group error per 4-bit format for the
    # block-32 and the full-dimension rotation.
    format_study = {}
    for fmt in ("mxfp4", "bfp4", "mxint4", "bint4"):
        format_study[fmt] = {}
        for b in (32, 0):
            bro.group_quant_error(xs[0], b, mse_buf, fmt=fmt)
            format_study[fmt][str(b if b else K)] = {"all": float(mse_buf.mean()), "regular": float(mse_buf[~outlier_gpu].mean()),
                                                     "outlier": float(mse_buf[outlier_gpu].mean())}
    # Rotation-dimension sweep (Sec. 5.2 / Fig. 7, in error terms): no rotation, the dimensions below the
    # MX group, the group itself, and above it, MXFP4, same tensor.
    dimension_sweep = {}
    if not args.only_block:
        for b in (1, 2, 4, 8, 16, 32, 64, 128, 0):
            bro.group_quant_error(xs[0], b, mse_buf)
            dimension_sweep[str(b if b else K)] = {"all": float(mse_buf.mean()), "regular": float(mse_buf[~outlier_gpu].mean()),
                                                   "outlier": float(mse_buf[outlier_gpu].mean()),
                                                   "median": float(mse_buf.flatten()[::7].median())}
    assert bro.last_device_status() == 0
    ms_total = t_all0.elapsed_time(t_all1)
    value = bytes_per_launch * len(blocks) * steps / (ms_total * 1e-3) / 1e9
    first = per_block[str(blocks[0] if blocks[0] else K)]
    out = {"metric": "rotate+quantize HBM GB/s", "value": value, "unit": "GB/s", "n_gpus": 1, "steps": steps,
           "warmup": max(args.warmup, 3), "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16 in, f32 rotation, mxfp4 out", "data": "synthetic",
           "config": {"workload": "cfg4", "shape_MK": [M, K], "blocks": [b if b else K for b in blocks],
                      "l2": f"ring of {ring} inputs (3 x 134 MB) > 126 MB L2", "layout": "gemm", "flags": args.flags},
           "clocks": sampler.stop(), "gpu_launches": steps * len(blocks), "per_block": per_block,
           "oracle_group_mse": oracle_mse, "gpu_group_mse": gpu_mse, "gpu_format_study": format_study,
           "gpu_rotation_dimension_sweep": dimension_sweep,
           "roofline": {"bound": "hbm", "kernel": "rotate_quantize_kernel", "achieved": first["gbs"], "peak": peaks["hbm_gbs"],
                        "unit": "GB/s", "frac": first["gbs"] / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                        "traffic": ncu_traffic("cfg4", [(M, K, blocks[0] if blocks[0] else K)]),
                        "algorithmic_bytes": bytes_per_launch,
                        "timing": f"CUDA events around groups of {group} back-to-back launches, {n_groups} groups per size"}}
    print(json.dumps(out), flush=True)


def launch_ranks(n, argv):
    """Start `n` ranks of this script on one node with torch.distributed.run and relay their output
    (the path does not shard: the ranks are independent replicas that only meet for the timing
    barrier and the max-over-ranks reduction).  Returns the launcher's exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.run(cmd).returncode


def run_rank_check(args):
    """Host logic of a multi-rank run, without a GPU: every rank reports a rank-dependent time, the
    job's time is the slowest rank's, rank 0 prints one line.  (Used by the CPU tests to cover the
    launcher and the rank plumbing with the gloo backend.)"""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks(10.0 + 5.0 * rank, dist if world > 1 else None, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"rank_check": True, "n_gpus": world, "ms": ms,
                          "value": aggregate_throughput(1000.0, 4, world, ms)}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--block", type=int, default=32)
    ap.add_argument("--shape-index", type=int, default=-1,
                    help="run only this shape of the workload (for profiling captures); -1 = all")
    ap.add_argument("--ref-rows", type=int, default=0,
                    help="rows per shape per step for --impl reference (0 = sized to finish in ~2 min)")
    ap.add_argument("--only-block", action="store_true", help="cfg4: run only --block instead of the sweep")
    ap.add_argument("--randomised", action="store_true",
                    help="use the randomised block rotation diag(s) H / sqrt(block) (the *_rs entry points)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-operand-effect", action="store_true",
                    help="skip the zero-codes / real-operands comparison of one GEMM launch")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the per-kernel figures of the other workloads (cfg2, cfg3, cfg4)")
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0,
                    help="kernel-selection flags (BRO_FLAG_* of include/bro.h) passed to the *_ex entry points")
    ap.add_argument("--rank-check", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        # no launcher around us: start the N replica ranks ourselves
        raise SystemExit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.rank_check:
        run_rank_check(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.workload == "cfg4":
        run_rotate_quantize_only(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
