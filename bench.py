#!/usr/bin/env python
"""Benchmark of the MDBF linear forward (libmdbf) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl mdbf|reference]

Prints ONE JSON line.  Default workload `decode_qproj`: the 7B-class q_proj
shape (d_out = d_in = 4096, l = 16, T = 1, bf16 activations with outlier
channels, fp16 envelopes) at k = 1664 (~1.0 bpw) and k = 2560 (~1.5 bpw).
A step is one forward through every layer of a rotation of distinct layers
whose packed weights exceed L2 several times over, launched back to back on
one stream, so that every step streams its weights from HBM.

Metric: GB/s of ALGORITHMIC bytes (packed signs + envelopes + x + y, each
once) for the decode workloads; TFLOP/s of the expanded sign contraction
2*l*T*k*(d_in + d_out) for the prefill workloads.

Multi-GPU: the path does not shard (one layer = one GPU); `--gpus N` under
torchrun runs N independent replicas ("replicas only", weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None until a capture exists for that workload).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {
    ("decode_qproj", "tmem_t1_kernel"): 1082112,                   # k = 1664 layer, stage B (stage A: 1080320)
    ("block70b_T1", "t1_stage_kernel"): 46402560,                  # gate/up stage A in one launch (45.3 MB algorithmic); down stage B: 23289856
    ("decode_mlp_T1", "tmem_t1_kernel"): 5998592,                  # up / gate, either stage (down: 2342400)
    ("decode_mlp_T16", "mat_small_kernel"): 6340000,               # up stage B (stage A: 6.11 MB, down stage A: 2.47 MB)
    ("prefill_4096_l16_bpw10", "mat_stage_kernel"): 17858048,      # stage B: x read once + signs + images; nothing reaches DRAM on the way out
    ("prefill_4096_l16_bpw10", "gemm_stage_kernel"): 370142976,    # stage B: 269.4 MB read + 100.7 MB written
    ("msvid_28672x6016_l16", "envelope_product_tc_kernel"): 708300000,   # Z once per pass (689.9 MB) + operand images and partial sums,
                                                                           # scaled by rows x cols from the 8192 x 8192 capture
    ("msvid_8192x8192_l16", "envelope_product_tc_kernel"): 275523328,      # 269.6 MB read + 5.9 MB written for 268.4 MB of Z
    ("admm_8192x8192_r3712_l16", "gemm3x_kernel"): 1156590808,            # its largest launch, W V: 1.038 GB read (images 0.78 GB; V's are re-read
                                                                           # by every row tile, four fifths of that from L2) + 118.6 MB written
    ("block70b_T2048", "mat_stage_kernel"): 197116928,             # its largest launch, down stage B (185.9 MB read: 117 MB of x, partly twice,
                                                                   # + signs; 11.3 MB written); gate / up stage A: 123.3 MB
}


def dominant_kernel(workload, T, kernels_used, M):
    """Name of the kernel that takes most of the step's device time (the one the roofline line is about)."""
    if T == 1:
        # the integer kernel streams the large stages (gate/up stage A and down stage B of the 70B-class block)
        return "t1_stage_kernel" if workload.startswith("block70b") or M.KERNEL_I8 in kernels_used else "tmem_t1_kernel"
    if M.KERNEL_MAT in kernels_used:
        return "mat_stage_kernel" if T > 64 else "mat_small_kernel"
    return "gemm_stage_kernel"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------- accounting
def algorithmic_bytes(spec, T):
    env_b = 4 if spec.env_dtype == "f32" else 2
    act_b = 4 if spec.act_dtype == "f32" else 2
    signs = spec.k * (spec.d_in + spec.d_out) // 8
    env = env_b * spec.l * (spec.d_in + spec.d_out + 2 * spec.k)
    act = act_b * T * (spec.d_in + spec.d_out)
    return signs + env + act


def expanded_flops(spec, T):
    return 2.0 * spec.l * T * spec.k * (spec.d_in + spec.d_out)


def rated_materialised(spec, T, forced="auto"):
    """Whether a tensor-bound workload is rated in FLOPs of the materialised order: mirrors the library's
    dispatch (every T >= 2 runs the materialised-order kernel; the bench shapes all qualify for it)."""
    if forced != "auto":
        return forced == "mat"
    return T >= 2


def materialised_flops(spec, T):
    """Tensor FLOPs when the factor tiles are rebuilt on the fly: rank-l envelope product + one GEMM of width T."""
    return (2.0 * T + 2.0 * spec.l) * spec.k * (spec.d_in + spec.d_out)


# ---------------------------------------------------------------- workloads
def workload_specs(name):
    """-> (list of (LayerSpec, copies), T, metric kind, description)."""
    from paper_2512_24545_b200 import inputs
    if name == "decode_qproj":
        return [(inputs.qproj(1664), 64), (inputs.qproj(2560), 64)], 1, "hbm", \
            "q_proj 4096x4096 l=16 T=1, k=1664 and k=2560, 64 distinct layers each"
    if name.startswith("decode_mlp"):
        T = int(name.split("_T")[1]) if "_T" in name else 1
        return [(inputs.mlp("up"), 16), (inputs.mlp("down"), 16)], T, "hbm", \
            f"MLP up 11008x4096 and down 4096x11008, k=3968 l=16 T={T}, 16 distinct layers each"
    if name.startswith("block70b"):
        T = int(name.split("_T")[1]) if "_T" in name else 1
        return [(s, 4 if T <= 16 else 1) for s in inputs.block70b()], T, "hbm" if T <= 16 else "tensor", \
            f"70B-class decoder block, 7 linears, l=16 ~1.0 bpw, T={T}"
    if name.startswith("sum_qproj"):
        # sum_qproj_l<l>P<P>: P terms of envelope rank l on the 4096^2 shape, together ~1.0 bpw; the
        # residual-compensation format ((l, P) = (1, 2) is the two-DBF-term case); T = 1
        import re as _re
        m = _re.match(r"sum_qproj_l(\d+)P(\d+)", name)
        l, P = (int(m.group(1)), int(m.group(2))) if m else (1, 2)
        bits = (1.0 / P) * 4096 * 4096                    # budget per term; k = largest multiple of 128 that meets it
        k = int((bits - 16 * l * 8192) / (8192 + 32 * l)) // 128 * 128
        base = inputs.qproj(1664)
        terms = [(inputs.scaled(base, name=f"sum_qproj_l{l}_term{p}", k=k, l=l, seed=6 + 37 * p,
                                env_std=0.02 * 0.6 ** p), 64) for p in range(P)]
        return terms, 1, "hbm", f"sum of {P} terms 4096x4096 l={l} k={k} (~1.0 bpw together) T=1, 64 distinct sums"
    if name.startswith("prefill"):
        # prefill_<d_out>_l<l>_<bpw10|bpw15>
        parts = name.split("_")
        d_out = int(parts[1]) if len(parts) > 1 else 4096
        l = int(parts[2][1:]) if len(parts) > 2 else 16
        bpw = 1.5 if (len(parts) > 3 and parts[3] == "bpw15") else 1.0
        return [(inputs.prefill(d_out, l, bpw), 1)], 2048, "tensor", \
            f"prefill {d_out}x4096 l={l} ~{bpw} bpw T=2048"
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """SM clock and throttle reasons sampled during the timed region: NVML polled every few milliseconds (a timed
    region of some tens of milliseconds still gets a handful of samples), nvidia-smi as the fallback.  Read-only."""

    def __init__(self, index):
        self.index = index
        self.samples = []          # (sm_mhz, max_mhz, reasons bitmask)
        self.stop_flag = False
        self.thread = None
        self.nvml = None
        self.proc = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll_nvml(self):
        n = self.nvml
        while not self.stop_flag:
            try:
                sm = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                try:
                    reasons = int(n.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    reasons = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                self.samples.append((sm, self.max_mhz, reasons))
            except Exception:
                break
            time.sleep(0.002)

    def _read_smi(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
        for line in self.proc.stdout:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm, mx = float(f[0]), float(f[1])
            except ValueError:
                continue
            mask = 0
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    mask |= bits[nm]
            self.samples.append((sm, mx, mask))

    def stop(self):
        self.stop_flag = True
        if self.nvml is None and self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            time.sleep(0.05)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=1.0)
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}
        sm = [x[0] for x in self.samples]
        mx = [x[1] for x in self.samples]
        reasons = set()
        for (_s, _m, mask) in self.samples:
            for bit, nm in names.items():
                if mask & bit:
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "source": "nvml" if self.nvml is not None else "nvidia-smi"}


def dist_setup(n_gpus):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return dist, rank, world, local
    return None, 0, 1, 0


# ------------------------------------------------------------------ mdbf arm
def measure(workload, kernel, steps, warmup, dist, world, local, no_graph=False, no_siblings=False, copies=0,
            want_e2e=True, fuse_block=False, min_timed_ms=0.0):
    """Time `steps` steps of one workload (after >= 3 untimed ones) and return the measured fields.  min_timed_ms > 0
    raises `steps` (the returned dict says to what) until the timed region lasts about that long, so that the
    clock record of a short workload holds more than a sample or two."""
    import torch
    from paper_2512_24545_b200 import inputs, mdbf as M, replicas
    peaks, peak_kind = load_peaks()
    groups, T, bound, desc = workload_specs(workload)
    stream = torch.cuda.Stream()
    st = stream.cuda_stream

    P_sum = len(groups) if workload.startswith("sum_") else 0     # > 0: every P_sum consecutive layers are one sum
    if P_sum:
        ncopies = copies if copies > 0 else groups[0][1]
        groups = [(inputs.scaled(sp, seed=sp.seed + 1000 * c), 1) for c in range(ncopies) for (sp, _n) in groups]
    layers = []          # (handle, spec, x_dev, y_dev, x_host, y_host)
    total_bytes = 0
    total_flops = 0.0
    total_mat_flops = 0.0
    weight_bytes = 0
    xs = {}
    if workload.startswith("block70b"):       # block by block: q, k, v, o, gate, up, down of copy 0, then copy 1, ...
        nc = copies if copies > 0 else groups[0][1]
        groups = [(inputs.scaled(sp, seed=sp.seed + 1000 * c) if c else sp, 1) for c in range(nc) for (sp, _n) in groups]
    for spec, default_copies in groups:
        for c in range(1 if (P_sum or workload.startswith("block70b")) else (copies if copies > 0 else default_copies)):
            sp = inputs.scaled(spec, seed=spec.seed + 1000 * (c + 1)) if c else spec
            lay = inputs.make_layer(sp)
            h = M.mdbf_pack(sp.d_out, sp.d_in, sp.k, sp.l, M.DTYPES[sp.env_dtype], T,
                            *[np.ascontiguousarray(lay[n]) for n in ("S_A", "S_B", "U_A", "V_A", "U_B", "V_B")])
            if T > 1 and kernel in ("prefill", "mat"):
                M.mdbf_set_kernel(h, {"prefill": M.KERNEL_PREFILL, "mat": M.KERNEL_MAT}[kernel])
            if T == 1 and kernel in ("tmem", "i8"):
                M.mdbf_set_kernel(h, {"tmem": M.KERNEL_TMEM, "i8": M.KERNEL_I8}[kernel])
            if sp.d_in not in xs:
                xh = torch.from_numpy(inputs.make_activations(sp, T)).to(torch.bfloat16).pin_memory()
                xs[sp.d_in] = (xh, xh.cuda())
            xh, xd = xs[sp.d_in]
            yd = torch.zeros((T, sp.d_out), dtype=torch.bfloat16, device="cuda")
            yh = torch.zeros((T, sp.d_out), dtype=torch.bfloat16).pin_memory()
            layers.append((h, sp, xd, yd, xh, yh))
            total_bytes += algorithmic_bytes(sp, T)
            total_flops += expanded_flops(sp, T)
            total_mat_flops += materialised_flops(sp, T)
            weight_bytes += algorithmic_bytes(sp, 0)
    torch.cuda.synchronize()

    flush = None
    if weight_bytes < 2 * 126e6:       # rotation too small to defeat L2: flush between steps
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")

    acc = torch.zeros((T, max(sp.d_out for (_h, sp, *_r) in layers)), dtype=torch.float32, device="cuda") if P_sum else None

    # the 70B-class block at one token: q/k/v share the hidden input and gate/up share the MLP input, so they
    # go through the sibling entry point (one pair of launches per group); o and down stand alone
    sib_groups = None
    if workload.startswith("block70b") and T == 1 and not no_siblings:
        sib_groups = []
        for b0 in range(0, len(layers), 7):
            blk = layers[b0:b0 + 7]
            if len(blk) == 7:
                sib_groups += [blk[0:3], blk[3:4], blk[4:6], blk[6:7]]
            else:
                sib_groups += [[l] for l in blk]

    def step():
        if fuse_block and workload.startswith("block70b") and T == 1:
            # the seven layers of a block as independent forwards (their inputs are seeded, not produced by one another):
            # one set of launches per block through the group entry point
            for b0 in range(0, len(layers), 7):
                blk = layers[b0:b0 + 7]
                M.mdbf_linear_forward_group([g[0] for g in blk], [g[2].data_ptr() for g in blk], [g[3].data_ptr() for g in blk],
                                            T, M.BF16, st)
            return
        if sib_groups is not None:
            for grp in sib_groups:
                if len(grp) == 1:
                    (h, sp, xd, yd, _, _) = grp[0]
                    M.mdbf_linear_forward(h, xd.data_ptr(), yd.data_ptr(), T, M.BF16, st)
                else:
                    M.mdbf_linear_forward_siblings([g[0] for g in grp], grp[0][2].data_ptr(), [g[3].data_ptr() for g in grp],
                                                   T, M.BF16, st)
            return
        if P_sum:
            for i in range(0, len(layers), P_sum):
                hs = [layers[i + p][0] for p in range(P_sum)]
                M.mdbf_linear_forward_sum(hs, layers[i][2].data_ptr(), layers[i][3].data_ptr(), acc.data_ptr(), T, M.BF16, st)
            return
        for (h, sp, xd, yd, _, _) in layers:
            M.mdbf_linear_forward(h, xd.data_ptr(), yd.data_ptr(), T, M.BF16, st)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    graph = None
    with torch.cuda.stream(stream):
        step()                       # first call sets kernel attributes (not capturable state)
        torch.cuda.synchronize()
        if not no_graph:
            # one CUDA graph per step: removes the host launch cost of the back-to-back forwards
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step()
            run_step = graph.replay
        else:
            run_step = step
        for _ in range(max(3, warmup)):
            run_step()
        barrier()
        if min_timed_ms > 0:
            w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if flush is not None:
                flush.fill_(1)
            w0.record(stream)
            run_step()
            w1.record(stream)
            torch.cuda.synchronize()
            steps = max(steps, min(2000, int(min_timed_ms / max(w0.elapsed_time(w1), 1e-3)) + 1))
        sampler = ClockSampler(local)
        sampler.start()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(steps)]
        for (e0, e1) in ev:
            if flush is not None:
                flush.fill_(1)
            e0.record(stream)
            run_step()
            e1.record(stream)
        barrier()
        clocks = sampler.stop()
        ms = sum(e0.elapsed_time(e1) for e0, e1 in ev)
    launches = (sum(M.mdbf_last_launch_count(h) for (h, *_rest) in layers) + (len(layers) // P_sum if (P_sum and T > 1) else 0)) * steps     # the cast pass of a sum runs only for T > 1
    kernels_used = sorted({M.mdbf_last_kernel(h) for (h, *_r) in layers})
    mat = M.KERNEL_MAT in kernels_used

    # end to end: host buffers through the C-ABI, copies inside the timed region
    e2e_steps = max(1, min(steps, 10))
    e2e_s = 0.0
    if want_e2e:
        for (h, *_r) in layers:
            M.mdbf_prepare_host_staging(h)
        for _ in range(2):
            for (h, sp, _, _, xh, yh) in layers:
                M.mdbf_linear_forward_host(h, xh.data_ptr(), yh.data_ptr(), T, M.BF16, st)
        barrier()
        # a step: every layer's pinned input copied in, its forward, its output copied out - enqueued through the
        # asynchronous host-buffer entry point - and one synchronisation, after which all outputs are in host memory
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            for (h, sp, _, _, xh, yh) in layers:
                M.mdbf_linear_forward_host_async(h, xh.data_ptr(), yh.data_ptr(), T, M.BF16, st)
            stream.synchronize()
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
    h2d = sum(T * sp.d_in * 2 for (_, sp, *_r) in layers)
    d2h = sum(T * sp.d_out * 2 for (_, sp, *_r) in layers)

    ms_max, e2e_ms_max = replicas.max_over_ranks([ms, e2e_s * 1e3], dist, device="cuda")
    sec = ms_max / 1e3
    if bound == "hbm":
        metric, unit = "decode_algorithmic_GBps", "GB/s"
        per_step = total_bytes / 1e9
        peak = peaks["hbm_gbs"]
    else:
        # the expanded-order kernel is rated in FLOPs of the expanded contraction (which it executes); the
        # materialised-order kernel executes l x fewer and is rated in those, never in expanded FLOPs
        assert mat == rated_materialised(groups[0][0], T, kernel), "bench.py's copy of the dispatch rule is stale"
        metric, unit = ("prefill_executed_TFLOPs" if mat else "prefill_expanded_TFLOPs"), "TFLOP/s"
        per_step = (total_mat_flops if mat else total_flops) / 1e12
        peak = peaks["bf16_tflops"] if sec < 1.0 else peaks["bf16_tflops_sustained"]
    value = replicas.aggregate_throughput(per_step * steps, world, sec)
    per_gpu = per_step * steps / sec
    e2e_value = replicas.aggregate_throughput(per_step * e2e_steps, world, e2e_ms_max / 1e3) if want_e2e else None

    dom = dominant_kernel(workload, T, kernels_used, M)
    out = {
        "metric": metric, "value": value, "unit": unit, "steps": steps, "warmup": max(3, warmup),
        "ms_per_step": ms_max / steps,
        "config": {"workload": workload, "description": desc, "layers": len(layers), "T": T,
                   "weights_MB": round(weight_bytes / 1e6, 1),
                   "l2_policy": ("rotation of distinct layers larger than L2" if flush is None
                                 else "256 MiB L2 flush between steps"),
                   "launch": "CUDA graph replay per step" if graph is not None else "stream launches",
                   "kernel": kernel, "grouping": ("seven independent forwards per set of launches" if fuse_block else "q/k/v and gate/up as siblings, o and down alone" if sib_groups is not None else "one forward per layer"),
                   "GFLOP_expanded_per_step": round(total_flops / 1e9, 1),
                   "GFLOP_materialised_per_step": round(total_mat_flops / 1e9, 1),
                   "replicas": world},
        "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h} if want_e2e else None,
        "gpu_launches": launches,
        "clocks": clocks,
        "roofline": {"bound": bound, "achieved": per_gpu, "peak": peak, "unit": unit,
                     "frac": per_gpu / peak, "peak_source": f"of {peak_kind}", "kernel": dom,
                     "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get((workload, dom))},
    }
    cpu_args = (groups[0][0], T, bound, bound != "hbm" and mat)
    for (h, *_r) in layers:
        M.mdbf_destroy(h)
    del layers, xs, flush
    torch.cuda.empty_cache()
    return out, cpu_args


# ------------------------------------------------------------ quantizer, first step (MSVID)
def measure_msvid(workload, steps, warmup, dist, world, local, want_e2e=True, min_timed_ms=0.0):
    """msvid_<rows>x<cols>_l<l>[_it<n>]: one step = one mdbf_msvid call on a resident rows x cols fp32 matrix (sign mask +
    rank-l envelope, n subspace iterations).  Algorithmic bytes: the 2 n + 1 product passes each read Z once (rows * cols * 4
    bytes; |Z| is never stored, and the sign mask comes out of the first pass), plus the mask and the factors written."""
    import re
    import torch
    from paper_2512_24545_b200 import inputs, mdbf as M, replicas
    m = re.match(r"msvid_(\d+)x(\d+)_l(\d+)(?:_it(\d+))?$", workload)
    if not m:
        raise SystemExit(f"unknown workload {workload}")
    rows, cols, l = int(m.group(1)), int(m.group(2)), int(m.group(3))
    n_iter = int(m.group(4)) if m.group(4) else 4
    peaks, peak_kind = load_peaks()
    stream = torch.cuda.Stream()
    st = stream.cuda_stream
    Zh = torch.from_numpy(inputs.make_factor_matrix(rows, cols, seed=8)).pin_memory()
    Qh = torch.from_numpy(inputs.make_start_block(cols, l, seed=8)).pin_memory()
    Zd, Qd = Zh.cuda(), Qh.cuda()
    nwords = (cols + 31) // 32
    Sd = torch.zeros((rows, nwords), dtype=torch.int32, device="cuda")
    Ud = torch.zeros((rows, l), dtype=torch.float32, device="cuda")
    Vd = torch.zeros((cols, l), dtype=torch.float32, device="cuda")
    sd = torch.zeros((l,), dtype=torch.float32, device="cuda")
    Sh, Uh, Vh = (torch.zeros_like(t, device="cpu").pin_memory() for t in (Sd, Ud, Vd))
    ws_bytes = M.mdbf_msvid_workspace_bytes(rows, cols, l)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    passes = 2 * n_iter + 1
    step_bytes = passes * rows * cols * 4 + rows * nwords * 4 + (rows + cols) * l * 4
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda") if rows * cols * 4 < 2 * 126e6 else None

    def step():
        M.mdbf_msvid(Zd.data_ptr(), rows, cols, l, n_iter, Qd.data_ptr(), Sd.data_ptr(), Ud.data_ptr(), Vd.data_ptr(), sd.data_ptr(),
                     ws.data_ptr(), ws_bytes, st)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(max(3, warmup)):
            step()
        barrier()
        if min_timed_ms > 0:
            w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            w0.record(stream); step(); w1.record(stream)
            torch.cuda.synchronize()
            steps = max(steps, min(2000, int(min_timed_ms / max(w0.elapsed_time(w1), 1e-3)) + 1))
        sampler = ClockSampler(local)
        sampler.start()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for (e0, e1) in ev:
            if flush is not None:
                flush.fill_(1)
            e0.record(stream)
            step()
            e1.record(stream)
        barrier()
        clocks = sampler.stop()
        ms = sum(e0.elapsed_time(e1) for e0, e1 in ev)
        e2e_steps = max(1, min(steps, 3))
        e2e_s = 0.0
        if want_e2e:
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                Zd.copy_(Zh, non_blocking=True)
                Qd.copy_(Qh, non_blocking=True)
                step()
                Sh.copy_(Sd, non_blocking=True); Uh.copy_(Ud, non_blocking=True); Vh.copy_(Vd, non_blocking=True)
                stream.synchronize()
            e2e_s = time.perf_counter() - t0
    ms_max, e2e_ms_max = replicas.max_over_ranks([ms, e2e_s * 1e3], dist, device="cuda")
    value = replicas.aggregate_throughput(step_bytes * steps / 1e9, world, ms_max / 1e3)
    per_gpu = step_bytes * steps / 1e9 / (ms_max / 1e3)
    peak = peaks["hbm_gbs"]
    # as msvid.cu issues them for these shapes: start block 1 + 2 x 2, per iteration 2 products + 2 x 2 (+ 1 where the narrow
    # transposed product takes the scalar kernel and its partial-sum pass), last block once more 2, final product and factors 5
    launches_per_call = 1 + 4 + n_iter * (6 + (1 if l <= 4 else 0)) + 2 + 5
    out = {
        "metric": "msvid_algorithmic_GBps", "value": value, "unit": "GB/s", "steps": steps, "warmup": max(3, warmup),
        "ms_per_step": ms_max / steps,
        "config": {"workload": workload, "description": f"MSVID_l of a {rows} x {cols} fp32 factor, l={l}, {n_iter} subspace iterations "
                                                        f"({passes} passes over Z)", "layers": 1, "T": 0, "weights_MB": round(rows * cols * 4 / 1e6, 1),
                   "l2_policy": "matrix larger than L2" if flush is None else "256 MiB L2 flush between steps",
                   "launch": "stream launches", "kernel": "msvid", "grouping": "one call per step", "replicas": world},
        "e2e": ({"value": replicas.aggregate_throughput(step_bytes * e2e_steps / 1e9, world, e2e_ms_max / 1e3), "unit": "GB/s",
                 "h2d_bytes_per_step": rows * cols * 4 + cols * l * 4, "d2h_bytes_per_step": rows * nwords * 4 + (rows + cols) * l * 4}
                if want_e2e else None),
        "gpu_launches": launches_per_call * steps,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": per_gpu, "peak": peak, "unit": "GB/s", "frac": per_gpu / peak,
                     "peak_source": f"of {peak_kind}", "kernel": "envelope_product_tc_kernel",
                     "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get((workload, "envelope_product_tc_kernel"))},
    }
    del Zd, Qd, Sd, Ud, Vd, ws, flush
    torch.cuda.empty_cache()
    return out, ("msvid", rows, cols, l, n_iter)


def cpu_baseline_msvid(rows, cols, l, n_iter):
    """The oracle's MSVID (sign mask + full SVD of |Z|, fp64) on a leading block of the workload's matrix, rated in the
    algorithmic bytes the GPU arm's call counts for the same elements (2 n + 1 passes)."""
    from oracle import mdbf_oracle as orc
    from paper_2512_24545_b200 import inputs
    Z = inputs.make_factor_matrix(min(rows, 2048), min(cols, 4096), seed=8)
    t0 = time.perf_counter()
    orc.msvid(Z, l)
    dt = time.perf_counter() - t0
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    return {"value": (2 * n_iter + 1) * Z.size * 4 / 1e9 / dt, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": f"fp64 sign mask + full SVD of a {Z.shape[0]} x {Z.shape[1]} block of the workload's matrix, one call, {dt:.1f} s"}


# ------------------------------------------------------------ quantizer, refinement (ADMM factor update)
def admm_shape(workload):
    import re
    m = re.match(r"admm_(\d+)x(\d+)_r(\d+)_l(\d+)(?:_in(\d+))?$", workload)
    if not m:
        raise SystemExit(f"unknown workload {workload}")
    return int(m.group(1)), int(m.group(2)), int(m.group(3)), int(m.group(4)), int(m.group(5)) if m.group(5) else 1


def admm_flops(N, Mc, R, n_inner):
    """Dense-algebra flops of the least-squares step as a plain implementation counts them: W V, V^T V (one triangle), the
    Cholesky factor, two triangular solves with N right-hand sides per inner iteration.  The MSVID step's flops (a few per
    cent) are not counted, nor is the extra work of the library's own arrangement (the three-term split executes three
    tensor-core products per product counted here; the inverse of the R x R system is formed once per call)."""
    return 2.0 * N * Mc * R + 1.0 * Mc * R * R + R ** 3 / 3.0 + n_inner * 2.0 * N * R * R


def measure_admm(workload, steps, warmup, dist, world, local, want_e2e=True):
    """admm_<N>x<M>_r<R>_l<l>[_in<n>]: one step = one mdbf_admm_factor_update call (n inner iterations, 4 subspace
    iterations in each MSVID step) on resident fp32 matrices W (N x M), V (M x R), U and Lambda (N x R)."""
    import torch
    from paper_2512_24545_b200 import inputs, mdbf as M, replicas
    N, Mc, R, l, n_inner = admm_shape(workload)
    n_iter = 4
    stream = torch.cuda.Stream()
    st = stream.cuda_stream
    host = [torch.from_numpy(inputs.make_factor_matrix(a, b, seed=60 + i, special_values=False)).pin_memory()
            for i, (a, b) in enumerate([(N, Mc), (Mc, R), (N, R)])]
    Wd, Vd, U0 = (h.cuda() for h in host)
    Ud, Ld = U0.clone(), torch.zeros_like(U0)
    Qd = torch.from_numpy(inputs.make_start_block(R, l, seed=8)).cuda()
    nwords = (R + 31) // 32
    Sd = torch.zeros((N, nwords), dtype=torch.int32, device="cuda")
    Uld = torch.zeros((N, l), dtype=torch.float32, device="cuda")
    Vld = torch.zeros((R, l), dtype=torch.float32, device="cuda")
    sd = torch.zeros((l,), dtype=torch.float32, device="cuda")
    Uh, Lh, Sh = (torch.zeros_like(t, device="cpu").pin_memory() for t in (Ud, Ld, Sd))
    ws_bytes = M.mdbf_admm_workspace_bytes(N, Mc, R, l)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    rho = float((host[1].double() ** 2).sum()) / R
    flops = admm_flops(N, Mc, R, n_inner)
    peaks, peak_kind = load_peaks()
    peak = peaks["bf16_tflops_sustained" if "bf16_tflops_sustained" in peaks else "bf16_tflops"]

    def step():
        M.mdbf_admm_factor_update(Wd.data_ptr(), N, Mc, False, Vd.data_ptr(), R, Ud.data_ptr(), Ld.data_ptr(), rho, l, n_inner, n_iter,
                                  Qd.data_ptr(), Sd.data_ptr(), Uld.data_ptr(), Vld.data_ptr(), sd.data_ptr(), None, ws.data_ptr(),
                                  ws_bytes, st)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(max(3, warmup)):
            step()
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for (e0, e1) in ev:
            e0.record(stream)
            step()
            e1.record(stream)
        barrier()
        clocks = sampler.stop()
        ms = sum(e0.elapsed_time(e1) for e0, e1 in ev)
        e2e_steps, e2e_s = max(1, min(steps, 3)), 0.0
        if want_e2e:
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                Wd.copy_(host[0], non_blocking=True); Vd.copy_(host[1], non_blocking=True); Ud.copy_(host[2], non_blocking=True)
                Ld.zero_()
                step()
                Uh.copy_(Ud, non_blocking=True); Lh.copy_(Ld, non_blocking=True); Sh.copy_(Sd, non_blocking=True)
                stream.synchronize()
            e2e_s = time.perf_counter() - t0
    ms_max, e2e_ms_max = replicas.max_over_ranks([ms, e2e_s * 1e3], dist, device="cuda")
    value = replicas.aggregate_throughput(flops * steps / 1e12, world, ms_max / 1e3)
    per_gpu = flops * steps / 1e12 / (ms_max / 1e3)
    msvid_launches = 1 + 4 + n_iter * (6 + (1 if l <= 4 else 0)) + 2 + 5
    out = {
        "metric": "admm_update_TFLOPs", "value": value, "unit": "TFLOP/s", "steps": steps, "warmup": max(3, warmup),
        "ms_per_step": ms_max / steps,
        "config": {"workload": workload, "description": f"ADMM update of an {N} x {R} factor for a {N} x {Mc} matrix, l={l}, {n_inner} inner "
                                                        f"iteration(s), {n_iter} subspace iterations per MSVID step; dense-algebra flops of the "
                                                        "least-squares step counted",
                   "layers": 1, "T": 0, "weights_MB": round(N * Mc * 4 / 1e6, 1), "l2_policy": "matrices larger than L2",
                   "launch": "stream launches", "kernel": "admm", "grouping": "one call per step", "replicas": world},
        "e2e": ({"value": replicas.aggregate_throughput(flops * e2e_steps / 1e12, world, e2e_ms_max / 1e3), "unit": "TFLOP/s",
                 "h2d_bytes_per_step": (N * Mc + Mc * R + N * R) * 4, "d2h_bytes_per_step": 2 * N * R * 4 + N * nwords * 4}
                if want_e2e else None),
        # this library's kernels (the solver library's are not counted): 2 splits + 2 products + ridge + identity + split, product,
        # split for the inverse + flag; per inner iteration rhs, split, product, sum, MSVID, reconstruction
        "gpu_launches": (10 + n_inner * (5 + msvid_launches)) * steps,
        "clocks": clocks,
        "roofline": {"bound": "tensor", "achieved": per_gpu, "peak": peak, "unit": "TFLOP/s", "frac": per_gpu / peak,
                     "peak_source": f"of {peak_kind}: the sustained bf16 GEMM figure (kind::tf32 issues at the 16-bit rate on this part: 1.6 PFLOP/s "
                                    "executed with the tensor pipe 75 % busy); the three-term split spends three tensor-core products per "
                                    "product counted, so a third of the peak is this scheme's ceiling",
                     "kernel": "gemm3x_kernel", "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get((workload, "gemm3x_kernel"))},
    }
    del Wd, Vd, U0, Ud, Ld, ws
    torch.cuda.empty_cache()
    return out, ("admm", N, Mc, R, l, n_inner)


def cpu_baseline_admm(N, Mc, R, l, n_inner):
    """The oracle's update (fp64, exact SVD in the prox step) on a leading block of the workload, rated in the same flops."""
    from oracle import mdbf_oracle as orc
    from paper_2512_24545_b200 import inputs
    n, m, r = min(N, 1024), min(Mc, 1024), min(R, 512)
    W, V, U = (inputs.make_factor_matrix(a, b, seed=60 + i, special_values=False) for i, (a, b) in enumerate([(n, m), (m, r), (n, r)]))
    rho = float(np.sum(V.astype(np.float64) ** 2)) / r
    t0 = time.perf_counter()
    orc.admm_factor_update(W, V, U, np.zeros_like(U), rho, min(l, r), n_inner)
    dt = time.perf_counter() - t0
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    return {"value": admm_flops(n, m, r, n_inner) / 1e12 / dt, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
            "sample": f"fp64 update of a {n} x {r} factor for a {n} x {m} block, one call, {dt:.1f} s"}


# workloads the default line reports beside the headline one: the largest decode configuration, the MLP shapes at one
# and at sixteen tokens, the prefill point under the library's own choice and under the expanded order (the metric's
# own unit), the block prefill, the quantizer's first step on a factor of the block's largest layer and one refinement
# update at the shape of the block's q / o projections
ALSO = [("block70b_T1", "auto"), ("block70b_T1", "fused"), ("decode_mlp_T1", "auto"), ("decode_mlp_T16", "auto"), ("prefill_4096_l16_bpw10", "auto"),
        ("prefill_4096_l16_bpw10", "prefill"), ("block70b_T2048", "auto"), ("msvid_28672x6016_l16", "auto"),
        ("admm_8192x8192_r3712_l16", "auto")]


def run_mdbf(args):
    import torch
    from paper_2512_24545_b200 import build
    build.build()
    dist, rank, world, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    if args.workload.startswith("msvid"):
        main, cpu_args = measure_msvid(args.workload, args.steps, args.warmup, dist, world, local)
    elif args.workload.startswith("admm"):
        main, cpu_args = measure_admm(args.workload, args.steps, args.warmup, dist, world, local)
    else:
        main, cpu_args = measure(args.workload, args.kernel, args.steps, args.warmup, dist, world, local,
                                 no_graph=args.no_graph, no_siblings=args.no_siblings, copies=args.copies, fuse_block=args.fuse_block)
    out = {
        "metric": main["metric"], "value": main["value"], "unit": main["unit"], "n_gpus": world, "steps": main["steps"],
        "warmup": main["warmup"], "ms_per_step": main["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32" if args.workload.startswith(("msvid", "admm")) else "bf16", "data": "synthetic",
        "config": main["config"], "e2e": main["e2e"], "gpu_launches": main["gpu_launches"], "clocks": main["clocks"],
        "roofline": main["roofline"],
    }
    if world == 1 and args.also and args.workload == "decode_qproj" and args.kernel == "auto":
        also = {}
        for (wl, kern) in ALSO:
            if wl.startswith("msvid"):
                m, _ = measure_msvid(wl, max(3, min(args.steps, 10)), args.warmup, None, 1, local, want_e2e=False, min_timed_ms=60.0)
            elif wl.startswith("admm"):
                m, _ = measure_admm(wl, max(3, min(args.steps, 10)), args.warmup, None, 1, local, want_e2e=False)
            else:
                m, _ = measure(wl, "auto" if kern == "fused" else kern, max(3, min(args.steps, 10)), args.warmup, None, 1, local,
                               want_e2e=False, fuse_block=kern == "fused", min_timed_ms=60.0)
            also[wl if kern == "auto" else f"{wl}:{kern}"] = {
                "metric": m["metric"], "value": m["value"], "unit": m["unit"], "ms_per_step": m["ms_per_step"],
                "steps": m["steps"], "gpu_launches": m["gpu_launches"], "clocks": m["clocks"], "roofline": m["roofline"],
                "config": {k: m["config"][k] for k in ("layers", "T", "weights_MB", "l2_policy", "kernel", "grouping")}}
        out["also"] = also
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        if cpu_args[0] == "msvid":
            out["cpu_baseline"] = cpu_baseline_msvid(*cpu_args[1:])
        elif cpu_args[0] == "admm":
            out["cpu_baseline"] = cpu_baseline_admm(*cpu_args[1:])
        else:
            spec0, T, bound, mat0 = cpu_args
            out["cpu_baseline"] = cpu_baseline(spec0, T, bound, budget_s=20.0, mat=mat0)
    if dist:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


# -------------------------------------------------------- oracle (CPU) arm
def oracle_sample(spec, T, rows_frac):
    """One bounded sample of the oracle: the dense definition restricted to a
    leading fraction of the output rows of one layer.  Returns (seconds, fraction)."""
    from oracle import mdbf_oracle as orc
    from paper_2512_24545_b200 import inputs
    lay = inputs.make_layer(spec)
    x = inputs.make_activations(spec, T)
    n = max(1, int(round(spec.d_out * rows_frac)))
    rows = np.arange(n)
    args = (lay["S_A"], lay["S_B"], lay["U_A"], lay["V_A"], lay["U_B"], lay["V_B"])
    t0 = time.perf_counter()
    W = orc.reconstruct_rows(rows, *args)
    y = W @ x.T.astype(np.float64)
    dt = time.perf_counter() - t0
    assert np.all(np.isfinite(y))
    return dt, n / spec.d_out


def cpu_baseline(spec, T, bound, budget_s=15.0, mat=False):
    cores = len(os.sched_getaffinity(0))
    dt, frac = oracle_sample(spec, T, 1.0 / 64)          # probe
    frac_target = min(1.0, max(1.0 / 64, frac * budget_s / max(dt, 1e-3) * 0.5))
    dt, frac = oracle_sample(spec, T, frac_target)
    reps, total = 1, dt
    while total < budget_s and reps < 200:               # repeat the sample until ~budget_s of CPU work
        d2, _ = oracle_sample(spec, T, frac_target)
        total += d2
        reps += 1
    dt = total / reps
    if bound == "hbm":
        v, unit = algorithmic_bytes(spec, T) * frac / 1e9 / dt, "GB/s"
    else:
        v, unit = (materialised_flops if mat else expanded_flops)(spec, T) * frac / 1e12 / dt, "TFLOP/s"
    return {"value": v, "unit": unit, "cores": cores, "kind": "oracle",
            "sample": f"fp64 dense definition on the first {frac:.3f} of the output rows of one "
                      f"{spec.name} layer, T={T}, {reps} repetitions of {dt:.2f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    if args.workload.startswith("msvid"):
        # the oracle's MSVID (sign mask + full SVD, fp64) on a leading block of the workload's matrix per step; the metric
        # counts the same algorithmic bytes per element of Z as the GPU arm's call (2 n + 1 passes)
        import re
        from oracle import mdbf_oracle as orc
        from paper_2512_24545_b200 import inputs
        m = re.match(r"msvid_(\d+)x(\d+)_l(\d+)(?:_it(\d+))?$", args.workload)
        if not m:
            raise SystemExit(f"unknown workload {args.workload}")
        rows, cols, l = int(m.group(1)), int(m.group(2)), int(m.group(3))
        n_iter = int(m.group(4)) if m.group(4) else 4
        sub_r, sub_c = min(rows, 1024), min(cols, 2048)
        Z = inputs.make_factor_matrix(sub_r, sub_c, seed=8)
        for _ in range(args.warmup):
            orc.msvid(Z, l)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            orc.msvid(Z, l)
        total = time.perf_counter() - t0
        value = (2 * n_iter + 1) * Z.size * 4 / 1e9 * args.steps / total
        sample = f"fp64 sign mask + full SVD of a {sub_r} x {sub_c} block of the workload's matrix per step"
        print(json.dumps({
            "impl": "reference", "metric": "msvid_algorithmic_GBps", "value": value, "unit": "GB/s",
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "description": f"MSVID_l of a {rows} x {cols} fp32 factor, l={l}"},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return
    if args.workload.startswith("admm"):
        from oracle import mdbf_oracle as orc
        from paper_2512_24545_b200 import inputs
        N, Mc, R, l, n_inner = admm_shape(args.workload)
        n, m, r = min(N, 512), min(Mc, 512), min(R, 256)
        W, V, U = (inputs.make_factor_matrix(a, b, seed=60 + i, special_values=False) for i, (a, b) in enumerate([(n, m), (m, r), (n, r)]))
        rho = float(np.sum(V.astype(np.float64) ** 2)) / r
        for _ in range(args.warmup):
            orc.admm_factor_update(W, V, U, np.zeros_like(U), rho, min(l, r), n_inner)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            orc.admm_factor_update(W, V, U, np.zeros_like(U), rho, min(l, r), n_inner)
        total = time.perf_counter() - t0
        value = admm_flops(n, m, r, n_inner) / 1e12 * args.steps / total
        sample = f"fp64 update of a {n} x {r} factor for a {n} x {m} block of the workload per step"
        print(json.dumps({
            "impl": "reference", "metric": "admm_update_TFLOPs", "value": value, "unit": "TFLOP/s",
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "description": f"ADMM update of an {N} x {R} factor for a {N} x {Mc} matrix, l={l}"},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return
    groups, T, bound, desc = workload_specs(args.workload)
    spec = groups[0][0]
    dt, frac = oracle_sample(spec, T, 1.0 / 64)
    budget = 120.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, max(1.0 / 64, frac * budget / max(dt, 1e-3) * 0.5))
    for _ in range(args.warmup):
        oracle_sample(spec, T, frac)
    total = 0.0
    for _ in range(args.steps):
        dt, fr = oracle_sample(spec, T, frac)
        total += dt
    if bound == "hbm":
        metric, unit = "decode_algorithmic_GBps", "GB/s"
        per = algorithmic_bytes(spec, T) * fr / 1e9
    else:
        mat = rated_materialised(spec, T, args.kernel)    # same work unit as the arm it is compared with
        metric, unit = ("prefill_executed_TFLOPs" if mat else "prefill_expanded_TFLOPs"), "TFLOP/s"
        per = (materialised_flops if mat else expanded_flops)(spec, T) * fr / 1e12
    value = per * args.steps / total
    sample = (f"fp64 dense definition on the first {fr:.3f} of the output rows of one {spec.name} "
              f"layer per step, T={T}")
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": unit,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "description": desc},
        "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="decode_qproj")
    ap.add_argument("--impl", default="mdbf", choices=["mdbf", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every forward from the host")
    ap.add_argument("--kernel", default="auto", choices=["auto", "prefill", "mat", "tmem", "i8"],
                    help="T > 1: force the expanded-order (prefill) or the materialised-order (mat) kernel; "
                         "T = 1: force the bf16 TMEM-operand (tmem) or the integer (i8) kernel")
    ap.add_argument("--fuse-block", action="store_true",
                    help="block workloads at one token: the seven layers as independent forwards in one set of launches")
    ap.add_argument("--no-also", dest="also", action="store_false",
                    help="default workload only: skip the extra workloads reported under \"also\"")
    ap.add_argument("--no-siblings", action="store_true", help="block workloads: one forward per layer instead of fused q/k/v and gate/up")
    ap.add_argument("--copies", type=int, default=0, help="distinct layers per shape (0 = workload default); small values for ncu captures")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_mdbf(args)


if __name__ == "__main__":
    main()
