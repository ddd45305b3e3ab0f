#!/usr/bin/env python
"""Benchmark of the quantised-linear hot path on the Llama-2-7B w2g64 block workload.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One step = one pass of the whole path over the seven linear layers of a
Llama-2-7B decoder block at 2 bits, group 64:
    min/max init, Block-AP forward and backward at 4096 tokens (batch 2 x 2048),
    hand-off (quantise + pack, unpack), E2E-QP forward / dX / ds at 16384 tokens.
Prints one JSON line (rank 0).  `value` is the tensor-core throughput of the six
contractions per linear (2*T*in*out flop each) over the whole step, all kernels
included in the time; dequantisation, STE and epilogue arithmetic are not counted
as flops.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from workloads import LINEARS

BITS, GROUP = 2, 64
T_BLOCK_AP, T_E2E = 4096, 16384
WORKLOAD = "llama2-7b decoder-block linears, w2g64: Block-AP fwd+bwd @4096 tok, hand-off, E2E-QP fwd/dX/ds @16384 tok"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM bytes (read + write) per launch of the packed-weight GEMMs at 16384 tokens, w2g64, by linear shape: ncu
# `dram__bytes_read.sum + dram__bytes_write.sum`, one capture per shape with `bench.py --kernel-case` (the summaries
# under profiles/ give the command).  They describe the kernels whose sources hash to `sources_sha256`; once those
# files change (comments and white space aside) the figures are stale and `roofline.traffic` is reported as null.
NCU_TRAFFIC = {
    "sources": ("gemm.cu", "ptx.cuh"),
    "sources_sha256": "3b2106bc3b7354efc28822654a030b5243cf54848a42562f6390b2b582091a92",
    "packed_fwd": {"qkvo": 139.26e6 + 93.10e6, "gate_up": 147.72e6 + 314.19e6, "down": 448.65e6 + 114.63e6},
    "packed_bwd_dx": {"qkvo": 139.26e6 + 93.85e6, "gate_up": 449.56e6 + 114.69e6, "down": 147.73e6 + 315.56e6},
    "packed_bwd_ds": {"qkvo": 416.23e6 + 0.85e6, "gate_up": 1306.73e6 + 3.00e6, "down": 1073.39e6 + 2.82e6},
}


def sources_fingerprint():
    """SHA-256 of the kernel sources with // comments and white space removed: what the compiler sees."""
    import hashlib
    import re
    h = hashlib.sha256()
    for f in NCU_TRAFFIC["sources"]:
        with open(os.path.join(ROOT, "paper_2407_11062_b200", "csrc", f), "r") as fh:
            text = re.sub(r"//[^\n]*", "", fh.read())
        h.update("".join(text.split()).encode())
    return h.hexdigest()


def traffic_per_launch(kernel_class):
    """Launch-weighted mean of the captured DRAM bytes over the class's launches in one step, or None if the
    kernel sources have changed since the capture."""
    table = NCU_TRAFFIC.get(kernel_class)
    if table is None or sources_fingerprint() != NCU_TRAFFIC["sources_sha256"]:
        return None
    n = sum(l.count for l in LINEARS["7b"])
    return sum(table[l.name] * l.count for l in LINEARS["7b"]) / n


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


def step_flops(t_block_ap=T_BLOCK_AP, t_e2e=T_E2E):
    per_token = sum(2 * l.in_features * l.out_features * l.count for l in LINEARS["7b"])
    return 3 * per_token * t_block_ap, 3 * per_token * t_e2e


# ----------------------------------------------------------------------------- distributed plumbing
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def max_over_ranks(value: float, device) -> float:
    """Largest value over all ranks (the slowest rank defines the step time)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the two datetimes (the timed region)."""
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        power = []
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                if t_begin is not None and not (t_begin <= ts <= t_end):
                    continue
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- the workload on one GPU
class BlockWorkload:
    """Device buffers for the seven linears; activations shared per shape, weights per linear."""

    def __init__(self, eqat, device, seed, t_block_ap=T_BLOCK_AP, t_e2e=T_E2E):
        self.eqat, self.device = eqat, device
        self.t_ap, self.t_e2e = t_block_ap, t_e2e
        g = torch.Generator(device=device); g.manual_seed(seed)
        bf, dev = torch.bfloat16, device
        self.shapes, self.layers = {}, []
        for lin in LINEARS["7b"]:
            out, in_f, ng = lin.out_features, lin.in_features, lin.in_features // GROUP
            sh = dict(lin=lin,
                      X=torch.randn(t_e2e, in_f, generator=g, device=dev, dtype=torch.float32).to(bf),
                      dY=(torch.randn(t_e2e, out, generator=g, device=dev, dtype=torch.float32) * 1e-2).to(bf),
                      Y=torch.empty(t_e2e, out, dtype=bf, device=dev), dX=torch.empty(t_e2e, in_f, dtype=bf, device=dev),
                      What=torch.empty(out, in_f, dtype=bf, device=dev), dW=torch.empty(out, in_f, dtype=bf, device=dev),
                      ds=torch.empty(out, ng, device=dev), dz=torch.empty(out, ng, device=dev),
                      ds2=torch.empty(out, ng, device=dev),
                      codes=torch.empty(out, in_f, dtype=torch.uint8, device=dev),
                      d_ap=eqat.make_desc(BITS, GROUP, out, in_f, t_block_ap), d_e2e=eqat.make_desc(BITS, GROUP, out, in_f, t_e2e))
            sh["ws"] = torch.empty(eqat.workspace_bytes(sh["d_ap"], eqat.EQAT_OP_FAKEQUANT_BWD), dtype=torch.uint8, device=dev)
            self.shapes[lin.name] = sh
            for i in range(lin.count):
                W = (torch.randn(out, in_f, generator=g, device=dev, dtype=torch.float32) * 0.02).to(bf)
                self.layers.append(dict(shape=lin.name, W=W,
                                        s=torch.empty(out, ng, device=dev), z=torch.empty(out, ng, device=dev),
                                        P=torch.empty(out, in_f * BITS // 8, dtype=torch.uint8, device=dev),
                                        z8=torch.empty(out, ng, dtype=torch.uint8, device=dev),
                                        s16=torch.empty(out, ng, dtype=torch.float16, device=dev)))
        self.calls_per_step = 8 * len(self.layers)
        self.kernels_per_step = 10 * len(self.layers)     # fwd = 2 kernels, bwd = 2 (group <= 256), the other six calls 1 each

    def step(self, timers=None):
        e = self.eqat
        def timed(name, fn):
            if timers is None:
                fn(); return
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            timers.setdefault(name, []).append((a, b))
        for L in self.layers:
            S = self.shapes[L["shape"]]
            Xa, dYa, Ya, dXa = S["X"][: self.t_ap], S["dY"][: self.t_ap], S["Y"][: self.t_ap], S["dX"][: self.t_ap]
            tag = L["shape"]
            timed("minmax_init/" + tag, lambda: e.eqat_minmax_init(S["d_ap"], L["W"], L["s"], L["z"]))
            timed("fakequant_fwd/" + tag, lambda: e.qlinear_fakequant_fwd(S["d_ap"], Xa, L["W"], L["s"], L["z"], Ya, S["What"]))
            timed("fakequant_bwd/" + tag, lambda: e.qlinear_fakequant_bwd(S["d_ap"], Xa, dYa, L["W"], L["s"], L["z"], S["What"],
                                                                            dXa, S["dW"], S["ds"], S["dz"], S["ws"]))
            timed("quantize_pack/" + tag, lambda: e.eqat_quantize_pack(S["d_ap"], L["W"], L["s"], L["z"], L["P"], L["z8"], L["s16"]))
            timed("unpack/" + tag, lambda: e.eqat_unpack(S["d_ap"], L["P"], S["codes"]))
            timed("packed_fwd/" + tag, lambda: e.qlinear_packed_fwd(S["d_e2e"], S["X"], L["P"], L["s16"], L["z8"], S["Y"]))
            timed("packed_bwd_dx/" + tag, lambda: e.qlinear_packed_bwd_dx(S["d_e2e"], S["dY"], L["P"], L["s16"], L["z8"], S["dX"]))
            timed("packed_bwd_ds/" + tag, lambda: e.qlinear_packed_bwd_ds(S["d_e2e"], S["X"], S["dY"], L["P"], L["z8"], L["s16"], S["ds2"]))


class HostStaging:
    """End-to-end leg: every step's X and dY come from pinned host memory and the weight-side
    gradients (dW, ds, dz of Block-AP, ds of E2E-QP) go back to pinned host memory, all inside the
    timed region.  Copies run on their own streams and are double-buffered per linear shape, so the
    upload of the next linear and the download of the previous one overlap the kernels of the
    current one (the step is then bound by whichever of PCIe and the GPU is slower)."""

    OUT = ("dW", "ds", "dz", "ds2")

    def __init__(self, wl: BlockWorkload):
        self.wl = wl
        self.host, self.sets, self.uses = {}, {}, {}
        for name, S in wl.shapes.items():
            self.host[name] = dict(
                X=S["X"].cpu().pin_memory(), dY=S["dY"].cpu().pin_memory(),
                **{k: torch.empty(S[k].shape, dtype=S[k].dtype).pin_memory() for k in self.OUT})
            second = {k: torch.empty_like(S[k]) for k in ("X", "dY") + self.OUT}
            self.sets[name] = [{k: S[k] for k in ("X", "dY") + self.OUT}, second]
            self.uses[name] = 0
        self.h2d = sum(self.host[L["shape"]]["X"].nbytes + self.host[L["shape"]]["dY"].nbytes for L in wl.layers)
        self.d2h = sum(sum(self.host[L["shape"]][k].nbytes for k in self.OUT) for L in wl.layers)
        self.up, self.down = torch.cuda.Stream(), torch.cuda.Stream()
        self.last_done = {}        # (shape, set) -> event: kernels that read/wrote this set have finished
        self.last_down = {}        # (shape, set) -> event: its gradients have been downloaded

    def step(self):
        wl, e = self.wl, self.wl.eqat
        main = torch.cuda.current_stream()
        start = torch.cuda.Event(); start.record(main)
        self.up.wait_event(start)                       # copies of this step start inside the timed region
        def upload(L):
            """Enqueue the upload of one linear's X and dY into the free buffer set of its shape."""
            name = L["shape"]
            k = self.uses[name] % 2
            self.uses[name] += 1
            D, H = self.sets[name][k], self.host[name]
            if (name, k) in self.last_done:             # the kernels that last read this set must be done
                self.up.wait_event(self.last_done[(name, k)])
            with torch.cuda.stream(self.up):
                D["X"].copy_(H["X"], non_blocking=True)
                D["dY"].copy_(H["dY"], non_blocking=True)
                ev = torch.cuda.Event(); ev.record(self.up)
            return k, ev

        nxt = upload(wl.layers[0])
        for i, L in enumerate(wl.layers):
            k, ev = nxt
            if i + 1 < len(wl.layers):
                nxt = upload(wl.layers[i + 1])          # one linear ahead: overlaps this linear's kernels
            name = L["shape"]
            S, D, H = wl.shapes[name], self.sets[name][k], self.host[name]
            main.wait_event(ev)
            if (name, k) in self.last_down:
                main.wait_event(self.last_down[(name, k)])
            X, dY = D["X"], D["dY"]
            Xa, dYa, Ya, dXa = X[: wl.t_ap], dY[: wl.t_ap], S["Y"][: wl.t_ap], S["dX"][: wl.t_ap]
            e.eqat_minmax_init(S["d_ap"], L["W"], L["s"], L["z"])
            e.qlinear_fakequant_fwd(S["d_ap"], Xa, L["W"], L["s"], L["z"], Ya, S["What"])
            e.qlinear_fakequant_bwd(S["d_ap"], Xa, dYa, L["W"], L["s"], L["z"], S["What"], dXa, D["dW"], D["ds"], D["dz"], S["ws"])
            e.eqat_quantize_pack(S["d_ap"], L["W"], L["s"], L["z"], L["P"], L["z8"], L["s16"])
            e.eqat_unpack(S["d_ap"], L["P"], S["codes"])
            e.qlinear_packed_fwd(S["d_e2e"], X, L["P"], L["s16"], L["z8"], S["Y"])
            e.qlinear_packed_bwd_dx(S["d_e2e"], dY, L["P"], L["s16"], L["z8"], S["dX"])
            e.qlinear_packed_bwd_ds(S["d_e2e"], X, dY, L["P"], L["z8"], L["s16"], D["ds2"])
            done = torch.cuda.Event(); done.record(main)
            self.last_done[(name, k)] = done
            self.down.wait_event(done)
            with torch.cuda.stream(self.down):
                for o in self.OUT:
                    H[o].copy_(D[o], non_blocking=True)
                dn = torch.cuda.Event(); dn.record(self.down)
            self.last_down[(name, k)] = dn
        main.wait_stream(self.up)
        main.wait_stream(self.down)                     # the step ends when its last gradient is on the host


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(seed=0):
    """The oracle on a bounded sample of the same workload: the 4096x4096 linear,
    element-wise steps on 512 output rows, contractions on 256 token rows x 512
    output rows.  Returns (flops counted the same way, seconds, description)."""
    from oracle import eqat_oracle as O
    from workloads import from_bf16_bits, get_config, normal_bf16
    rows, toks, in_f = 512, 256, 4096
    Wb = normal_bf16((rows, in_f), 0.02, "bench_oracle", seed, "W")
    Xb = normal_bf16((toks, in_f), 1.0, "bench_oracle", seed, "X")
    dYb = normal_bf16((toks, rows), 1e-2, "bench_oracle", seed, "dY")
    W, X, dY = from_bf16_bits(Wb), from_bf16_bits(Xb), from_bf16_bits(dYb)
    t0 = time.perf_counter()
    s, z = O.minmax_init(W, BITS, GROUP)
    What = O.fake_quant_weight(W, s, z, BITS, GROUP)
    Y = O.linear_fwd(X, What); dX = O.linear_bwd_dx(dY, What)
    G = O.weight_grad(dY, X)
    O.ste_bwd(G, W, s, z, BITS, GROUP)
    P, z8, s16 = O.quantize_pack(W, s, z, BITS, GROUP)
    q = O.unpack_rows(P, BITS, in_f)
    Wq = O.dequantize(q, s16.astype(np.float32), z8, GROUP)
    O.linear_fwd(X, Wq); O.linear_bwd_dx(dY, Wq)
    O.e2e_ds(dY, X, q, z8, GROUP)
    dt = time.perf_counter() - t0
    flops = 6 * 2 * toks * in_f * rows
    return flops, dt, f"4096-wide linear, {rows} output rows x {toks} tokens, all steps of the path (w2g64)"


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(budget_s=15.0):
    flops, dt, what = oracle_sample(0)
    reps, total_f, total_t = 1, flops, dt
    while total_t < budget_s and reps < 64:
        f, t, _ = oracle_sample(reps)
        total_f += f; total_t += t; reps += 1
    return {"value": total_f / total_t / 1e12, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle",
            "sample": f"{reps} x ({what}); {total_t:.1f} s of CPU time"}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    times, flops = [], 0
    for i in range(args.warmup + args.steps):
        f, t, what = oracle_sample(i)
        if i >= args.warmup:
            times.append(t); flops = f
    ms = 1e3 * sum(times) / len(times)
    val = flops / (ms * 1e-3) / 1e12
    out = {"impl": "reference", "metric": "QLinear fwd+bwd TFLOP/s", "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": WORKLOAD, "step": "bounded sample: " + what},
           "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle", "sample": what},
           "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# ----------------------------------------------------------------------------- main
def summarise(timers):
    out = {}
    for name, pairs in timers.items():
        ms = [a.elapsed_time(b) for a, b in pairs]
        out[name] = {"launches": len(ms), "avg_ms": sum(ms) / len(ms), "total_ms": sum(ms)}
    return out


def run_ours(args):
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding as eqat
    peaks = load_peaks()

    import datetime
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    wl = BlockWorkload(eqat, device, seed=20240711 + rank)     # each rank: its own token batch (weak scaling)
    for _ in range(max(args.warmup, 3)):
        wl.step()
    torch.cuda.synchronize()
    timers = {}
    barrier(); torch.cuda.synchronize()
    t_begin = datetime.datetime.now()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        wl.step(timers)
    t1.record()
    torch.cuda.synchronize(); barrier()
    t_end = datetime.datetime.now()
    ms_local = t0.elapsed_time(t1) / args.steps
    ms = max_over_ranks(ms_local, device)
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    st = eqat.device_status()
    if st != (0, 0):
        raise SystemExit(f"device status {st}: a kernel abandoned a wait")

    # end-to-end leg: host buffers in, gradients out, copies inside the timed region
    stage = HostStaging(wl)
    e2e_steps = max(1, min(args.steps, 3))
    stage.step(); torch.cuda.synchronize(); barrier()
    t0.record()
    for _ in range(e2e_steps):
        stage.step()
    t1.record()
    torch.cuda.synchronize(); barrier()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1) / e2e_steps, device)

    f_ap, f_e2e = step_flops()
    flops = (f_ap + f_e2e) * world
    if rank == 0:
        kern = summarise(timers)
        by_class = {}
        for name, v in kern.items():
            c = name.split("/")[0]
            by_class.setdefault(c, 0.0)
            by_class[c] += v["total_ms"]
        top_class = max(by_class, key=by_class.get)
        # roofline of the dominant kernel (each packed_* call is exactly one kernel launch)
        t_tok = {"packed_fwd": T_E2E, "packed_bwd_dx": T_E2E, "packed_bwd_ds": T_E2E}
        roof = None
        if top_class in t_tok:
            tot_f = sum(2 * T_E2E * l.in_features * l.out_features * l.count for l in LINEARS["7b"]) * args.steps
            tot_ms = by_class[top_class]
            ach = tot_f / (tot_ms * 1e-3) / 1e12
            peak = peaks["bf16_tflops_sustained"]
            roof = {"kernel": "gemm_kernel (" + top_class + ")", "bound": "tensor", "achieved": ach, "peak": peak,
                    "unit": "TFLOP/s", "frac": ach / peak, "peak_source": peaks["source"] + " (sustained)", "traffic": traffic_per_launch(top_class),
                    "traffic_unit": "DRAM bytes per launch (ncu, launch-weighted mean over the class)",
                    "algorithmic_bytes": sum((T_E2E * (l.in_features + l.out_features) * 2
                                              + l.in_features * l.out_features * BITS // 8) * l.count
                                             for l in LINEARS["7b"]) / sum(l.count for l in LINEARS["7b"])}
        classes = {c: {"total_ms_per_step": t / args.steps, "share": t / sum(by_class.values())} for c, t in by_class.items()}
        # every class that is exactly one kernel launch per call also gets its own roofline figure:
        # the contractions against the sustained bf16 peak, the streaming kernels against the copy bandwidth
        n_elem = sum(l.in_features * l.out_features * l.count for l in LINEARS["7b"])
        n_grp = n_elem / GROUP
        hbm_bytes = {"minmax_init": 2 * n_elem + 8 * n_grp,
                     "quantize_pack": (2 + BITS / 8) * n_elem + 11 * n_grp,
                     "unpack": (1 + BITS / 8) * n_elem}
        e2e_flops = sum(2 * T_E2E * l.in_features * l.out_features * l.count for l in LINEARS["7b"])
        for c, t in by_class.items():
            sec = t * 1e-3 / args.steps
            if c in hbm_bytes:
                ach = hbm_bytes[c] / sec / 1e9
                classes[c]["roofline"] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                          "frac": ach / peaks["hbm_gbs"]}
            elif c in t_tok:
                ach = e2e_flops / sec / 1e12
                classes[c]["roofline"] = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                                          "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                                          "traffic": traffic_per_launch(c)}
        out = {"metric": "QLinear fwd+bwd TFLOP/s", "value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "n_gpus": world,
               "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": {"workload": WORKLOAD, "bits": BITS, "group": GROUP, "tokens_block_ap": T_BLOCK_AP, "tokens_e2e_qp": T_E2E,
                          "l2": "inputs larger than L2 (working set > 2 GB per shape, weights per linear)"},
               "pct_of_bf16_peak": 100.0 * flops / world / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
               "block_tokens_per_s": {"block_ap": None, "e2e_qp": None},
               "roofline": roof, "kernel_classes": classes, "clocks": clocks,
               "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": stage.h2d, "d2h_bytes_per_step": stage.d2h},
               "gpu_launches": wl.kernels_per_step * args.steps}
        ap_ms = sum(by_class.get(c, 0.0) for c in ("fakequant_fwd", "fakequant_bwd")) / args.steps
        qp_ms = sum(by_class.get(c, 0.0) for c in ("packed_fwd", "packed_bwd_dx", "packed_bwd_ds")) / args.steps
        out["block_tokens_per_s"] = {"block_ap": world * T_BLOCK_AP / (ap_ms * 1e-3), "e2e_qp": world * T_E2E / (qp_ms * 1e-3)}
        out["tflops_by_mode"] = {"block_ap": f_ap / (ap_ms * 1e-3) / 1e12, "e2e_qp": f_e2e / (qp_ms * 1e-3) / 1e12}
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline()
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_kernel_case(args):
    """One call class on one linear shape, a few launches: the small case used for ncu captures."""
    torch.cuda.set_device(0)
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding as eqat
    wl = BlockWorkload(eqat, torch.device("cuda", 0), seed=1, t_block_ap=args.case_tokens, t_e2e=args.case_tokens)
    wl.layers = [L for L in wl.layers if L["shape"] == args.case_shape][:1]
    for _ in range(2):
        wl.step()                       # fills s, z, packed codes
    torch.cuda.synchronize()
    timers = {}
    for _ in range(args.case_iters):
        wl.step(timers)
    torch.cuda.synchronize()
    assert eqat.device_status() == (0, 0)
    print(json.dumps({k: v for k, v in summarise(timers).items()}), flush=True)


def run_decode_case(args):
    """Few-token packed forward (the matrix-vector kernel) on the block's three linear shapes: device time per
    launch from a CUDA graph of launches over rotating weight copies (more than L2 in total), and the bandwidth that
    time means for the bytes one launch must read."""
    torch.cuda.set_device(0)
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding as eqat
    peaks = load_peaks()
    dev = torch.device("cuda", 0)
    out = {"metric": "packed forward, few tokens", "unit": "us per launch", "bits": BITS, "group": GROUP,
           "hbm_gbs_peak": peaks["hbm_gbs"], "cases": {}}
    for lin in LINEARS["7b"]:
        o, i = lin.out_features, lin.in_features
        ng = i // GROUP
        wbytes = o * i * BITS // 8
        copies = max(4, int(320e6 // wbytes))
        Ps = [torch.randint(0, 256, (o, i * BITS // 8), dtype=torch.uint8, device=dev) for _ in range(copies)]
        z8 = torch.randint(0, 1 << BITS, (o, ng), dtype=torch.uint8, device=dev)
        s16 = (torch.rand(o, ng, device=dev) * 0.01 + 0.001).half()
        for T in (1, 4):
            X = torch.randn(T, i, device=dev).to(torch.bfloat16)
            Y = torch.empty(T, o, dtype=torch.bfloat16, device=dev)
            d = eqat.make_desc(BITS, GROUP, o, i, T)
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                for P in Ps[:3]:
                    eqat.qlinear_packed_fwd(d, X, P, s16, z8, Y)       # warm-up, outside the capture
                side.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for P in Ps:
                        eqat.qlinear_packed_fwd(d, X, P, s16, z8, Y)
                g.replay(); side.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(side)
                for _ in range(args.case_iters):
                    g.replay()
                e1.record(side)
                side.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (args.case_iters * copies)
            nbytes = wbytes + o * ng * 3 + T * (i + o) * 2
            out["cases"][f"{lin.name}/T{T}"] = {"us": us, "bytes": nbytes, "gbs": nbytes / us / 1e3,
                                                 "frac_of_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}
        del Ps
    assert eqat.device_status() == (0, 0)
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel-case", action="store_true", help="run one linear shape a few times (for profilers)")
    ap.add_argument("--decode-case", action="store_true",
                    help="time the few-token packed forward on the block's linear shapes (uses --case-iters)")
    ap.add_argument("--case-shape", default="qkvo", choices=[l.name for l in LINEARS["7b"]])
    ap.add_argument("--case-tokens", type=int, default=16384)
    ap.add_argument("--case-iters", type=int, default=2)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.kernel_case:
        run_kernel_case(args)
    elif args.decode_case:
        run_decode_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
