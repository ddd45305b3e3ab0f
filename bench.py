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

On one GPU the same run then times, outside the headline's timed region and reported under their own keys:
the other workloads (7B w4g128 Block-AP, 13B w3g128 E2E-QP, 70B w2g64 both modes) under "configs", and the five
streaming kernels on cold data, back to back over buffer sets several times the L2, under "streaming" (once before
the GEMM phases of the run and again after them, with the GPU's clocks read beside each).
`--gpus N` started without a launcher spawns the N ranks itself.
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
# Nominal figures of the part, for context beside the measured denominators: dense bf16 tensor throughput and the
# HBM3e bandwidth the workload description quotes ("~8 TB/s").
NOMINAL_PEAKS = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}

# The other workloads: same path, other bit widths, group sizes and models.  Each is timed after the headline
# step and reported under "configs" (the headline line itself stays the 7B w2g64 step).
#   model, bits, group, Block-AP tokens (0 = mode not run), E2E-QP tokens, weight recipe (dist, scale, outlier fraction)
EXTRA_CONFIGS = {
    "c2_7b_w4g128_block_ap": dict(model="7b", bits=4, group=128, t_ap=4096, t_e2e=0, w=("student_t4", 0.02, 0.01), steps=10),
    "c4_13b_w3g128_e2e_qp": dict(model="13b", bits=3, group=128, t_ap=0, t_e2e=8192, w=("student_t4", 0.02, 0.01), steps=10),
    "c5_70b_w2g64_both": dict(model="70b", bits=2, group=64, t_ap=8192, t_e2e=8192, w=("student_t4", 0.015, 0.0), steps=5),
}


# DRAM bytes (read + write) per launch of the packed-weight GEMMs at 16384 tokens, w2g64, by linear shape: ncu
# `dram__bytes_read.sum + dram__bytes_write.sum`, one capture per shape with `bench.py --kernel-case` (the summaries
# under profiles/ give the command).  They describe the kernels whose sources hash to `sources_sha256`; once those
# files change (comments and white space aside) the figures are stale and `roofline.traffic` is reported as null.
NCU_TRAFFIC = {
    "sources": ("gemm.cu", "ptx.cuh"),
    "sources_sha256": "80fde187933896517192d9f4487bb958fba6b2499e62d11aadddd993f376ce5e",
    "packed_fwd": {"qkvo": 141.3e6 + 96.9e6, "gate_up": 163.8e6 + 315.0e6, "down": 503.9e6 + 116.0e6},
    "packed_bwd_dx": {"qkvo": 140.5e6 + 96.6e6, "gate_up": 514.8e6 + 116.0e6, "down": 153.7e6 + 315.5e6},
    "packed_bwd_ds": {"qkvo": 416.2e6 + 0.8e6, "gate_up": 1306.4e6 + 2.8e6, "down": 1073.4e6 + 2.8e6},
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


def step_flops(t_block_ap=T_BLOCK_AP, t_e2e=T_E2E, model="7b"):
    per_token = sum(2 * l.in_features * l.out_features * l.count for l in LINEARS[model])
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


def gpu_state(index: int):
    """One reading of the GPU's clocks, power and temperature (None where nvidia-smi is not available)."""
    try:
        o = subprocess.run(["nvidia-smi", "-i", str(index), "--query-gpu=clocks.sm,clocks.mem,power.draw,temperature.gpu",
                            "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
        f = [float(x) for x in o.strip().split(",")]
        return {"sm_mhz": f[0], "mem_mhz": f[1], "power_w": f[2], "temp_c": f[3]}
    except (OSError, ValueError, IndexError, subprocess.SubprocessError):
        return None


# ----------------------------------------------------------------------------- the workload on one GPU
def synth_weight(shape, recipe, gen, device):
    """Synthetic stand-in for a trained weight, drawn on the device: N(0, scale^2) or scale * Student-t(4)
    (Z / sqrt(mean of four squared normals)), optionally with a fraction of the input channels scaled by 10."""
    dist, scale, outlier_frac = recipe
    w = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if dist == "student_t4":
        chi = torch.zeros(shape, device=device, dtype=torch.float32)
        for _ in range(4):
            chi += torch.randn(shape, generator=gen, device=device, dtype=torch.float32) ** 2
        w = w / torch.sqrt(chi / 4)
    w *= scale
    if outlier_frac > 0:
        n = int(np.ceil(outlier_frac * shape[1]))
        cols = torch.randperm(shape[1], generator=gen, device=device)[:n]
        w[:, cols] *= 10.0
    return w.to(torch.bfloat16)


# kernels launched by one call of each class (groups of at most 256 elements)
KERNELS_PER_CALL = {"minmax_init": 1, "fakequant_fwd": 2, "fakequant_bwd": 2, "quantize_pack": 1, "unpack": 1,
                    "packed_fwd": 1, "packed_bwd_dx": 1, "packed_bwd_ds": 1}
# contractions (2*T*in*out flop each) inside one call of each class
CONTRACTIONS = {"fakequant_fwd": 1, "fakequant_bwd": 2, "packed_fwd": 1, "packed_bwd_dx": 1, "packed_bwd_ds": 1}


class BlockWorkload:
    """Device buffers for the linears of one decoder block; activations shared per shape, weights per linear.

    One step = for every linear: [min/max init,] Block-AP forward + backward at `t_ap` tokens, [quantise + pack,
    unpack,] E2E-QP forward / dX / ds at `t_e2e` tokens.  A mode with 0 tokens is left out; the bracketed
    hand-off calls are part of the step only with `handoff` (the headline step), otherwise they run once here."""

    def __init__(self, eqat, device, seed, t_block_ap=T_BLOCK_AP, t_e2e=T_E2E, model="7b", bits=BITS, group=GROUP,
                 weight=("normal", 0.02, 0.0), handoff=True, store_w_hat=True):
        self.eqat, self.device = eqat, device
        self.store_w_hat = store_w_hat                     # False: W_hat is not kept, the GEMMs fake-quantise W themselves
        self.t_ap, self.t_e2e, self.model, self.bits, self.group, self.handoff = t_block_ap, t_e2e, model, bits, group, handoff
        g = torch.Generator(device=device); g.manual_seed(seed)
        bf, dev = torch.bfloat16, device
        t_max = max(t_block_ap, t_e2e)
        self.shapes, self.layers = {}, []
        for lin in LINEARS[model]:
            out, in_f, ng = lin.out_features, lin.in_features, lin.in_features // group
            sh = dict(lin=lin,
                      X=torch.randn(t_max, in_f, generator=g, device=dev, dtype=torch.float32).to(bf),
                      dY=(torch.randn(t_max, out, generator=g, device=dev, dtype=torch.float32) * 1e-2).to(bf),
                      Y=torch.empty(t_max, out, dtype=bf, device=dev), dX=torch.empty(t_max, in_f, dtype=bf, device=dev),
                      What=torch.empty(out, in_f, dtype=bf, device=dev), dW=torch.empty(out, in_f, dtype=bf, device=dev),
                      ds=torch.empty(out, ng, device=dev), dz=torch.empty(out, ng, device=dev),
                      ds2=torch.empty(out, ng, device=dev),
                      codes=torch.empty(out, in_f, dtype=torch.uint8, device=dev) if handoff else None,
                      d_ap=eqat.make_desc(bits, group, out, in_f, max(t_block_ap, 1)),
                      d_e2e=eqat.make_desc(bits, group, out, in_f, max(t_e2e, 1)))
            n_ws = eqat.workspace_bytes(sh["d_ap"], eqat.EQAT_OP_FAKEQUANT_BWD)
            sh["ws"] = torch.empty(n_ws, dtype=torch.uint8, device=dev) if n_ws else None
            self.shapes[lin.name] = sh
            for i in range(lin.count):
                W = synth_weight((out, in_f), weight, g, dev)
                L = dict(shape=lin.name, W=W,
                         s=torch.empty(out, ng, device=dev), z=torch.empty(out, ng, device=dev),
                         P=torch.empty(out, in_f * bits // 8, dtype=torch.uint8, device=dev),
                         z8=torch.empty(out, ng, dtype=torch.uint8, device=dev),
                         s16=torch.empty(out, ng, dtype=torch.float16, device=dev))
                eqat.eqat_minmax_init(sh["d_ap"], W, L["s"], L["z"])
                eqat.eqat_quantize_pack(sh["d_ap"], W, L["s"], L["z"], L["P"], L["z8"], L["s16"])
                self.layers.append(L)
        self.classes = ((["minmax_init"] if handoff else []) + (["fakequant_fwd", "fakequant_bwd"] if t_block_ap else [])
                        + (["quantize_pack", "unpack"] if handoff else [])
                        + (["packed_fwd", "packed_bwd_dx", "packed_bwd_ds"] if t_e2e else []))
        self.calls_per_step = len(self.classes) * len(self.layers)
        self.kernels_per_step = sum(KERNELS_PER_CALL[c] for c in self.classes) * len(self.layers)

    def flops(self):
        return step_flops(self.t_ap, self.t_e2e, self.model)

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
            tag = L["shape"]
            if self.handoff:
                timed("minmax_init/" + tag, lambda: e.eqat_minmax_init(S["d_ap"], L["W"], L["s"], L["z"]))
            if self.t_ap:
                Xa, dYa, Ya, dXa = S["X"][: self.t_ap], S["dY"][: self.t_ap], S["Y"][: self.t_ap], S["dX"][: self.t_ap]
                What = S["What"] if self.store_w_hat else None
                timed("fakequant_fwd/" + tag, lambda: e.qlinear_fakequant_fwd(S["d_ap"], Xa, L["W"], L["s"], L["z"], Ya, What))
                timed("fakequant_bwd/" + tag, lambda: e.qlinear_fakequant_bwd(S["d_ap"], Xa, dYa, L["W"], L["s"], L["z"], What,
                                                                                dXa, S["dW"], S["ds"], S["dz"], S["ws"]))
            if self.handoff:
                timed("quantize_pack/" + tag, lambda: e.eqat_quantize_pack(S["d_ap"], L["W"], L["s"], L["z"], L["P"], L["z8"], L["s16"]))
                timed("unpack/" + tag, lambda: e.eqat_unpack(S["d_ap"], L["P"], S["codes"]))
            if self.t_e2e:
                Xe, dYe, Ye, dXe = S["X"][: self.t_e2e], S["dY"][: self.t_e2e], S["Y"][: self.t_e2e], S["dX"][: self.t_e2e]
                timed("packed_fwd/" + tag, lambda: e.qlinear_packed_fwd(S["d_e2e"], Xe, L["P"], L["s16"], L["z8"], Ye))
                timed("packed_bwd_dx/" + tag, lambda: e.qlinear_packed_bwd_dx(S["d_e2e"], dYe, L["P"], L["s16"], L["z8"], dXe))
                timed("packed_bwd_ds/" + tag, lambda: e.qlinear_packed_bwd_ds(S["d_e2e"], Xe, dYe, L["P"], L["z8"], L["s16"], S["ds2"]))


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
    output rows.  Returns (flops counted the same way, seconds, description, seconds
    spent inside the five matrix products)."""
    from oracle import eqat_oracle as O
    from workloads import from_bf16_bits, get_config, normal_bf16
    rows, toks, in_f = 512, 256, 4096
    Wb = normal_bf16((rows, in_f), 0.02, "bench_oracle", seed, "W")
    Xb = normal_bf16((toks, in_f), 1.0, "bench_oracle", seed, "X")
    dYb = normal_bf16((toks, rows), 1e-2, "bench_oracle", seed, "dY")
    W, X, dY = from_bf16_bits(Wb), from_bf16_bits(Xb), from_bf16_bits(dYb)
    mm = [0.0]
    def product(fn, *a):
        t = time.perf_counter(); r = fn(*a); mm[0] += time.perf_counter() - t
        return r
    t0 = time.perf_counter()
    s, z = O.minmax_init(W, BITS, GROUP)
    What = O.fake_quant_weight(W, s, z, BITS, GROUP)
    Y = product(O.linear_fwd, X, What); dX = product(O.linear_bwd_dx, dY, What)
    G = product(O.weight_grad, dY, X)
    O.ste_bwd(G, W, s, z, BITS, GROUP)
    P, z8, s16 = O.quantize_pack(W, s, z, BITS, GROUP)
    q = O.unpack_rows(P, BITS, in_f)
    Wq = O.dequantize(q, s16.astype(np.float32), z8, GROUP)
    product(O.linear_fwd, X, Wq); product(O.linear_bwd_dx, dY, Wq)
    O.e2e_ds(dY, X, q, z8, GROUP)            # forms the weight gradient once more (a sixth product), then the group sums
    dt = time.perf_counter() - t0
    flops = 6 * 2 * toks * in_f * rows
    return flops, dt, f"4096-wide linear, {rows} output rows x {toks} tokens, all steps of the path (w2g64)", mm[0]


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_threads(matmul_share):
    """What the oracle really ran on: numpy hands its fp64 matrix products to the BLAS thread pool; everything else
    (Eq. 1-5 element by element, the group sums, the bit packing with its Python loop over rows) is one thread."""
    n = blas_threads()
    return {"cores": n,
            "threads": {"matrix products (BLAS pool)": n, "element-wise steps, group sums, bit packing": 1},
            "time_share_of_matrix_products": round(matmul_share, 3)}


def cpu_baseline(budget_s=15.0):
    flops, dt, what, mm = oracle_sample(0)
    reps, total_f, total_t, total_mm = 1, flops, dt, mm
    while total_t < budget_s and reps < 64:
        f, t, _, m = oracle_sample(reps)
        total_f += f; total_t += t; total_mm += m; reps += 1
    out = {"value": total_f / total_t / 1e12, "unit": "TFLOP/s", "kind": "oracle",
           "sample": f"{reps} x ({what}); {total_t:.1f} s of CPU time"}
    out.update(oracle_threads(total_mm / total_t))
    return out


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    times, flops, mm = [], 0, 0.0
    for i in range(args.warmup + args.steps):
        f, t, what, m = oracle_sample(i)
        if i >= args.warmup:
            times.append(t); flops = f; mm += m
    ms = 1e3 * sum(times) / len(times)
    val = flops / (ms * 1e-3) / 1e12
    base = {"value": val, "unit": "TFLOP/s", "kind": "oracle", "sample": what}
    base.update(oracle_threads(mm / sum(times)))
    out = {"impl": "reference", "metric": "QLinear fwd+bwd TFLOP/s", "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": WORKLOAD, "step": "bounded sample: " + what},
           "cpu_baseline": base,
           "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# ----------------------------------------------------------------------------- reporting
def summarise(timers):
    out = {}
    for name, pairs in timers.items():
        ms = [a.elapsed_time(b) for a, b in pairs]
        out[name] = {"launches": len(ms), "avg_ms": sum(ms) / len(ms), "total_ms": sum(ms)}
    return out


def tensor_roofline(achieved_tflops, peaks, region_s, sm_mhz):
    """A tensor-bound figure against every denominator there is.  `frac` uses the burst peak for a timed region of
    under two seconds (the GPU has not settled under its power cap yet, like the burst measurement) and the
    sustained one for a longer region; the other fractions are given beside it."""
    burst, sust = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    use_burst = region_s < 2.0
    peak = burst if use_burst else sust
    r = {"bound": "tensor", "achieved": achieved_tflops, "peak": peak, "unit": "TFLOP/s", "frac": achieved_tflops / peak,
         "peak_source": f"{peaks['source']} ({'burst' if use_burst else 'sustained'}; timed region {region_s:.2f} s)",
         "frac_vs_burst": achieved_tflops / burst, "frac_vs_sustained": achieved_tflops / sust,
         "frac_vs_nominal": achieved_tflops / NOMINAL_PEAKS["bf16_tflops"],
         "peaks": {"burst": burst, "sustained": sust, "nominal_dense_bf16": NOMINAL_PEAKS["bf16_tflops"]},
         "sm_mhz": {"this_run_median": sm_mhz,
                    "sustained_peak_measured_at": (peaks.get("clocks_under_load") or {}).get("sm_mhz_median")}}
    return r


def hbm_roofline(achieved_gbs, peaks):
    return {"bound": "hbm", "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (copy)",
            "frac_vs_nominal": achieved_gbs / NOMINAL_PEAKS["hbm_gbs"]}


def class_report(wl, timers, steps, peaks, region_s, sm_mhz):
    """Per call class: time per step, share, and the roofline figure of the class (contractions against the
    tensor peaks; the three one-kernel streaming calls of the hand-off against the copy bandwidth: those are
    per-call events around 10-50 us kernels inside the step, launch gaps included - the cold, back-to-back
    figures are in the streaming leg)."""
    kern = summarise(timers)
    by_class = {}
    for name, v in kern.items():
        c = name.split("/")[0]
        by_class[c] = by_class.get(c, 0.0) + v["total_ms"]
    total = sum(by_class.values())
    lin = LINEARS[wl.model]
    n_elem = sum(l.in_features * l.out_features * l.count for l in lin)
    n_grp = n_elem / wl.group
    hbm_bytes = {"minmax_init": 2 * n_elem + 8 * n_grp,
                 "quantize_pack": (2 + wl.bits / 8) * n_elem + 11 * n_grp,
                 "unpack": (1 + wl.bits / 8) * n_elem}
    classes = {}
    for c, t in by_class.items():
        sec = t * 1e-3 / steps
        classes[c] = {"total_ms_per_step": t / steps, "share": t / total, "kernels_per_call": KERNELS_PER_CALL[c]}
        if c in CONTRACTIONS:
            tok = wl.t_ap if c.startswith("fakequant") else wl.t_e2e
            fl = CONTRACTIONS[c] * 2 * tok * n_elem
            classes[c]["roofline"] = tensor_roofline(fl / sec / 1e12, peaks, region_s, sm_mhz)
        elif c in hbm_bytes:
            classes[c]["roofline"] = hbm_roofline(hbm_bytes[c] / sec / 1e9, peaks)
    return by_class, classes


def mode_figures(wl, by_class, steps, world=1):
    f_ap, f_e2e = wl.flops()
    ap_ms = sum(by_class.get(c, 0.0) for c in ("fakequant_fwd", "fakequant_bwd")) / steps
    qp_ms = sum(by_class.get(c, 0.0) for c in ("packed_fwd", "packed_bwd_dx", "packed_bwd_ds")) / steps
    tok, tf = {}, {}
    if wl.t_ap:
        tok["block_ap"] = world * wl.t_ap / (ap_ms * 1e-3); tf["block_ap"] = f_ap / (ap_ms * 1e-3) / 1e12
    if wl.t_e2e:
        tok["e2e_qp"] = world * wl.t_e2e / (qp_ms * 1e-3); tf["e2e_qp"] = f_e2e / (qp_ms * 1e-3) / 1e12
    return tok, tf


def time_steps(wl, steps, warmup):
    for _ in range(warmup):
        wl.step()
    torch.cuda.synchronize()
    timers = {}
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        wl.step(timers)
    t1.record()
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / steps, timers


def run_extra_config(eqat, device, name, spec, peaks):
    """One of the other workloads: the same path at its bit width, group size, model shapes and token counts."""
    wl = BlockWorkload(eqat, device, seed=20240711, t_block_ap=spec["t_ap"], t_e2e=spec["t_e2e"], model=spec["model"],
                       bits=spec["bits"], group=spec["group"], weight=spec["w"], handoff=False)
    sampler = ClockSampler(device.index or 0)
    sampler.start()
    import datetime
    t_begin = datetime.datetime.now()
    ms, timers = time_steps(wl, spec["steps"], 3)
    clocks = sampler.stop(t_begin, datetime.datetime.now())
    if eqat.device_status() != (0, 0):
        raise SystemExit(f"{name}: a kernel abandoned a wait")
    region_s = ms * spec["steps"] * 1e-3
    by_class, classes = class_report(wl, timers, spec["steps"], peaks, region_s, clocks["sm_mhz"])
    tok, tf = mode_figures(wl, by_class, spec["steps"])
    f_ap, f_e2e = wl.flops()
    top = max(by_class, key=by_class.get)
    out = {"workload": f"llama2-{spec['model']} decoder-block linears, w{spec['bits']}g{spec['group']}"
                       + (f", Block-AP fwd+bwd @{spec['t_ap']} tok" if spec["t_ap"] else "")
                       + (f", E2E-QP fwd/dX/ds @{spec['t_e2e']} tok" if spec["t_e2e"] else ""),
           "steps": spec["steps"], "warmup": 3, "ms_per_step": ms, "value": (f_ap + f_e2e) / (ms * 1e-3) / 1e12,
           "unit": "TFLOP/s", "tflops_by_mode": tf, "block_tokens_per_s": tok,
           "dominant": dict(kernel_class=top, **classes[top].get("roofline", {})),
           "kernel_classes": {c: {"ms_per_step": v["total_ms_per_step"], "share": v["share"],
                                  **({"achieved": v["roofline"]["achieved"], "unit": v["roofline"]["unit"],
                                      "frac_vs_burst": v["roofline"].get("frac_vs_burst"),
                                      "frac_vs_sustained": v["roofline"].get("frac_vs_sustained")} if "roofline" in v else {})}
                              for c, v in classes.items()},
           "per_shape_ms": {k: v["avg_ms"] for k, v in summarise(timers).items()},
           "clocks": clocks, "gpu_launches": wl.kernels_per_step * spec["steps"]}
    del wl
    torch.cuda.empty_cache()
    return out


def run_block_ap_forms(eqat, device, steps=10):
    """Block-AP forward + backward of the headline workload in its two forms, timed in the same process: W_hat
    written once by the streaming fake quantiser and read by the GEMMs (what the headline step uses), against
    W_hat never stored, each tile of W fake-quantised inside the forward and the dX GEMM."""
    out = {}
    f_ap = step_flops(T_BLOCK_AP, 0)[0]
    for name, stored in (("stored_w_hat", True), ("fake_quantised_in_the_gemm", False), ("stored_w_hat_again", True)):
        wl = BlockWorkload(eqat, device, seed=3, t_block_ap=T_BLOCK_AP, t_e2e=0, handoff=False, store_w_hat=stored)
        ms, timers = time_steps(wl, steps, 3)
        by = {}
        for k, v in summarise(timers).items():
            by[k.split("/")[0]] = by.get(k.split("/")[0], 0.0) + v["total_ms"] / steps
        out[name] = {"ms_per_step": ms, "tflops": f_ap / (ms * 1e-3) / 1e12, "fwd_ms": by["fakequant_fwd"], "bwd_ms": by["fakequant_bwd"]}
        del wl
        torch.cuda.empty_cache()
    out["tokens"] = T_BLOCK_AP
    out["used_by_the_headline_step"] = "stored_w_hat"
    return out


def run_block_driver(eqat, device, steps=10):
    """The headline block (without the hand-off) through the library's block-level entry points, one C call per
    phase and step, beside the same work as one call per linear and pass: same kernels, so the difference is what
    the host spends on crossing the boundary."""
    wl = BlockWorkload(eqat, device, seed=5, handoff=False)
    ap, e2e = [], []
    for L in wl.layers:
        S = wl.shapes[L["shape"]]
        ap.append(dict(desc=S["d_ap"], X=S["X"][: wl.t_ap], dY=S["dY"][: wl.t_ap], W=L["W"], s=L["s"], z=L["z"],
                       Y=S["Y"][: wl.t_ap], W_hat=S["What"], dX=S["dX"][: wl.t_ap], dW=S["dW"], ds=S["ds"], dz=S["dz"],
                       workspace=S["ws"]))
        e2e.append(dict(desc=S["d_e2e"], X=S["X"][: wl.t_e2e], dY=S["dY"][: wl.t_e2e], Wq_packed=L["P"], s16=L["s16"],
                        z=L["z8"], Y=S["Y"][: wl.t_e2e], dX=S["dX"][: wl.t_e2e], ds=S["ds2"], dz=None, workspace=None))

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / steps

    ms_layer = timed(lambda: wl.step())
    ms_block = timed(lambda: (eqat.eqat_block_ap_step(ap), eqat.eqat_e2e_qp_step(e2e)))
    f = sum(wl.flops())
    return {"calls": "eqat_block_ap_step + eqat_e2e_qp_step over the 7 linears", "ms_per_step": ms_block,
            "tflops": f / (ms_block * 1e-3) / 1e12, "per_linear_calls_ms_per_step": ms_layer,
            "per_linear_calls_tflops": f / (ms_layer * 1e-3) / 1e12}


def time_rotation(calls, rounds, windows=1):
    """Device time per launch (us) of `calls` issued in order, `rounds` times over: one pass is captured in a CUDA
    graph (so the host's launch cost is not in the figure) and replayed between a pair of events on its stream.
    With `windows` > 1 the measurement is repeated back to back and the median window is returned (a short window
    of a few milliseconds can fall into a transient of the GPU's clocks)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for c in calls:
            c()                                           # warm-up: one pass over every set, outside the capture
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for c in calls:
                c()
        graph.replay()
        side.synchronize()
        times = []
        for _ in range(windows):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(rounds):
                graph.replay()
            e1.record(side)
            side.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3 / (rounds * len(calls)))
    torch.cuda.current_stream().wait_stream(side)
    return statistics.median(times)


def run_streaming_leg(eqat, device, peaks, bits, group, shape=(11008, 4096), min_launches=56, min_bytes=640e6):
    """The five streaming kernels, each timed cold: `n` distinct sets of inputs and outputs whose combined size is
    several times the L2 (so no launch finds its operands or leaves its results in cache for the next one), at
    least `min_launches` launches back to back between one pair of events.  Bytes counted are the algorithmic
    ones (every input read once, every output written once)."""
    out_f, in_f = shape
    n_elem, ng = out_f * in_f, out_f * in_f // group
    d = eqat.make_desc(bits, group, out_f, in_f)
    bf = torch.bfloat16
    state_before = gpu_state(device.index or 0)
    g = torch.Generator(device=device); g.manual_seed(7)
    per = {"fakequant_weight": (4 + 8 / group) * n_elem, "ste_bwd": (6 + 16 / group) * n_elem,
           "minmax_init": (2 + 8 / group) * n_elem, "quantize_pack": (2 + bits / 8 + 11 / group) * n_elem,
           "unpack": (1 + bits / 8) * n_elem}
    res = {}
    for name, nbytes in per.items():
        n = max(4, int(np.ceil(min_bytes / nbytes)))
        sets = []
        for i in range(n):
            W = (torch.randn(out_f, in_f, generator=g, device=device, dtype=torch.float32) * 0.02).to(bf)
            S = dict(W=W, s=torch.empty(out_f, in_f // group, device=device), z=torch.empty(out_f, in_f // group, device=device))
            eqat.eqat_minmax_init(d, W, S["s"], S["z"])
            if name == "fakequant_weight":
                S["What"] = torch.empty_like(W)
                S["call"] = lambda S=S: eqat.eqat_fakequant_weight(d, S["W"], S["s"], S["z"], S["What"])
            elif name == "ste_bwd":
                S["G"] = (torch.randn(out_f, in_f, generator=g, device=device, dtype=torch.float32) * 1e-2).to(bf)
                S["dW"] = torch.empty_like(W); S["ds"] = torch.empty_like(S["s"]); S["dz"] = torch.empty_like(S["s"])
                S["call"] = lambda S=S: eqat.eqat_ste_bwd(d, S["G"], S["W"], S["s"], S["z"], S["dW"], S["ds"], S["dz"])
            elif name == "minmax_init":
                S["call"] = lambda S=S: eqat.eqat_minmax_init(d, S["W"], S["s"], S["z"])
            else:
                S["P"] = torch.empty(out_f, in_f * bits // 8, dtype=torch.uint8, device=device)
                S["z8"] = torch.empty(out_f, in_f // group, dtype=torch.uint8, device=device)
                S["s16"] = torch.empty(out_f, in_f // group, dtype=torch.float16, device=device)
                eqat.eqat_quantize_pack(d, W, S["s"], S["z"], S["P"], S["z8"], S["s16"])
                if name == "quantize_pack":
                    S["call"] = lambda S=S: eqat.eqat_quantize_pack(d, S["W"], S["s"], S["z"], S["P"], S["z8"], S["s16"])
                else:
                    S["codes"] = torch.empty(out_f, in_f, dtype=torch.uint8, device=device)
                    S["call"] = lambda S=S: eqat.eqat_unpack(d, S["P"], S["codes"])
                    del S["W"]
            sets.append(S)
        rounds = int(np.ceil(min_launches / n))
        us = time_rotation([S["call"] for S in sets], rounds, windows=3)
        launches = rounds * n
        r = hbm_roofline(nbytes / us / 1e3, peaks)
        r.update({"us_per_launch": us, "launches": launches, "distinct_buffer_sets": n,
                  "bytes_per_launch": nbytes, "bytes_touched_per_round": n * nbytes})
        res[name] = r
        del sets
        torch.cuda.empty_cache()
    # yardstick: a device-to-device copy of the same weight (read 2 bytes, write 2 bytes per element), timed the same
    # way on the same GPU in the same state; what a kernel with no arithmetic at all reaches at this size
    n = max(4, int(np.ceil(min_bytes / (4 * n_elem))))
    src = [torch.empty(out_f, in_f, dtype=bf, device=device).normal_(generator=g) for _ in range(n)]
    dst = [torch.empty_like(t) for t in src]
    rounds = int(np.ceil(min_launches / n))
    us = time_rotation([lambda a=a, b=b: b.copy_(a) for a, b in zip(src, dst)], rounds, windows=3)
    yard = hbm_roofline(4 * n_elem / us / 1e3, peaks)
    yard.update({"us_per_launch": us, "launches": rounds * n, "distinct_buffer_sets": n, "bytes_per_launch": 4.0 * n_elem,
                 "what": "torch copy_ of one weight-sized bf16 tensor (not a kernel of this library)"})
    for r in res.values():
        r["frac_of_same_size_copy"] = r["achieved"] / yard["achieved"]
    del src, dst
    torch.cuda.empty_cache()
    return {"shape": f"{out_f} x {in_f}", "bits": bits, "group": group,
            "method": "distinct input/output sets per launch (combined > 4 x L2); the launches of one pass over the sets are "
                      "captured in a CUDA graph and the graph is replayed back to back between one pair of CUDA events; "
                      "median of three such windows",
            "kernels": res, "copy_yardstick": yard,
            "gpu_state": {"before": state_before, "after": gpu_state(device.index or 0)}}


# ----------------------------------------------------------------------------- main
def spawn_ranks(args):
    """`--gpus N` without a launcher: start N copies of this script, one per GPU, with the environment
    torch.distributed's launcher would have given them; rank 0's line is the job's line."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    rc = 0
    for pr in procs:
        rc = max(rc, abs(pr.wait()))
    return rc


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
    warmup = max(args.warmup, 3)

    # The streaming kernels are timed twice: here, before the GEMM phases have heated the GPU (a kernel timed alone),
    # and again after them.  They are bound by instruction issue as much as by memory, so they follow the SM clock,
    # which stays low for seconds after a phase at the power cap.
    extras = rank == 0 and world == 1 and not args.headline_only
    streaming_first = run_streaming_leg(eqat, device, peaks, BITS, GROUP) if extras else None

    import datetime
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    wl = BlockWorkload(eqat, device, seed=20240711 + rank)     # each rank: its own token batch (weak scaling)
    for _ in range(warmup):
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
    e2e_steps = max(1, args.steps)
    stage.step(); torch.cuda.synchronize(); barrier()
    t0.record()
    for _ in range(e2e_steps):
        stage.step()
    t1.record()
    torch.cuda.synchronize(); barrier()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1) / e2e_steps, device)
    wl_h2d, wl_d2h = stage.h2d, stage.d2h
    del stage

    f_ap, f_e2e = wl.flops()
    flops = (f_ap + f_e2e) * world
    if rank == 0:
        region_s = ms * args.steps * 1e-3
        by_class, classes = class_report(wl, timers, args.steps, peaks, region_s, clocks["sm_mhz"])
        top_class = max(by_class, key=by_class.get)
        roof = None
        if top_class in CONTRACTIONS:
            roof = dict(kernel="gemm_kernel (" + top_class + ")", **classes[top_class]["roofline"])
            roof["traffic"] = traffic_per_launch(top_class)
            roof["traffic_unit"] = "DRAM bytes per launch (ncu, launch-weighted mean over the class)"
            lin = LINEARS["7b"]
            roof["algorithmic_bytes"] = sum((T_E2E * (l.in_features + l.out_features) * 2
                                             + l.in_features * l.out_features * BITS // 8) * l.count for l in lin) / sum(l.count for l in lin)
        for c in ("packed_fwd", "packed_bwd_dx", "packed_bwd_ds"):
            if c in classes:
                classes[c]["roofline"]["traffic"] = traffic_per_launch(c)
        tok, tf = mode_figures(wl, by_class, args.steps, world)
        value = flops / (ms * 1e-3) / 1e12
        out = {"metric": "QLinear fwd+bwd TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": world,
               "steps": args.steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": {"workload": WORKLOAD, "bits": BITS, "group": GROUP, "tokens_block_ap": T_BLOCK_AP, "tokens_e2e_qp": T_E2E,
                          "l2": "inputs larger than L2 (working set > 2 GB per shape, weights per linear)"},
               "pct_of_bf16_peak": {"vs_burst": 100.0 * value / world / peaks["bf16_tflops"],
                                    "vs_sustained": 100.0 * value / world / peaks["bf16_tflops_sustained"],
                                    "vs_nominal_dense": 100.0 * value / world / NOMINAL_PEAKS["bf16_tflops"]},
               "block_tokens_per_s": tok, "tflops_by_mode": tf,
               "roofline": roof, "kernel_classes": classes, "clocks": clocks,
               "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms, "steps": e2e_steps,
                       "h2d_bytes_per_step": wl_h2d, "d2h_bytes_per_step": wl_d2h},
               "gpu_launches": wl.kernels_per_step * args.steps}
    del wl
    torch.cuda.empty_cache()
    if rank == 0:
        if world == 1 and not args.headline_only:
            # the other workloads and the cold streaming figures (one GPU is enough for them: the path is replicated)
            out["configs"] = {name: run_extra_config(eqat, device, name, spec, peaks) for name, spec in EXTRA_CONFIGS.items()}
            out["block_ap_forms"] = run_block_ap_forms(eqat, device)
            out["few_tokens"] = decode_leg(eqat, device, peaks, 10)
            out["few_tokens_w4g128"] = decode_leg(eqat, device, peaks, 10, bits=4, group=128, tokens=(1, 8))
            out["block_driver"] = run_block_driver(eqat, device)
            streaming_first["when"] = "before the GEMM phases of this run"
            out["streaming"] = {"w2g64": streaming_first,
                                "w2g64_after_gemm_phases": run_streaming_leg(eqat, device, peaks, 2, 64),
                                "w4g128_after_gemm_phases": run_streaming_leg(eqat, device, peaks, 4, 128)}
            alias = {"fakequant_weight": "fakequant_weight", "ste_bwd": "ste_bwd", "minmax_init": "minmax_init_cold",
                     "quantize_pack": "quantize_pack_cold", "unpack": "unpack_cold"}
            for k, v in out["streaming"]["w2g64"]["kernels"].items():
                out["kernel_classes"][alias[k]] = {"roofline": v, "timed": "streaming leg (cold data, back to back, before the "
                                                    "GEMM phases of this run), not part of the step"}
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline()
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_kernel_case(args):
    """One linear shape of one workload, a few steps: the small case used for ncu captures."""
    torch.cuda.set_device(0)
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding as eqat
    mode = args.case_mode
    wl = BlockWorkload(eqat, torch.device("cuda", 0), seed=1, model=args.case_model, bits=args.case_bits, group=args.case_group,
                       t_block_ap=args.case_tokens if mode in ("both", "block_ap") else 0,
                       t_e2e=args.case_tokens if mode in ("both", "e2e_qp") else 0, handoff=(mode == "both"),
                       store_w_hat=not args.case_no_w_hat)
    wl.layers = [L for L in wl.layers if L["shape"] == args.case_shape][:1]
    assert wl.layers, f"no linear named {args.case_shape} in model {args.case_model}"
    for _ in range(2):
        wl.step()
    torch.cuda.synchronize()
    timers = {}
    for _ in range(args.case_iters):
        wl.step(timers)
    torch.cuda.synchronize()
    assert eqat.device_status() == (0, 0)
    print(json.dumps({k: v for k, v in summarise(timers).items()}), flush=True)


def run_streaming_case(args):
    """The cold streaming leg alone (for profiler captures and kernel work)."""
    torch.cuda.set_device(0)
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding as eqat
    lin = next(l for l in LINEARS[args.case_model] if l.name == args.case_shape)
    r = run_streaming_leg(eqat, torch.device("cuda", 0), load_peaks(), args.case_bits, args.case_group,
                          (lin.out_features, lin.in_features), min_launches=args.case_iters * 4, min_bytes=640e6)
    assert eqat.device_status() == (0, 0)
    print(json.dumps(r), flush=True)


def decode_leg(eqat, dev, peaks, iters, model="7b", bits=BITS, group=GROUP, only_shape=None, tokens=(1, 4, 8, 16),
               fp16_zero_points=False):
    """Few-token packed forward (the matrix-vector kernels) on the linear shapes of one block: device time per
    launch from a CUDA graph of launches over rotating weight copies (more than L2 in total), and the bandwidth that
    time means for the bytes one launch must read."""
    out = {"metric": "packed forward, few tokens", "unit": "us per call", "bits": bits, "group": group,
           "zero_points": "fp16" if fp16_zero_points else "uint8", "model": model, "hbm_gbs_peak": peaks["hbm_gbs"],
           "method": "CUDA graph of one call per weight copy (copies total > 2 x L2), replayed back to back; a call "
                     "is one kernel launch for up to 8 tokens where the staged activations fit, else one per token slice",
           "cases": {}}
    for lin in LINEARS[model]:
        if only_shape is not None and lin.name != only_shape:
            continue
        o, i = lin.out_features, lin.in_features
        ng = i // group
        wbytes = o * i * bits // 8
        copies = max(4, int(320e6 // wbytes))
        Ps = [torch.randint(0, 256, (o, i * bits // 8), dtype=torch.uint8, device=dev) for _ in range(copies)]
        if fp16_zero_points:
            z8 = (torch.rand(o, ng, device=dev) * ((1 << bits) - 1)).half()
        else:
            z8 = torch.randint(0, 1 << bits, (o, ng), dtype=torch.uint8, device=dev)
        s16 = (torch.rand(o, ng, device=dev) * 0.01 + 0.001).half()
        for T in tokens:
            X = torch.randn(T, i, device=dev).to(torch.bfloat16)
            Y = torch.empty(T, o, dtype=torch.bfloat16, device=dev)
            d = eqat.make_desc(bits, group, o, i, T, 0, eqat.EQAT_ZP_FP16 if fp16_zero_points else eqat.EQAT_ZP_U8)
            us = time_rotation([lambda P=P: eqat.qlinear_packed_fwd(d, X, P, s16, z8, Y) for P in Ps], iters)
            nbytes = wbytes + o * ng * (4 if fp16_zero_points else 3) + T * (i + o) * 2
            out["cases"][f"{lin.name}/T{T}"] = {"us": us, "bytes": nbytes, "gbs": nbytes / us / 1e3,
                                                 "frac_of_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}
        del Ps
        torch.cuda.empty_cache()
    return out


def run_decode_case(args):
    """The few-token forward leg alone (for profiler captures and kernel work)."""
    torch.cuda.set_device(0)
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding as eqat
    out = decode_leg(eqat, torch.device("cuda", 0), load_peaks(), args.case_iters, args.case_model, args.case_bits,
                     args.case_group, args.decode_shape, tuple(int(t) for t in args.decode_tokens.split(",")),
                     args.decode_fp16_zero_points)
    assert eqat.device_status() == (0, 0)
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel-case", action="store_true", help="run one linear shape a few times (for profilers)")
    ap.add_argument("--decode-case", action="store_true",
                    help="time the few-token packed forward on the linear shapes of --case-model (uses --case-iters)")
    ap.add_argument("--decode-shape", default=None, help="decode case: only this linear of the block (e.g. gate_up)")
    ap.add_argument("--decode-tokens", default="1,4,8,16", help="decode case: token counts, comma separated")
    ap.add_argument("--decode-fp16-zero-points", action="store_true", help="decode case: zero points as fp16 values")
    ap.add_argument("--streaming-case", action="store_true", help="the cold streaming-kernel leg alone")
    ap.add_argument("--case-model", default="7b", choices=sorted(LINEARS))
    ap.add_argument("--case-shape", default="qkvo")
    ap.add_argument("--case-tokens", type=int, default=16384)
    ap.add_argument("--case-bits", type=int, default=BITS)
    ap.add_argument("--case-group", type=int, default=GROUP)
    ap.add_argument("--case-mode", default="both", choices=["both", "block_ap", "e2e_qp"])
    ap.add_argument("--case-iters", type=int, default=2)
    ap.add_argument("--case-no-w-hat", action="store_true",
                    help="kernel case: Block-AP without a stored W_hat (Eq. 1-2 inside the forward and dX GEMMs)")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the other workloads and the streaming leg")
    args = ap.parse_args()
    if args.kernel_case:
        run_kernel_case(args)
    elif args.decode_case:
        run_decode_case(args)
    elif args.streaming_case:
        run_streaming_case(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
