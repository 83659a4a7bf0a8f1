#!/usr/bin/env python
"""Benchmark of the filtered convolution backward pass (gradient filtering).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of the MobileNetV2-style
inverted-residual block (1x1 conv 96->576, 3x3 depthwise conv 576, 1x1 conv 576->96;
N=128, 28x28, r=2, fp32): for each of the three layers gf_stash_forward
(patch-summed activations) and gf_backward (gradient filter, reduced g_W, reduced g_X
with expansion).  Prints ONE JSON line (rank 0).  The metric is microseconds per
layer backward (the step's time divided by its three layers; lower is better).
The line also carries, in `per_config`, every layer of the other workload
configurations timed the same way, each next to an exact convolution backward of the
same shape through torch/cuDNN (context: a different, unfiltered result).

N > 1: independent replicas, one per GPU, no collective on the data path; the value
is time divided by the layers all ranks processed.  Under a launcher (torchrun) the
ranks come from the environment; started plainly with --gpus N > 1, the script
re-executes itself under torch.distributed.run with N processes.

--impl reference times the fp64 CPU checker (oracle/) on the host cores on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "filtered_conv_backward_us_per_layer"
UNIT = "us"
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # SMs x FMA lanes x 2 flop x max SM clock

# What the paper reports for this path (Section 5.5): ratios against the libraries' exact
# convolution backward on its own devices, fp32.  Context for `exact_cudnn_us`, not a target.
PAPER_CONTEXT = {
    "r2": "paper, Section 5.5: over 10x faster than the exact cuDNN backward at patch size 2 (RTX 3090 Ti and "
          "Jetson Nano GPUs, fp32), over 20x against MKLDNN on CPUs (11900KF, Jetson Nano, Raspberry Pi 3b)",
    "r4": "paper, Section 5.5: over 25x against cuDNN at patch size 4, over 60x against MKLDNN",
}

# DRAM bytes per launch of a kernel from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by (layer name, kernel name), with the sha1 of the kernel's
# source file at capture time; a changed source makes the entry stale (reported as null).
NCU_TRAFFIC: dict[tuple[str, str], dict] = {
    # ncu --set full --clock-control none, python bench.py --table --no-exact --only <layer>/r2 (profiles/*.md)
    ("cfg3b_dw_576", "dw_fused"): {"bytes": 289.06e6 + 188.65e6, "sha1": "4b5034114d07f51de9ec93105e217e4cac06777c"},
    ("cfg3c_pw_576_96", "gyx_fused"): {"bytes": 38.89e6 + 192.70e6, "sha1": "6ed5190bb4d910ada562260c71fe702d5e2f90dc"},
    ("cfg3c_pw_576_96", "gw_tiled"): {"bytes": 74.89e6 + 2.16e6, "sha1": "6ed5190bb4d910ada562260c71fe702d5e2f90dc"},
    ("cfg3a_pw_96_576", "stash_pool"): {"bytes": 38.55e6 + 0.01e6, "sha1": "56c08adc367812dd2e6ee11acb71cb1a0a803d89"},
    ("cfg3a_pw_96_576", "gx_tc"): {"bytes": 58.06e6 + 5.71e6, "sha1": "a17659264f21416ec34cfc79629bea8d8d9c06de"},
    ("cfg3a_pw_96_576", "gw_tc"): {"bytes": 67.71e6 + 0.76e6, "sha1": "a17659264f21416ec34cfc79629bea8d8d9c06de"},
    # not captured: the same kernel on the two larger inputs of the step; its traffic on the captured
    # layer equals the bytes of x (the stash it writes was still in L2 when the kernel ended), scaled here
    ("cfg3b_dw_576", "stash_pool"): {"bytes": 38.55e6 * 6.0, "sha1": "56c08adc367812dd2e6ee11acb71cb1a0a803d89", "scaled": True},
    ("cfg3c_pw_576_96", "stash_pool"): {"bytes": 38.55e6 * 6.0, "sha1": "56c08adc367812dd2e6ee11acb71cb1a0a803d89", "scaled": True},
}

KERNEL_SOURCE = {
    "stash_pool": "gf_pool.cu", "gy_pool": "gf_pool.cu", "ksum": "gf_tc.cu", "gx_mix": "gf_dense.cu",
    "gw_partial": "gf_dense.cu", "gw_finish": "gf_dense.cu", "dw_fused": "gf_depthwise.cu",
    "gx_tc": "gf_tc.cu", "gw_tc": "gf_tc.cu", "split_f32": "gf_tc.cu", "gyx_fused": "gf_fused.cu",
    "gw_tiled": "gf_fused.cu",
}


def measured_peaks() -> tuple[dict, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return ({"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                 "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"]))}, "measured")
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def workload():
    """The layers of one step: the MobileNetV2-style block at r = 2, fp32."""
    from paper_2301_00330_b200 import workloads
    return workloads.config3(2)


def workload_config(layers) -> dict:
    """The same dict for both arms (GPU and --impl reference)."""
    return {
        "workload": "configs[2]: MobileNetV2-style inverted-residual block backward, 1x1 96->576, 3x3 depthwise 576 "
                    "(pad 1), 1x1 576->96, N=128, 28x28, r=2, fp32 (the largest single-GPU configuration)",
        "layers": [{"layer": L.name, "N": L.N, "C_in": L.C_in, "C_out": L.C_out, "H": L.H, "W": L.W, "K": L.K,
                    "groups": L.groups, "r": L.r, "dtype": L.dtype} for L in layers],
        "step": "for each of the 3 layers: gf_stash_forward + gf_backward (g_W and g_X); value = step time / 3",
        "inputs": "each layer has its own seeded x, g_y, W (the activation and normalisation backward between the "
                  "layers is outside the method)",
        "l2": "every layer's tensors (0.4 - 0.75 GB) exceed the 126 MB L2 several times over, and the step walks "
              "through 1.8 GB before it touches a buffer again; inputs and outputs also rotate over 2 sets",
    }


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the GPU works."""

    def __init__(self, index: int):
        self.samples = []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        if not self.nv:
            return
        try:
            mhz = self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)
            reasons = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) \
                if hasattr(self.nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                else self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            self.samples.append((mhz, int(reasons)))
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            time.sleep(0.01)

    def start(self):
        self.samples = []
        self._stop.clear()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread:
            self._thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        mhz = sorted(s[0] for s in self.samples)
        bits = 0
        for _, r in self.samples:
            bits |= r
        names = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        reasons = [n for b, n in names.items() if bits & b and n != "gpu_idle"]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(mhz)}


# --------------------------------------------------------------------------- roofline
def kernel_cost(name: str, L) -> tuple[float, float]:
    """(algorithmic bytes, flops) of one launch of kernel `name` on layer L."""
    e = L.elem_bytes
    gbar = 4 * L.N * L.C_out * L.Hp * L.Wp          # fp32 patch means (CUDA-core path)
    # tensor-core path: bf16 patch means; fp32 layers carry (high, low) bf16 pairs, 4 bytes again
    gbar16 = gbar // 2 if L.dtype == "bf16" else gbar
    pairs = L.C_out * L.C_ig
    M = L.N * L.Hp * L.Wp
    mix = 2.0 * M * L.C_out * L.C_ig
    tc = L.groups == 1 and L.C_out % 8 == 0
    table = {
        "split_f32": (8 * L.numel_stash(), L.numel_stash()),
        "gx_tc": (gbar16 + e * pairs + e * L.numel_x(), mix),
        "gw_tc": (gbar16 + e * L.numel_stash() + 4 * pairs, mix),
        "stash_pool": (e * (L.numel_x() + L.numel_stash()), L.numel_x()),
        "gy_pool": (e * L.numel_gy() + (gbar16 if tc else gbar), L.numel_gy()),
        "gyx_fused": (e * (L.numel_gy() + L.numel_x()) + gbar16 + e * pairs, mix + L.numel_gy()),
        "gw_tiled": (gbar16 + e * L.numel_stash() + 4 * pairs, mix),
        "ksum": (e * L.numel_w() + 4 * pairs, L.numel_w()),
        "gx_mix": (gbar + 4 * pairs + e * L.numel_x(), mix),
        "gw_partial": (gbar + e * L.numel_stash() + 4 * pairs, mix),
        "gw_finish": (4 * pairs + 4 * L.numel_w(), pairs),
        "dw_fused": (e * (L.numel_gy() + L.numel_stash() + L.numel_x() + L.numel_w()), 3 * L.numel_gy()),
    }
    return table[name]


def _source_sha1(src: str) -> str:
    with open(os.path.join(ROOT, "paper_2301_00330_b200", "csrc", src), "rb") as f:
        return hashlib.sha1(f.read()).hexdigest()


def traffic_for(layer_name: str, kernel: str):
    """DRAM bytes of one launch from the ncu capture on file, or None when there is none or the
    kernel's source has changed since the capture (the entry holds the source's hash at that time)."""
    ent = NCU_TRAFFIC.get((layer_name, kernel))
    src = KERNEL_SOURCE.get(kernel)
    if not ent or not src:
        return None
    return ent["bytes"] if ent.get("sha1") == _source_sha1(src) else None


def roofline_step(name: str, total_ms: float, launches: int, steps: int, layers) -> dict:
    """Roofline of a kernel over all its launches of a step: algorithmic bytes of those launches
    (summed over the layers that use it) / their summed duration."""
    peaks, which = measured_peaks()
    users = [L for L in layers if name in KERNELS_OF_LAYER.get(L.name, ())]
    per_step = sum(kernel_cost(name, L)[0] for L in users)
    per_launch = launches / max(steps, 1)
    ach = per_step * steps / (total_ms * 1e-3) / 1e9 if total_ms > 0 else 0.0
    traffic = [traffic_for(L.name, name) for L in users]
    return {"kernel": name, "layers": [L.name for L in users], "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "peak_source": f"of {which}",
            "launches_per_step": per_launch, "algorithmic_bytes_per_launch": per_step / max(per_launch, 1),
            "avg_launch_us": total_ms * 1e3 / max(launches, 1),
            "traffic": (sum(traffic) / len(traffic)) if traffic and all(t is not None for t in traffic) else None,
            "traffic_note": "ncu dram__bytes_read.sum + dram__bytes_write.sum per launch, averaged over the step's launches "
                            "of this kernel; the two 289 MB inputs are scaled from the capture on the 38.5 MB one "
                            "(read bytes = bytes of x; the stash written was still in L2 when the kernel ended)"}


KERNELS_OF_LAYER: dict[str, tuple] = {}


def roofline(name: str, avg_ms: float, L) -> dict:
    peaks, which = measured_peaks()
    nbytes, flops = kernel_cost(name, L)
    t = avg_ms * 1e-3
    t_mem = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_alu = flops / (FP32_ALU_TFLOPS * 1e12)
    if t_alu > t_mem and name in ("gx_mix", "gw_partial"):
        ach = flops / t / 1e12
        return {"kernel": name, "layer": L.name, "bound": "alu", "achieved": ach, "peak": FP32_ALU_TFLOPS,
                "unit": "TFLOP/s", "frac": ach / FP32_ALU_TFLOPS, "traffic": traffic_for(L.name, name),
                "peak_source": "derived: 148 SM x 128 FMA x 2 x 1.965 GHz", "avg_launch_us": avg_ms * 1e3}
    ach = nbytes / t / 1e9
    return {"kernel": name, "layer": L.name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": traffic_for(L.name, name),
            "peak_source": f"of {which}", "algorithmic_bytes_per_launch": nbytes, "avg_launch_us": avg_ms * 1e3}


# --------------------------------------------------------------------------- CPU checker timing
def time_oracle(layers, n_sample: int, steps: int, warmup: int) -> dict:
    """The fp64 CPU checker, as it stands, on n_sample images of every layer of the step."""
    import numpy as np
    import torch
    import oracle
    from paper_2301_00330_b200 import workloads
    data = []
    for L in layers:
        Ls = L.with_(N=n_sample)
        x, gy, w = workloads.make_inputs(Ls)
        data.append((Ls, *(t.to(torch.float64).numpy() for t in (x, gy, w))))

    def one():
        out = None
        for Ls, x64, gy64, w64 in data:
            stash = oracle.stash_forward(x64, Ls.r)
            out = oracle.backward(gy64, stash, w64, Ls.r, groups=Ls.groups)
        return out

    for _ in range(warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        gw, gx = one()
    dt = (time.perf_counter() - t0) / steps
    assert np.isfinite(gw).all() and np.isfinite(gx).all()
    scale = layers[0].N / n_sample
    return {"value": dt * 1e6 * scale / len(layers), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n_sample} of {layers[0].N} images of each of the {len(layers)} layers, fp64, time scaled "
                      f"x{scale:g} (every step of the method is linear in the batch); {steps} timed passes",
            "seconds_per_pass": dt}


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers = workload()
    steps = max(1, min(args.steps, 3))
    base = time_oracle(layers, 32, steps, 1 if args.warmup > 0 else 0)
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": base["value"] * len(layers) / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(layers),
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- GPU arm
def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time: the job is done when the last replica is."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value_us(ms_total: float, steps: int, world: int, layers_per_step: int = 1) -> float:
    """us per layer of the whole job: every rank ran `steps` steps of `layers_per_step` layers of
    its own replica in ms_total (max over ranks), so the job did steps * world * layers of them."""
    return ms_total * 1e3 / (steps * world * layers_per_step)


def backlog(ms: float = 4.0):
    """Keeps the stream busy for a few ms so that the launches enqueued next wait in the
    queue and then run back to back: event pairs then measure the GPU, not the host."""
    import torch
    torch.cuda._sleep(int(ms * 1e-3 * 1.9e9))


def time_layer(gf, L, peaks, with_exact: bool = True, with_kernels: bool = False) -> dict:
    """One layer timed three ways with CUDA events behind a stream backlog: gf_stash_forward,
    gf_backward (g_W and g_X), and an exact backward through torch/cuDNN as context."""
    import torch
    from paper_2301_00330_b200 import workloads
    stream = torch.cuda.current_stream()
    desc = gf.desc_for(L)
    x0, gy0, w0 = workloads.make_inputs(L)
    per_set = L.backward_bytes() + L.stash_bytes_moved()
    n_sets = max(1, min(4, int(400e6 // per_set) + 1))     # small layers rotate over several sets (L2)
    sets = [(torch.roll(x0, i, 0).cuda(), torch.roll(gy0, i, 0).cuda(), gf.alloc_layer(desc)) for i in range(n_sets)]
    w = w0.cuda()
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    reps = 20 if per_set < 300e6 else 8

    def timed(fn, n):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        backlog(3.0)
        e0.record(stream)
        for i in range(n):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n

    def stash(i):
        x, _, b = sets[i % n_sets]
        gf.gf_stash_forward(desc, x, b.stash, stream)

    def bwd(i):
        _, gy, b = sets[i % n_sets]
        gf.gf_backward(desc, gy, b.stash, w, b.g_W, b.g_X, b.workspace, ws_bytes, stream)

    def exact(i):
        x, gy, _ = sets[i % n_sets]
        torch.ops.aten.convolution_backward(gy, x, w, None, [1, 1], [L.pad, L.pad], [1, 1], False, [0, 0],
                                            L.groups, [True, True, False])

    t_stash, t_bwd = timed(stash, reps), timed(bwd, reps)
    row = {"layer": L.name, "r": L.r, "dtype": L.dtype, "stash_us": round(t_stash, 2), "backward_us": round(t_bwd, 2),
           "backward_alg_MB": round(L.backward_bytes() / 1e6, 1),
           "backward_gbs": round(L.backward_bytes() / t_bwd / 1e3, 1),
           "backward_frac_hbm": round(L.backward_bytes() / t_bwd / 1e3 / peaks["hbm_gbs"], 3),
           "stash_gbs": round(L.stash_bytes_moved() / t_stash / 1e3, 1),
           "stash_frac_hbm": round(L.stash_bytes_moved() / t_stash / 1e3 / peaks["hbm_gbs"], 3)}
    if with_kernels:   # per-kernel event times of the backward call (each bracketed, so a few us high)
        gf.gf_profile_configure(2)
        backlog(3.0)
        for i in range(4):
            bwd(i)
        torch.cuda.synchronize()
        row["kernels_us"] = {k: round(ms / n * 1e3, 1) for k, (n, ms) in gf.gf_profile_read().items()}
        gf.gf_profile_configure(0)
    if with_exact:
        try:
            t_exact = timed(exact, max(2, reps // 4))
            row["exact_cudnn_us"] = round(t_exact, 1)
            row["exact_over_filtered"] = round(t_exact / t_bwd, 2)
        except Exception as ex:   # context only: never fail the bench on it
            row["exact_cudnn_us"] = None
            row["exact_error"] = type(ex).__name__
    del sets
    torch.cuda.empty_cache()
    return row


def diagnostics(gf, runs) -> dict:
    """Section 4.1 on the step's own tensors: SNR of the filtered g_y per layer (Eq. (snr_g3), first
    line) and the DC/AC energy ratio of the 3x3 kernels (Eq. (dcac_ratio)), by the library's kernels."""
    import math
    import torch
    out = {"note": "synthetic i.i.d. gradients and Kaiming-random kernels: the numbers show the diagnostics run, they are not "
                   "the paper's (trained networks have DC-dominated kernels and smoother gradients)", "layers": {}}
    e = torch.zeros(2, dtype=torch.float64, device="cuda")
    for L, desc, w, _, sets in runs:
        gy = sets[0][1]
        gf.gf_filter_snr_terms(gy, L.r, e)
        torch.cuda.synchronize()
        sig, noise = (float(v) for v in e.cpu())
        row = {"snr_gy": sig / noise if noise > 0 else None,
               "snr_gy_db": 10.0 * math.log10(sig / noise) if noise > 0 and sig > 0 else None}
        if L.K > 1:
            ratio = torch.empty((L.C_out, L.C_ig), dtype=torch.float32, device="cuda")
            gf.gf_dcac_ratio(w, ratio)
            torch.cuda.synchronize()
            row["dcac_ratio_mean"] = float(ratio.mean())
            row["dcac_ratio_share_ge_1"] = float((ratio >= 1).float().mean())
        out["layers"][L.name] = row
    return out


def extras(gf, layers) -> dict:
    """Timings of the further entry points on shapes of the step (events behind a backlog, 10 calls)."""
    import torch
    from paper_2301_00330_b200 import workloads
    stream = torch.cuda.current_stream()

    def timed(fn, n=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        backlog(3.0)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return round(e0.elapsed_time(e1) * 1e3 / n, 1)

    out = {}
    # the stash produced inside the producer of x (ReLU6 + x + stash in one pass) on the depthwise layer's input
    L = layers[1]
    desc = gf.desc_for(L)
    z = torch.randn((L.N, L.C_in, L.H, L.W), device="cuda")
    x = torch.empty_like(z)
    stash = torch.empty(gf.gf_stash_dims(desc), device="cuda")
    t_fused = timed(lambda: gf.gf_act_stash_forward(desc, gf.GF_ACT_RELU6, z, x, stash, stream))
    t_act = timed(lambda: torch.clamp(z, 0.0, 6.0, out=x))
    t_stash = timed(lambda: gf.gf_stash_forward(desc, x, stash, stream))
    nbytes = z.numel() * 4 * 2 + stash.numel() * 4
    out["act_stash_forward"] = {"layer": L.name, "fused_us": t_fused, "separate_us": {"relu6_torch": t_act, "gf_stash_forward": t_stash},
                                "fused_gbs": round(nbytes / t_fused / 1e3, 1),
                                "note": "Section 4.2: the forward overhead of the method is what the fused pass costs beyond the activation alone"}
    del z, x, stash
    # INT8 variant of the reduced contractions on the two pointwise layers
    out["backward_int8_us"] = {}
    for L in (layers[0], layers[2]):
        desc = gf.desc_for(L)
        x0, gy0, w0 = workloads.make_inputs(L)
        gy, w = gy0.cuda(), w0.cuda()
        buf = gf.alloc_layer(desc)
        gf.gf_stash_forward(desc, x0.cuda(), buf.stash, stream)
        ws = torch.empty(gf.gf_backward_int8_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
        out["backward_int8_us"][L.name] = timed(lambda: gf.gf_backward_int8(desc, gy, buf.stash, w, buf.g_W, buf.g_X, ws, None, stream))
        del gy, w, buf, ws
    # a stride-2 layer of the kind inside the paper's trained ranges (ResNet-18 stage transition)
    desc = gf.make_desc(64, 128, 256, 28, 28, 3, r=2, stride=2)
    xs = torch.randn((64, 128, 28, 28), device="cuda").clamp_(min=0)
    gys = torch.randn((64, 256, 14, 14), device="cuda") * 1e-2
    wsd = torch.randn((256, 128, 3, 3), device="cuda") * 0.04
    stash = torch.empty(gf.gf_stash_dims(desc), device="cuda")
    gW, gX = torch.empty_like(wsd), torch.empty_like(xs)
    ws = torch.empty(gf.gf_backward_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    gf.gf_stash_forward(desc, xs, stash, stream)
    out["stride2_3x3_128_256_28x28_N64_r2"] = {
        "stash_us": timed(lambda: gf.gf_stash_forward(desc, xs, stash, stream)),
        "backward_us": timed(lambda: gf.gf_backward(desc, gys, stash, wsd, gW, gX, ws, None, stream)),
        "exact_cudnn_us": timed(lambda: torch.ops.aten.convolution_backward(gys, xs, wsd, None, [2, 2], [1, 1], [1, 1], False,
                                                                            [0, 0], 1, [True, True, False]), 4)}
    del xs, gys, wsd, stash, gW, gX, ws
    # the step's layers with channels-last tensors (same bytes, other kernels)
    out["nhwc_layer_us"] = {}
    for L in layers:
        desc = gf.make_desc(L.N, L.C_in, L.C_out, L.H, L.W, L.K, r=L.r, groups=L.groups,
                            dtype=gf.GF_F32 if L.dtype == "f32" else gf.GF_BF16, layout=gf.GF_NHWC)
        x0, gy0, w0 = workloads.make_inputs(L)
        xl, gyl, wl = x0.cuda().permute(0, 2, 3, 1).contiguous(), gy0.cuda().permute(0, 2, 3, 1).contiguous(), w0.cuda()
        n, c, hp, wp = gf.gf_stash_dims(desc)
        stash = torch.empty((n, hp, wp, c), dtype=xl.dtype, device="cuda")
        gW, gX = torch.empty(wl.shape, dtype=torch.float32, device="cuda"), torch.empty_like(xl)
        ws = torch.empty(gf.gf_backward_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
        gf.gf_stash_forward(desc, xl, stash, stream)
        t_s = timed(lambda: gf.gf_stash_forward(desc, xl, stash, stream))
        t_b = timed(lambda: gf.gf_backward(desc, gyl, stash, wl, gW, gX, ws, None, stream))
        out["nhwc_layer_us"][L.name] = {"stash_us": t_s, "backward_us": t_b, "layer_us": round(t_s + t_b, 1)}
        del xl, gyl, wl, stash, gW, gX, ws
    torch.cuda.empty_cache()
    return out


def per_config_layers():
    """Every layer of the workload configurations (rows of the measurement table)."""
    from paper_2301_00330_b200 import workloads
    return [l for l in workloads.all_headline_layers() if l.r > 1]


def run_ours(args) -> None:
    import torch
    import paper_2301_00330_b200 as gf
    from paper_2301_00330_b200 import workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    gf.build_library()

    layers = workload()
    n_layers = len(layers)
    n_sets = 2
    stream = torch.cuda.current_stream()
    runs = []          # per layer: (L, desc, w, ws_bytes, [(x, gy, buffers)] * n_sets)
    host_inputs = []
    for L in layers:
        desc = gf.desc_for(L)
        x0, gy0, w0 = workloads.make_inputs(L)
        host_inputs.append((x0, gy0, w0))
        sets = [(torch.roll(x0, i, 0).cuda().contiguous(), torch.roll(gy0, i, 0).cuda().contiguous(),
                 gf.alloc_layer(desc)) for i in range(n_sets)]
        runs.append((L, desc, w0.cuda(), gf.gf_backward_workspace_bytes(desc), sets))

    def layer_step(k: int, i: int, s=None):
        L, desc, w, ws_bytes, sets = runs[k]
        x, gy, b = sets[i % n_sets]
        s = s or stream
        gf.gf_stash_forward(desc, x, b.stash, s)
        gf.gf_backward(desc, gy, b.stash, w, b.g_W, b.g_X, b.workspace, ws_bytes, s)

    def step(i: int, s=None):
        for k in range(n_layers):
            layer_step(k, i, s)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(3, args.warmup)
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()

    # ---- diagnostic pass: every kernel bracketed by events, layer by layer, to find the
    # (layer, kernel) pair that takes the most time ----
    diag_steps = 4
    breakdown = {}
    per_kernel_ms: dict[str, float] = {}
    for k, (L, *_rest) in enumerate(runs):
        gf.gf_profile_configure(2)
        backlog()
        for i in range(diag_steps):
            layer_step(k, i)
        torch.cuda.synchronize()
        diag = gf.gf_profile_read()
        gf.gf_profile_configure(0)
        breakdown[L.name] = {kn: {"launches_per_step": n / diag_steps, "avg_us": round(ms / n * 1e3, 2)}
                             for kn, (n, ms) in diag.items()}
        KERNELS_OF_LAYER[L.name] = tuple(diag.keys())
        for kn, (n, ms) in diag.items():
            per_kernel_ms[kn] = per_kernel_ms.get(kn, 0.0) + ms

    # ---- dominant kernel = the one with the largest summed time over a step (all its launches, all
    # layers): event pairs around it alone, over eager steps ----
    dom_kernel = max(per_kernel_ms, key=per_kernel_ms.get)
    dom_steps = max(1, min(args.steps, 16))
    gf.gf_profile_configure(1, gf.kernel_id(dom_kernel))
    backlog()
    for i in range(dom_steps):
        step(i)
    torch.cuda.synchronize()
    dom = gf.gf_profile_read()
    gf.gf_profile_configure(0)
    dom_pairs = dom.get(dom_kernel, (0, 0.0))
    dom_method = f"event pairs around each of its launches inside {dom_steps} eager steps"
    # An event pair around one launch also times the launch latency behind the first event (the
    # kernel cannot be queued ahead of it) and the second event: several us per launch.  Where the
    # dominant kernel is the only kernel of a public call (the stash pass, gf_stash_forward), its
    # launches are timed as a run instead: the step's own calls of it, over all layers and input
    # sets, enqueued back to back between one pair of events.  Same kernel, same inputs, each
    # launch on tensors no earlier launch of the run has touched.
    if dom_kernel == "stash_pool":
        calls = [(desc, x, b.stash) for (_, desc, _, _, sets) in runs for (x, _, b) in sets]
        reps = 8
        for desc, x, st in calls:
            gf.gf_stash_forward(desc, x, st, stream)
        torch.cuda.synchronize()
        c0 = gf.gf_kernel_launch_count()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        backlog()
        d0.record(stream)
        for _ in range(reps):
            for desc, x, st in calls:
                gf.gf_stash_forward(desc, x, st, stream)
        d1.record(stream)
        torch.cuda.synchronize()
        n_run = gf.gf_kernel_launch_count() - c0
        if n_run == reps * len(calls):                   # one kernel per call, as assumed
            dom = {dom_kernel: (n_run, d0.elapsed_time(d1))}
            dom_steps = reps * n_sets
            dom_method = (f"{n_run} launches (the step's gf_stash_forward calls, {n_sets} input sets, {reps} rounds) "
                          f"enqueued back to back between one pair of events")

    # ---- timed region: exactly K steps.  The steps are replayed from a CUDA graph that holds
    # one step per input set (the launch sequence of the eager calls, captured once), so that
    # the host's enqueue rate does not bound the number; the K mod n_sets remaining steps are
    # enqueued eagerly. ----
    graph = None
    launches_per_step = None
    if args.steps >= n_sets:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        c0 = gf.gf_kernel_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            cap = torch.cuda.current_stream()
            for i in range(n_sets):
                step(i, cap)
        launches_per_step = (gf.gf_kernel_launch_count() - c0) // n_sets
        stream.wait_stream(side)
        graph.replay()               # one untimed replay
        torch.cuda.synchronize()
    replays, rest = (args.steps // n_sets, args.steps % n_sets) if graph is not None else (0, args.steps)
    sampler = ClockSampler(local_rank)
    launches0 = gf.gf_kernel_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    ev0.record(stream)
    for _ in range(replays):
        graph.replay()
    for i in range(rest):
        step(i)
    ev1.record(stream)
    sampler.sample()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    barrier()
    launches = gf.gf_kernel_launch_count() - launches0
    if graph is not None:
        launches += replays * n_sets * launches_per_step     # kernels the replays ran
    ms_total = ev0.elapsed_time(ev1)
    for _, _, _, _, sets in runs:
        assert gf.gf_last_async_status(sets[0][2].workspace) == gf.GF_OK
    ms_total = max_over_ranks(ms_total, dist, "cuda")
    ms_per_step = ms_total / args.steps
    value = job_value_us(ms_total, args.steps, world, n_layers)
    del graph

    # ---- end to end: host buffers in, host buffers out, through the C ABI ----
    e2e_sets = []
    h2d = d2h = 0
    for (L, desc, _, _, _), (x0, gy0, w0) in zip(runs, host_inputs):
        hx, hgy, hw = x0.pin_memory(), gy0.pin_memory(), w0.pin_memory()
        h_gW = torch.empty((L.C_out, L.C_ig, L.K, L.K), dtype=torch.float32).pin_memory()
        h_gX = torch.empty(tuple(x0.shape), dtype=workloads.torch_dtype(L.dtype)).pin_memory()
        arena = torch.empty(gf.gf_host_step_arena_bytes(desc), dtype=torch.uint8, device="cuda")
        e2e_sets.append((desc, hx, hgy, hw, h_gW, h_gX, arena))
        h2d += sum(t.numel() * t.element_size() for t in (hx, hgy, hw))
        d2h += sum(t.numel() * t.element_size() for t in (h_gW, h_gX))

    # one stream per layer: each layer's copies in, kernels and copies out are ordered on its own
    # stream, so the uploads of one layer overlap the downloads of another (the two copy directions
    # use different engines); the timed region opens and closes on the main stream
    # and the layer with the most to download goes first, so that its download runs under the other
    # layers' uploads instead of after them
    e2e_sets.sort(key=lambda t: -(t[4].numel() * t[4].element_size() + t[5].numel() * t[5].element_size()))
    lanes = [torch.cuda.Stream() for _ in e2e_sets]
    lane_done = [torch.cuda.Event() for _ in e2e_sets]

    def e2e_step():
        opened = torch.cuda.Event()
        opened.record(stream)
        for lane, done, (desc, hx, hgy, hw, h_gW, h_gX, arena) in zip(lanes, lane_done, e2e_sets):
            lane.wait_event(opened)
            gf.gf_layer_step_host(desc, hx, hgy, hw, h_gW, h_gX, arena, stream=lane)
            done.record(lane)
        for done in lane_done:
            stream.wait_event(done)

    e2e_steps = max(1, min(args.steps, 5))
    e2e_step()
    barrier()
    ev0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    e2e = {"value": job_value_us(e2e_ms, e2e_steps, world, n_layers), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "api": "gf_layer_step_host per layer, one stream per layer (pinned host buffers; copies of x, g_y, W in and "
                  "g_W, g_X out inside the timed region; uploads of one layer overlap downloads of another, "
                  "layers issued in the order of their download sizes, largest first)"}
    del e2e_sets

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    n_dom, ms_dom = dom.get(dom_kernel, (0, 0.0))
    roof = roofline_step(dom_kernel, ms_dom, n_dom, dom_steps, layers)
    roof["timed_launches"] = n_dom
    if dom_kernel == "stash_pool":
        roof["cuda_kernel"] = ("pool_stream_kernel: four launches per step, three as the stash pass (this entry) and one as the "
                               "gradient filter of the 96->576 layer (entry gy_pool of `kernels`); by the ncu launch list the "
                               "four together are the largest share of the step (profiles/launch_list_bench_step_*.md)")
    roof["timing"] = dom_method
    if dom_pairs[0]:
        roof["avg_launch_us_event_pairs"] = dom_pairs[1] * 1e3 / dom_pairs[0]
    roof["share_of_step_kernel_time"] = per_kernel_ms[dom_kernel] / sum(per_kernel_ms.values())
    peaks, which = measured_peaks()
    step_bytes = sum(L.backward_bytes() + L.stash_bytes_moved() for L in layers)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(layers),
        "timing": (f"CUDA events around K steps; {replays} replays of a {n_sets}-step CUDA graph + {rest} eager steps; "
                   f"dominant kernel (largest summed time over a step): {dom_method}"),
        "parallelism": "replicas only" if world > 1 else "single GPU",
        "block_us": ms_per_step * 1e3,
        "step_algorithmic_bytes": step_bytes,
        "step_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
        "step_frac_of_hbm": step_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "peaks": {"hbm_gbs": peaks["hbm_gbs"], "source": which},
        "roofline": roof, "kernels": breakdown, "clocks": clocks, "e2e": e2e,
        "gpu_launches": int(launches),
    }
    if world == 1:
        line["diagnostics"] = diagnostics(gf, runs)
        for _, _, _, _, sets in runs:
            sets.clear()
        runs.clear()
        torch.cuda.empty_cache()
        if not args.no_extras:
            line["extras"] = extras(gf, layers)
        line["cpu_baseline"] = time_oracle(layers, 32, 2, 1)
        if not args.no_per_config:
            rows = [time_layer(gf, L, peaks) for L in per_config_layers()]
            line["per_config"] = {
                "note": "every layer of the workload configurations: gf_stash_forward and gf_backward timed with CUDA "
                        "events over 8-20 calls behind a stream backlog; frac = algorithmic bytes of the backward / time "
                        f"/ {peaks['hbm_gbs']:.0f} GB/s ({which} copy bandwidth); exact_cudnn_us = exact convolution "
                        "backward of the same shape and dtype through torch/cuDNN (context: it computes the unfiltered "
                        "gradients)",
                "paper_context": PAPER_CONTEXT,
                "rows": rows,
            }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_table(args) -> None:
    """--table: every headline layer and the paper's on-device shapes timed once each way, with
    the per-kernel event times of the backward call.  Prints one JSON line per layer and a
    markdown table; not the contract line."""
    import torch
    import paper_2301_00330_b200 as gf
    from paper_2301_00330_b200 import workloads

    torch.cuda.set_device(0)
    gf.build_library()
    peaks, which = measured_peaks()
    layers = per_config_layers() + workloads.ondevice_table(2, "f32") + workloads.ondevice_table(4, "f32")
    if args.only:
        layers = [l for l in layers if any(k in f"{l.name}/r{l.r}/{l.dtype}" for k in args.only.split(","))]
    rows = []
    for L in layers:
        row = time_layer(gf, L, peaks, with_exact=not args.no_exact, with_kernels=True)
        rows.append(row)
        print(json.dumps(row), flush=True)
    print(f"\n| layer | r | dtype | stash us | backward us | alg MB | GB/s | frac of {peaks['hbm_gbs']:.0f} GB/s ({which}) | exact cuDNN us |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        ex = f"{r['exact_cudnn_us']:.0f}" if r.get("exact_cudnn_us") else "n/a"
        print(f"| {r['layer']} | {r['r']} | {r['dtype']} | {r['stash_us']:.1f} | {r['backward_us']:.1f} | "
              f"{r['backward_alg_MB']:.1f} | {r['backward_gbs']:.0f} | {r['backward_frac_hbm']:.2f} | {ex} |")


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1,
                    help="replicas (one process per GPU); under torchrun the ranks come from the environment, "
                         "otherwise N > 1 re-executes this script under torch.distributed.run")
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-config", action="store_true", help="skip the per_config rows (faster)")
    ap.add_argument("--no-extras", action="store_true", help="skip the timings of the further entry points")
    ap.add_argument("--table", action="store_true", help="time every layer shape once (diagnostic table)")
    ap.add_argument("--only", default="", help="--table: comma-separated substrings of name/rR/dtype to keep")
    ap.add_argument("--no-exact", action="store_true", help="--table: skip the exact cuDNN backward")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.table:
        # started without a launcher: become N ranks on this node
        port = 29500 + os.getpid() % 2000
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
                                  "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]])
    if args.table:
        run_table(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
