#!/usr/bin/env python
"""Benchmark of the filtered convolution backward pass (gradient filtering).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of one layer:
gf_stash_forward (patch-summed activations) + gf_backward (gradient filter,
reduced g_W, reduced g_X with expansion), on the ResNet-style layer
3x3, 256->256, N=64, 28x28, r=2, bf16 inputs with fp32 accumulation.
Prints ONE JSON line (rank 0).  The metric is microseconds per layer backward
(lower is better).  N > 1: independent replicas, one per GPU, no collective on
the data path; the value is time divided by the layers all ranks processed.

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

# DRAM bytes per launch of a kernel from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by kernel name, with the sha1 of the source file
# at capture time; a changed source makes the entry stale (reported as null).
# Captured on the bench layer (profiles/step_resnet3x3_256_N64_28x28_r2_bf16.md).  Writes of a
# single launch stay in the 126 MB L2 past the end of the kernel, so dram__bytes_write is 0
# there and the figure is the read side.
NCU_TRAFFIC: dict[str, dict] = {
    "gx_tc": {"bytes": 6591488, "sha1": "89d154e96ff4d360afd232422b68bd39714d857e"},
    "gw_tc": {"bytes": 13128192, "sha1": "89d154e96ff4d360afd232422b68bd39714d857e"},
    "stash_pool": {"bytes": 25703936, "sha1": "c38ad61ccbdf77bc96e7bf40af6f901fbfce0590"},
    "gy_pool": {"bytes": 25703936, "sha1": "c38ad61ccbdf77bc96e7bf40af6f901fbfce0590"},
}

KERNEL_SOURCE = {
    "stash_pool": "gf_pool.cu", "gy_pool": "gf_pool.cu", "ksum": "gf_tc.cu", "gx_mix": "gf_dense.cu",
    "gw_partial": "gf_dense.cu", "gw_finish": "gf_dense.cu", "dw_fused": "gf_depthwise.cu",
    "gx_tc": "gf_tc.cu", "gw_tc": "gf_tc.cu",
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
    from paper_2301_00330_b200 import workloads
    (layer,) = workloads.config2()
    return layer


def workload_config(layer, extra=None) -> dict:
    cfg = {
        "workload": "configs[1]: ResNet-style 3x3 conv backward, stride 1, pad 1, N=64, 256->256, 28x28, r=2",
        "layer": layer.name, "N": layer.N, "C_in": layer.C_in, "C_out": layer.C_out, "H": layer.H,
        "W": layer.W, "K": layer.K, "groups": layer.groups, "r": layer.r,
        "step": "gf_stash_forward + gf_backward (g_W and g_X)",
    }
    if extra:
        cfg.update(extra)
    return cfg


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
def kernel_cost(name: str, L, splits: int) -> tuple[float, float]:
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
        "gw_tc": (gbar16 + e * L.numel_stash() + 4 * splits * pairs, mix),
        "stash_pool": (e * (L.numel_x() + L.numel_stash()), L.numel_x()),
        "gy_pool": (e * L.numel_gy() + (gbar16 if tc else gbar), L.numel_gy()),
        "ksum": (e * L.numel_w() + 4 * pairs, L.numel_w()),
        "gx_mix": (gbar + 4 * pairs + e * L.numel_x(), mix),
        "gw_partial": (gbar + e * L.numel_stash() + 4 * splits * pairs, mix),
        "gw_finish": (4 * splits * pairs + 4 * L.numel_w(), splits * pairs),
        "dw_fused": (e * (L.numel_gy() + L.numel_stash() + L.numel_x() + L.numel_w()), 3 * L.numel_gy()),
    }
    return table[name]


def traffic_for(name: str):
    ent = NCU_TRAFFIC.get(name)
    src = KERNEL_SOURCE.get(name)
    if not ent or not src:
        return None
    path = os.path.join(ROOT, "paper_2301_00330_b200", "csrc", src)
    with open(path, "rb") as f:
        sha = hashlib.sha1(f.read()).hexdigest()
    return ent["bytes"] if sha == ent.get("sha1") else None


def roofline(name: str, avg_ms: float, L, splits: int) -> dict:
    peaks, which = measured_peaks()
    nbytes, flops = kernel_cost(name, L, splits)
    t = avg_ms * 1e-3
    t_mem = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_alu = flops / (FP32_ALU_TFLOPS * 1e12)
    if t_alu > t_mem and name in ("gx_mix", "gw_partial"):
        ach = flops / t / 1e12
        return {"kernel": name, "bound": "alu", "achieved": ach, "peak": FP32_ALU_TFLOPS, "unit": "TFLOP/s",
                "frac": ach / FP32_ALU_TFLOPS, "traffic": traffic_for(name), "peak_source": "derived: 148 SM x 128 FMA x 2 x 1.965 GHz",
                "avg_launch_us": avg_ms * 1e3}
    ach = nbytes / t / 1e9
    return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "traffic": traffic_for(name), "peak_source": f"of {which}",
            "avg_launch_us": avg_ms * 1e3}


# --------------------------------------------------------------------------- CPU checker timing
def time_oracle(layer, n_sample: int, steps: int, warmup: int) -> dict:
    import numpy as np
    import torch
    import oracle
    from paper_2301_00330_b200 import workloads
    L = layer.with_(N=n_sample)
    x, gy, w = workloads.make_inputs(L)
    x64, gy64, w64 = (t.to(torch.float64).numpy() for t in (x, gy, w))

    def one():
        stash = oracle.stash_forward(x64, L.r)
        return oracle.backward(gy64, stash, w64, L.r, groups=L.groups)

    for _ in range(warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        gw, gx = one()
    dt = (time.perf_counter() - t0) / steps
    assert np.isfinite(gw).all() and np.isfinite(gx).all()
    scale = layer.N / n_sample
    return {"value": dt * 1e6 * scale, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n_sample} of {layer.N} images of the same layer, fp64, time scaled x{scale:g} "
                      f"(every step is linear in the batch); {steps} timed passes",
            "seconds_per_pass": dt}


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layer = workload()
    base = time_oracle(layer, layer.N, max(1, args.steps), max(0, args.warmup))
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": base["value"] / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(layer, {"dtype_in": "bf16 values widened to f64"}),
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


def job_value_us(ms_total: float, steps: int, world: int) -> float:
    """us per layer step of the whole job: every rank ran `steps` layer steps of its own
    replica in ms_total (max over ranks), so the job did steps * world of them."""
    return ms_total * 1e3 / (steps * world)


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

    layer = workload()
    desc = gf.desc_for(layer)
    dt = workloads.torch_dtype(layer.dtype)
    x0, gy0, w0 = workloads.make_inputs(layer)
    n_sets = 4   # rotating input/output sets: 4 x ~106 MB > 3 x the 126 MB L2
    sets = []
    for i in range(n_sets):
        buf = gf.alloc_layer(desc)
        sets.append((torch.roll(x0, i, 0).cuda().contiguous(), torch.roll(gy0, i, 0).cuda().contiguous(), buf))
    w = w0.cuda()
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    set_bytes = sum(t.numel() * t.element_size() for t in (sets[0][0], sets[0][1], sets[0][2].stash,
                                                            sets[0][2].g_X, sets[0][2].g_W, sets[0][2].workspace))
    stream = torch.cuda.current_stream()

    def step(i: int):
        x, gy, b = sets[i % n_sets]
        gf.gf_stash_forward(desc, x, b.stash, stream)
        gf.gf_backward(desc, gy, b.stash, w, b.g_W, b.g_X, b.workspace, ws_bytes, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up; its first steps bracket every kernel to find the dominant one ----
    warm = max(3, args.warmup)
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()

    def backlog(ms: float = 4.0):
        """Keeps the stream busy for a few ms so that the launches enqueued next
        wait in the queue and then run back to back: event pairs around a
        kernel then measure the GPU, not the enqueueing host thread."""
        torch.cuda._sleep(int(ms * 1e-3 * 1.9e9))

    # ---- diagnostic pass: every kernel bracketed by events, to find the dominant one ----
    diag_steps = 8
    gf.gf_profile_configure(2)
    backlog()
    for i in range(diag_steps):
        step(i)
    torch.cuda.synchronize()
    diag = gf.gf_profile_read()
    gf.gf_profile_configure(0)
    total_diag = sum(ms for _, ms in diag.values()) or 1.0
    breakdown = {k: {"launches_per_step": n / diag_steps, "avg_us": ms / n * 1e3, "share": ms / total_diag}
                 for k, (n, ms) in diag.items()}
    dominant = max(diag.items(), key=lambda kv: kv[1][1])[0]

    # ---- dominant kernel: event pairs around it alone, over eager steps ----
    dom_steps = max(1, min(args.steps, 64))
    gf.gf_profile_configure(1, gf.kernel_id(dominant))
    backlog()
    for i in range(dom_steps):
        step(i)
    torch.cuda.synchronize()
    dom = gf.gf_profile_read()
    gf.gf_profile_configure(0)

    # ---- timed region: exactly K steps.  The steps are replayed from a CUDA graph
    # that holds one step per input set (the launch sequence of the eager calls,
    # captured once), so that the host's enqueue rate does not bound the number;
    # the K mod n_sets remaining steps are enqueued eagerly. ----
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
                x, gy, b = sets[i]
                gf.gf_stash_forward(desc, x, b.stash, cap)
                gf.gf_backward(desc, gy, b.stash, w, b.g_W, b.g_X, b.workspace, ws_bytes, cap)
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
    assert gf.gf_last_async_status(sets[0][2].workspace) == gf.GF_OK
    ms_total = max_over_ranks(ms_total, dist, "cuda")
    ms_per_step = ms_total / args.steps
    value = job_value_us(ms_total, args.steps, world)

    # ---- end to end: host buffers in, host buffers out, through the C ABI ----
    hx, hgy, hw = x0.pin_memory(), gy0.pin_memory(), w0.pin_memory()
    h_gW = torch.empty((layer.C_out, layer.C_ig, layer.K, layer.K), dtype=torch.float32).pin_memory()
    h_gX = torch.empty(tuple(x0.shape), dtype=dt).pin_memory()
    arena = torch.empty(gf.gf_host_step_arena_bytes(desc), dtype=torch.uint8, device="cuda")
    e2e_steps = max(1, min(args.steps, 30))
    for _ in range(2):
        gf.gf_layer_step_host(desc, hx, hgy, hw, h_gW, h_gX, arena, stream=stream)
    barrier()
    ev0.record(stream)
    for _ in range(e2e_steps):
        gf.gf_layer_step_host(desc, hx, hgy, hw, h_gW, h_gX, arena, stream=stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = ev0.elapsed_time(ev1)
    e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
    h2d = sum(t.numel() * t.element_size() for t in (hx, hgy, hw))
    d2h = sum(t.numel() * t.element_size() for t in (h_gW, h_gX))
    e2e = {"value": job_value_us(e2e_ms, e2e_steps, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps, "api": "gf_layer_step_host (pinned host buffers)"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # split count of the reduced g_W contraction, needed for its byte count
    if layer.groups == 1 and layer.C_out % 8 == 0 and layer.r >= 2:      # tensor-core path: 128 x 128 tiles, one wave of CTAs
        tiles = ((layer.C_out + 127) // 128) * ((layer.C_in + 127) // 128)
        chunks = -(-(layer.N * layer.Hp * layer.Wp) // 64)
        splits = max(1, min(chunks, -(-148 // tiles)))
    else:
        tiles = ((layer.C_out // layer.groups + 63) // 64) * ((layer.C_ig + 63) // 64) * layer.groups
        splits = max(1, min(layer.N, -(-592 // tiles)))
    n_dom, ms_dom = dom.get(dominant, (0, 0.0))
    roof = roofline(dominant, ms_dom / max(n_dom, 1), layer, splits)
    roof["timed_launches"] = n_dom
    peaks, which = measured_peaks()
    step_bytes = layer.backward_bytes() + layer.stash_bytes_moved()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(layer, {
            "l2": f"inputs and outputs rotate over {n_sets} sets of {set_bytes / 1e6:.0f} MB (> 3x the 126 MB L2)",
            "timing": (f"CUDA events around K steps; {replays} replays of a {n_sets}-step CUDA graph + {rest} eager "
                       f"steps; dominant kernel timed by event pairs over {dom_steps} eager steps"),
            "parallelism": "replicas only" if world > 1 else "single GPU"}),
        "step_algorithmic_bytes": step_bytes,
        "step_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
        "step_frac_of_hbm": step_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "peaks": {"hbm_gbs": peaks["hbm_gbs"], "source": which},
        "roofline": roof, "kernels": breakdown, "clocks": clocks, "e2e": e2e,
        "gpu_launches": int(launches),
    }
    if world == 1:
        line["cpu_baseline"] = time_oracle(layer, layer.N, 5, 1)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_table(args) -> None:
    """--table: every headline layer (and the paper's on-device shapes) timed once each way:
    gf_stash_forward, gf_backward, and an exact backward through torch/cuDNN as context.
    Prints one JSON line per layer and a markdown table; not the contract line."""
    import torch
    import paper_2301_00330_b200 as gf
    from paper_2301_00330_b200 import workloads

    torch.cuda.set_device(0)
    gf.build_library()
    peaks, which = measured_peaks()
    layers = [l for l in workloads.all_headline_layers() if l.r > 1] + workloads.ondevice_table(2, "f32") \
        + workloads.ondevice_table(4, "f32")
    if args.only:
        layers = [l for l in layers if any(k in f"{l.name}/r{l.r}/{l.dtype}" for k in args.only.split(","))]
    stream = torch.cuda.current_stream()
    rows = []

    def timed(fn, reps):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(int(3e-3 * 1.9e9))       # backlog: the calls below queue up behind it
        e0.record(stream)
        for i in range(reps):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    for L in layers:
        desc = gf.desc_for(L)
        x0, gy0, w0 = workloads.make_inputs(L)
        per_set = L.backward_bytes() + L.stash_bytes_moved()
        n_sets = max(1, min(4, int(400e6 // per_set) + 1))
        sets = [(torch.roll(x0, i, 0).cuda(), torch.roll(gy0, i, 0).cuda(), gf.alloc_layer(desc)) for i in range(n_sets)]
        w = w0.cuda()
        ws_bytes = gf.gf_backward_workspace_bytes(desc)
        reps = 20 if per_set < 300e6 else 8

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
        # per-kernel event times of the backward call (each bracketed, so a few us high)
        gf.gf_profile_configure(2)
        torch.cuda._sleep(int(3e-3 * 1.9e9))
        for i in range(4):
            bwd(i)
        torch.cuda.synchronize()
        kern = {k: round(ms / n * 1e3, 1) for k, (n, ms) in gf.gf_profile_read().items()}
        gf.gf_profile_configure(0)
        try:
            t_exact = timed(exact, max(2, reps // 4))
        except Exception:
            t_exact = None
        row = {"layer": L.name, "r": L.r, "dtype": L.dtype, "stash_us": t_stash, "backward_us": t_bwd,
               "backward_alg_MB": L.backward_bytes() / 1e6,
               "backward_gbs": L.backward_bytes() / t_bwd / 1e3,
               "backward_frac_hbm": L.backward_bytes() / t_bwd / 1e3 / peaks["hbm_gbs"],
               "stash_gbs": L.stash_bytes_moved() / t_stash / 1e3,
               "stash_frac_hbm": L.stash_bytes_moved() / t_stash / 1e3 / peaks["hbm_gbs"],
               "exact_cudnn_us": t_exact, "reduced_gflop": L.reduced_flops() / 1e9, "kernels_us": kern}
        rows.append(row)
        print(json.dumps(row), flush=True)
        del sets
        torch.cuda.empty_cache()
    print(f"\n| layer | r | dtype | stash us | backward us | alg MB | GB/s | frac of {peaks['hbm_gbs']:.0f} GB/s ({which}) | exact cuDNN us |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        ex = f"{r['exact_cudnn_us']:.0f}" if r["exact_cudnn_us"] else "n/a"
        print(f"| {r['layer']} | {r['r']} | {r['dtype']} | {r['stash_us']:.1f} | {r['backward_us']:.1f} | "
              f"{r['backward_alg_MB']:.1f} | {r['backward_gbs']:.0f} | {r['backward_frac_hbm']:.2f} | {ex} |")


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--table", action="store_true", help="time every layer shape once (diagnostic table)")
    ap.add_argument("--only", default="", help="--table: comma-separated substrings of name/rR/dtype to keep")
    args = ap.parse_args()
    if args.table:
        run_table(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
