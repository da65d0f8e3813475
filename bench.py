#!/usr/bin/env python
"""Benchmark of the LBP-WHT linear-backward hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = Algorithm 1 (project x and g_y, the two low-rank products, expand
g_x) for the four linear layers of a ViT-B block (qkv, proj, fc1, fc2) on one
batch of B=128 images with a 16x16 token grid, WHT order k=8, rank r=8, bf16
data with fp32 accumulation.  The metric is tokens/s: tokens of the batch
(32768 per GPU) divided by the time of one step.

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on
a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "LBP-WHT linear backward tokens/s at rank r; % of HBM/tensor roofline"
UNIT = "tokens/s"
CONFIG = 3
RANK = 8
WORKLOAD = ("config3: ViT-B block linears qkv 768->2304, proj 768->768, fc1 768->3072, "
            "fc2 3072->768; B=128, grid 16x16, k=8, r=8 (PREFIX-8 low-pass set), bf16")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


# DRAM traffic per step (sum over the four layers, bytes) of the two kernels, from
# the ncu capture summarised in profiles/ (dram__bytes_read.sum + dram__bytes_write.sum);
# None = not captured for the current kernels.
NCU_TRAFFIC_PER_STEP = {"wht_project_mma_kernel": 830.1e6, "lbp_products_pair_kernel": 285.2e6}


# ------------------------------------------------------------------ clocks ----
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nvml = None
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        n = self._nvml
        names = {
            getattr(n, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(n, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(n, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(n, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM))
                try:
                    mask = n.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = n.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------- cpu oracle ----
def _oracle_sample(batch: int, repeats: int = 1):
    """Times the fp64 oracle's low-rank route on `batch` images of every layer."""
    import numpy as np
    import torch
    import synth
    from oracle import lbp_oracle as O

    cases = synth.config_cases(CONFIG)
    bases = O.select_bases(cases[0].k, O.RULE_PREFIX, RANK)
    data = []
    for c in cases:
        x, gy, w = synth.make_layer_inputs(c, batch=batch)
        data.append((c, x.to(torch.float64).numpy(), gy.to(torch.float64).numpy(),
                     w.to(torch.float64).numpy()))
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        for c, x, gy, w in data:
            O.backward_lowrank(x, gy, w, c.k, bases)
        times.append(time.perf_counter() - t0)
    tokens = batch * cases[0].H * cases[0].W
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    return tokens, times, cores


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    steps = max(1, args.steps)
    # bounded sample: about 0.07 s of oracle time per image; keep the whole run near 90 s
    batch = int(max(1, min(16, 90.0 / (steps + args.warmup) / 0.07)))
    tokens, times, cores = _oracle_sample(batch, repeats=args.warmup + steps)
    timed = times[args.warmup:]
    sec = sum(timed) / len(timed)
    value = tokens / sec
    sample = f"first {batch} of 128 images of all four layers, r={RANK}, fp64 numpy oracle"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------- main ----
def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2309_15275_b200 as lbp
    import synth
    from paper_2309_15275_b200.dist import allreduce_gw

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    from paper_2309_15275_b200.build import build_library
    if not os.path.exists(lbp.LIB_PATH):
        build_library()

    cases = synth.config_cases(CONFIG)
    k = cases[0].k
    bases = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, RANK)
    peaks = _peaks()

    # per-rank batch: every rank owns its own seeded batch of B images (weak scaling)
    layers = []
    for c in cases:
        x, gy, w = synth.make_layer_inputs(c, seed=synth.SEED + rank)
        L = {"case": c, "x_h": x.pin_memory(), "gy_h": gy.pin_memory(), "w_h": w.pin_memory()}
        L["x"], L["gy"], L["w"] = x.to(dev), gy.to(dev), w.to(dev)
        L["gx"] = torch.empty_like(L["x"])
        L["gw"] = torch.empty((c.Cout, c.Cin), dtype=torch.float32, device=dev)
        L["ws"] = lbp.alloc_workspace(L["x"], L["gy"], k, RANK)
        L["ws_full"] = lbp.alloc_workspace(L["x"], L["gy"], k, k * k)
        L["gx_h"] = torch.empty_like(L["x_h"]).pin_memory()
        L["gw_h"] = torch.empty((c.Cout, c.Cin), dtype=torch.float32).pin_memory()
        layers.append(L)
    tokens_per_step = cases[0].tokens          # per GPU

    def step(record=None):
        if record is None:
            # the four layers are independent problems with their own buffers: one call
            lbp.lbp_backward_batch([L["x"] for L in layers], [L["gy"] for L in layers],
                                   [L["w"] for L in layers], k, bases,
                                   g_xs=[L["gx"] for L in layers], g_Ws=[L["gw"] for L in layers],
                                   wss=[L["ws"] for L in layers])
            for L in layers:
                allreduce_gw(L["gw"])   # data-parallel exchange; no-op on one GPU
            return
        for li, L in enumerate(layers):
            # boundaries used: 0 start, 1 after the projection, 3 after the products kernel
            lbp.lbp_set_phase_events([e if i in (0, 1, 3) else None
                                      for i, e in enumerate(record[li])])
            lbp.lbp_backward(L["x"], L["gy"], L["w"], k, bases, g_x=L["gx"], g_W=L["gw"], ws=L["ws"])
            allreduce_gw(L["gw"])
        lbp.lbp_set_phase_events(None)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    nphase = lbp.lbp_phase_count()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- timed region: exactly K steps, CUDA events on the launching stream ----
    # phase events are recorded on (at most) 32 evenly spaced steps of the timed region
    ev_stride = max(1, args.steps // 32)
    ev = {s: [[torch.cuda.Event(enable_timing=True) for _ in range(nphase)] for _ in layers]
          for s in range(0, args.steps, ev_stride)}
    for s_ in ev.values():
        for l_ in s_:
            for e in l_:
                e.record()          # materialise the handles before the timed region
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = lbp.lbp_launch_count()
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_beg.record()
    for s in range(args.steps):
        step(ev.get(s))
    t_end.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    launches = lbp.lbp_launch_count() - launches0
    ms_total = t_beg.elapsed_time(t_end)
    for L in layers:
        st = lbp.lbp_poll_status(L["ws"])
        if st != 0:
            raise RuntimeError(f"device status {st}: {lbp.lbp_status_string(st)}")
    if world > 1:
        t = torch.tensor([ms_total], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_per_step = ms_total / args.steps
    value = tokens_per_step * world / (ms_per_step * 1e-3)

    # ---- per-phase device times from the events recorded inside the timed region ----
    phase_ms = [[0.0] * nphase for _ in layers]
    for s in ev:
        for li in range(len(layers)):
            phase_ms[li][1] += ev[s][li][0].elapsed_time(ev[s][li][1]) / len(ev)
            phase_ms[li][3] += ev[s][li][1].elapsed_time(ev[s][li][3]) / len(ev)

    es = 2
    layer_rows = []
    proj_bytes = proj_ms = prod_bytes = prod_flops = prod_ms = 0.0
    for li, L in enumerate(layers):
        c = L["case"]
        T, nb = c.tokens, c.blocks
        rows = nb * RANK
        alg_bytes = es * T * (2 * c.Cin + c.Cout) + es * c.Cin * c.Cout + 4 * c.Cin * c.Cout
        alg_flops = 4.0 * c.Cin * c.Cout * rows
        t_roof = max(alg_bytes / (peaks["hbm_gbs"] * 1e9), alg_flops / (peaks["bf16_tflops"] * 1e12))
        us = sum(phase_ms[li][1:]) * 1e3
        layer_rows.append({
            "layer": c.name, "us": round(us, 2), "tokens_per_s": T / (us * 1e-6),
            "roofline_us": round(t_roof * 1e6, 2), "roofline_frac": round(t_roof * 1e6 / us, 4),
            "phase_us": {"project_x_gy": round(phase_ms[li][1] * 1e3, 2),
                         "products_expand": round(phase_ms[li][3] * 1e3, 2)},
        })
        # projection launches: read T*C elements, write rows*C elements
        proj_bytes += es * (T + rows) * (c.Cin + c.Cout)
        proj_ms += phase_ms[li][1]
        # products + expansion launch: read x_hat, g_y_hat, W once, write g_x and g_W
        prod_bytes += es * rows * (c.Cin + c.Cout) + es * c.Cin * c.Cout + es * T * c.Cin \
            + 4 * c.Cin * c.Cout
        prod_flops += alg_flops
        prod_ms += phase_ms[li][3]

    # ---- speedup over the library's own full-rank mode (outside the timed region) ----
    if rank == 0:
        for li, L in enumerate(layers):
            for _ in range(2):
                lbp.lbp_backward_fullrank(L["x"], L["gy"], L["w"], k, g_x=L["gx"], g_W=L["gw"],
                                          ws=L["ws_full"])
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(5):
                lbp.lbp_backward_fullrank(L["x"], L["gy"], L["w"], k, g_x=L["gx"], g_W=L["gw"],
                                          ws=L["ws_full"])
            b.record()
            torch.cuda.synchronize()
            full_us = a.elapsed_time(b) * 1e3 / 5
            layer_rows[li]["fullrank_us"] = round(full_us, 2)
            layer_rows[li]["speedup_vs_fullrank"] = round(full_us / layer_rows[li]["us"], 3)
    # ---- the other ranks of the configuration (r = 2, 4, 16), outside the timed region ----
    rank_rows = []
    if rank == 0:
        full_step_us = sum(r_["fullrank_us"] for r_ in layer_rows)
        for rr in (2, 4, 8, 16):
            bases_r = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, rr)
            wss = [lbp.alloc_workspace(L["x"], L["gy"], k, rr) for L in layers]

            def one_step():
                lbp.lbp_backward_batch([L["x"] for L in layers], [L["gy"] for L in layers],
                                       [L["w"] for L in layers], k, bases_r,
                                       g_xs=[L["gx"] for L in layers], g_Ws=[L["gw"] for L in layers],
                                       wss=wss)
            for _ in range(3):
                one_step()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(10):
                one_step()
            b.record()
            torch.cuda.synchronize()
            us = a.elapsed_time(b) * 1e3 / 10
            roof = 0.0
            for L in layers:
                c = L["case"]
                ab = 2 * c.tokens * (2 * c.Cin + c.Cout) + 2 * c.Cin * c.Cout + 4 * c.Cin * c.Cout
                af = 4.0 * c.Cin * c.Cout * c.blocks * rr
                roof += max(ab / (peaks["hbm_gbs"] * 1e9), af / (peaks["bf16_tflops"] * 1e12)) * 1e6
            rank_rows.append({"r": rr, "us_per_step": round(us, 2),
                              "tokens_per_s": tokens_per_step / (us * 1e-6),
                              "roofline_us": round(roof, 2), "roofline_frac": round(roof / us, 4),
                              "speedup_vs_fullrank": round(full_step_us / us, 3)})
            del wss
    barrier()

    # ---- LHE profiling pass (Sec. 3.2) on g_y of every layer, outside the timed region ----
    lhe_rows = []
    if rank == 0:
        for L in layers:
            gy = L["gy"]
            Bq, Hq, Wq, Cq = gy.shape
            sws = torch.empty(lbp.lbp_spectrum_workspace_bytes(Bq, Hq, Wq, Cq, k, lbp.LBP_BF16),
                              dtype=torch.uint8, device=dev)
            e_out = torch.empty((k, k), dtype=torch.float64, device=dev)
            for _ in range(2):
                lbp.lbp_spectrum(gy, k, out=e_out, ws=sws)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(5):
                lbp.lbp_spectrum(gy, k, out=e_out, ws=sws)
            b.record()
            torch.cuda.synchronize()
            us = a.elapsed_time(b) * 1e3 / 5
            nbytes = gy.numel() * gy.element_size()
            lhe_rows.append({"layer": L["case"].name, "us": round(us, 2), "bytes": nbytes,
                             "gbs": round(nbytes / us / 1e3, 1),
                             "frac_of_hbm_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
            del sws
    barrier()

    # ---- end to end: host buffers, copies inside the timed region ----
    e2e_steps = max(1, min(args.steps, 3))
    h2d = sum(L[n].numel() * L[n].element_size() for L in layers for n in ("x_h", "gy_h", "w_h"))
    d2h = sum(L[n].numel() * L[n].element_size() for L in layers for n in ("gx_h", "gw_h"))

    # Copies run on two side streams so that the host-to-device copy of the next
    # layer, the kernels of this layer and the device-to-host copy of the previous
    # one overlap (PCIe is full duplex); events order every reuse of a buffer.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    for L in layers:
        L["ev_in"], L["ev_done"], L["ev_out"] = (torch.cuda.Event() for _ in range(3))
        L["ev_done"].record(cur)
        L["ev_out"].record(cur)

    def e2e_step():
        for L in layers:
            with torch.cuda.stream(s_in):
                s_in.wait_event(L["ev_done"])          # the previous step's kernels read these buffers
                L["x"].copy_(L["x_h"], non_blocking=True)
                L["gy"].copy_(L["gy_h"], non_blocking=True)
                L["w"].copy_(L["w_h"], non_blocking=True)
                L["ev_in"].record(s_in)
            cur.wait_event(L["ev_in"])
            cur.wait_event(L["ev_out"])                # the previous step's results have left g_x / g_W
            lbp.lbp_backward(L["x"], L["gy"], L["w"], k, bases, g_x=L["gx"], g_W=L["gw"], ws=L["ws"])
            allreduce_gw(L["gw"])
            L["ev_done"].record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(L["ev_done"])
                L["gx_h"].copy_(L["gx"], non_blocking=True)
                L["gw_h"].copy_(L["gw"], non_blocking=True)
                L["ev_out"].record(s_out)

    def e2e_join():
        for L in layers:
            cur.wait_event(L["ev_out"])

    e2e_step()
    e2e_join()
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_join()                                         # every result is in host memory
    b.record()
    barrier()
    e2e_ms = a.elapsed_time(b) / e2e_steps
    if world > 1:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_value = tokens_per_step * world / (e2e_ms * 1e-3)

    if rank == 0:
        # the two kernels of a step: the HBM-bound projection and the persistent
        # products + expansion kernel; the one with the larger share is reported
        # as `roofline`, the other as `roofline_other`
        all_ms = sum(sum(p[1:]) for p in phase_ms)
        proj_ach = proj_bytes / (proj_ms * 1e-3) / 1e9
        r_proj = {"bound": "hbm", "kernel": "wht_project_mma_kernel", "achieved": round(proj_ach, 1),
                  "peak": peaks["hbm_gbs"], "unit": "GB/s",
                  "frac": round(proj_ach / peaks["hbm_gbs"], 4),
                  "traffic": NCU_TRAFFIC_PER_STEP["wht_project_mma_kernel"],
                  "algorithmic_bytes": int(proj_bytes), "launches_per_step": len(layers),
                  "peak_source": peaks["source"], "share_of_step": round(proj_ms / all_ms, 4)}
        # products kernel: the slower of its bytes at HBM peak and its FLOPs at the
        # sustained bf16 peak (it runs inside a long step) decides the bound
        t_b = prod_bytes / (peaks["hbm_gbs"] * 1e9)
        t_f = prod_flops / (peaks["bf16_tflops_sustained"] * 1e12)
        if t_f >= t_b:
            ach = prod_flops / (prod_ms * 1e-3) / 1e12
            r_prod = {"bound": "tensor", "achieved": round(ach, 1),
                      "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                      "frac": round(ach / peaks["bf16_tflops_sustained"], 4)}
        else:
            ach = prod_bytes / (prod_ms * 1e-3) / 1e9
            r_prod = {"bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"],
                      "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4)}
        r_prod.update({"kernel": "lbp_products_pair_kernel",
                       "traffic": NCU_TRAFFIC_PER_STEP["lbp_products_pair_kernel"],
                       "algorithmic_bytes": int(prod_bytes), "algorithmic_flops": prod_flops,
                       "launches_per_step": len(layers), "peak_source": peaks["source"],
                       "share_of_step": round(prod_ms / all_ms, 4)})
        roofline, roofline_other = (r_proj, r_prod) if proj_ms >= prod_ms else (r_prod, r_proj)
        whole_roof_us = sum(r["roofline_us"] for r in layer_rows)
        whole_us = sum(r["us"] for r in layer_rows)
        cpu_tokens, cpu_times, cores = _oracle_sample(16, repeats=1) if world == 1 else (0, [1.0], 0)
        sample = f"first 16 of 128 images of all four layers, r={RANK}, fp64 numpy oracle"
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens_per_step_per_gpu": tokens_per_step,
                       "l2": "inputs larger than L2 (>= 150 MB per layer, 1.2 GB per step)",
                       "multi_gpu": "batch sharded per rank; g_W all-reduced (NCCL) when N > 1"},
            "roofline": roofline,
            "roofline_other": roofline_other,
            "path_roofline": {"roofline_us": round(whole_roof_us, 2),
                              "achieved_us": round(ms_per_step * 1e3, 2),
                              "frac": round(whole_roof_us / (ms_per_step * 1e3), 4),
                              "achieved_us_event_timed_steps": round(whole_us, 2),
                              "note": "sum over the four layers of max(algorithmic bytes / HBM "
                                      "peak, 4 Cin Cout M_hat / bf16 peak), of " + peaks["source"] +
                                      " peaks, against the step time; the per-layer and per-phase "
                                      "figures come from the steps that carry phase events, which "
                                      "cost about 2.5 us per event"},
            "layers": layer_rows,
            "rank_sweep": rank_rows,
            "lhe_spectrum": lhe_rows,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if world == 1:
            line["cpu_baseline"] = {"value": cpu_tokens / cpu_times[0], "unit": UNIT, "cores": cores,
                                    "kind": "oracle", "sample": sample}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
