#!/usr/bin/env python
"""Benchmark of the SketchSSM decode hot path on B200.

One *step* is one window of Algorithm 1 over a stack of layers: for every layer, L-1 non-flush decode
steps (sketchssm_decode_step) and one flush (sketchssm_state_update with the sketch refresh), over the
whole batch of the workload.  The metric is decode tokens/s per layer:  B * L * n_layers / step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed on a bounded sample of the
same workload instead.  Under torchrun (N > 1) every rank runs the same per-GPU workload (weak scaling,
no data-path collective: heads are independent); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_33051_b200 import synth, traffic  # noqa: E402

METRIC = "decode tokens/s per layer"
UNIT = "tokens/s/layer"
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/:
# (kernel, workload) -> (captured bytes, algorithmic bytes of the captured launches).  Traffic grows in proportion
# to the algorithmic bytes (ring fill), so the bench line scales the captured figure to its own average launch.
NCU_TRAFFIC_CAPTURES = {
    ("decode_kernel", "c2_mamba2"): (118.08e6, 0.5 * (traffic.decode_bytes("mamba2", 256, 64, 128, 64, 16, 4, "bf16")
                                                      + traffic.decode_bytes("mamba2", 256, 64, 128, 64, 16, 5, "bf16"))),
    ("update_kernel", "c2_mamba2"): (1194.56e6, float(traffic.update_bytes("mamba2", 256, 64, 128, 64, 16, 15, "bf16"))),
}


def ncu_traffic(kernel: str, workload: str, algorithmic_bytes_per_launch: float):
    cap = NCU_TRAFFIC_CAPTURES.get((kernel, workload))
    return None if cap is None else cap[0] * algorithmic_bytes_per_launch / cap[1]


def max_over_ranks(ms_local: float, dist, device="cuda") -> float:
    """Job time of a multi-rank run: the slowest rank's device time."""
    if dist is None:
        return ms_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(tokens_per_rank: float, world: int, ms_step: float) -> float:
    """Whole-job tokens/s/layer: every rank processes its own shard (weak scaling, no exchange)."""
    return world * tokens_per_rank / (ms_step * 1e-3)


def rank_shard(total_batch: int, rank: int, world: int):
    """[begin, end) of the batch entries a rank owns when one batch is split across ranks (heads and batch
    entries are independent, so shards never communicate)."""
    return (total_batch * rank) // world, (total_batch * (rank + 1)) // world


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, device_index: int, period_s: float = 0.01):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# ---------------------------------------------------------------------------------------------
# workload construction
# ---------------------------------------------------------------------------------------------
def fitted_basis(w: synth.Workload):
    """Omega [H,K,r], C [H,r,K] float32 from the workload's calibration queries (E_0 = I)."""
    from paper_2609_33051_b200 import calibrate
    if w.basis == "qr":
        Om = synth.qr_basis(w)
        return Om, np.ascontiguousarray(np.swapaxes(Om, 1, 2))
    Om = np.empty((w.heads, w.dk, w.rank), np.float32)
    C = np.empty((w.heads, w.rank, w.dk), np.float32)
    for h in range(w.heads):
        O, Cm = calibrate.fit_head(torch.from_numpy(synth.calibration_queries(w, 0, h)), w.rank)
        Om[h], C[h] = O.numpy().astype(np.float32), Cm.numpy().astype(np.float32)
    return Om, C


class Stack:
    """n_layers independent layers of one workload on one GPU, with one window of device-resident inputs each."""

    def __init__(self, w: synth.Workload, n_layers: int, device: int):
        from paper_2609_33051_b200.binding import SketchSSM
        self.w, self.n_layers, self.device = w, n_layers, device
        dev = torch.device("cuda", device)
        Om, C = fitted_basis(w)
        S0 = torch.from_numpy(synth.initial_state(w, 0)).to(dev)
        dec_io = w.io if w.kind == "kda" else "f32"
        window = []
        for t in range(w.buf_len):
            x = synth.step_inputs(w, 0, t)
            window.append(dict(q=synth.to_torch(x["q"], w.io, dev), k=synth.to_torch(x["k"], w.io, dev),
                               v=synth.to_torch(x["v"], w.io, dev), beta=synth.to_torch(x["beta"], "f32", dev),
                               decay=synth.to_torch(x["decay"], dec_io, dev)))
        self.host_window = None
        self.layers, self.inputs, self.outs = [], [], []
        for _ in range(n_layers):
            m = SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, out="f32", device=device)
            m.state.copy_(S0)
            m.omega.copy_(torch.from_numpy(Om))
            m.coef.copy_(torch.from_numpy(C))
            m.state_update(0)
            self.layers.append(m)
            # every layer gets its own copy of the window so that no input is served from L2 across layers
            self.inputs.append([{k: v.clone() for k, v in tok.items()} for tok in window])
            self.outs.append(m.new_output())
        self.window0 = window
        torch.cuda.synchronize(dev)

    def device_bytes(self) -> int:
        m = self.layers[0]
        per = m.state.numel() * 4 + m.sketch.numel() * 4 + m.ring.numel()
        per += sum(v.numel() * v.element_size() for tok in self.inputs[0] for v in tok.values())
        return per * self.n_layers

    def run_window(self, mode: str = "sketch", events=None):
        """One step: L tokens through every layer.  mode: "sketch" (decode_step + state_update),
        "full_read" (full_read_decode + state_update without the sketch write) or "standard" (no buffering: the
        state is read, updated with the one token and written back at every step; the flush kernel with an empty
        ring and no sketch).  `events`, if given, receives (kind, n_before, start_event, end_event) per launch."""
        from paper_2609_33051_b200.binding import NO_SKETCH
        L = self.w.buf_len
        launches = 0
        for t in range(L):
            for li, m in enumerate(self.layers):
                tok, o = self.inputs[li][t], self.outs[li]
                if events is not None:
                    e0 = torch.cuda.Event(enable_timing=True)
                    e1 = torch.cuda.Event(enable_timing=True)
                    e0.record()
                if mode == "standard":
                    m.state_update(0, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], o, flags=NO_SKETCH)
                elif t < L - 1:
                    if mode == "sketch":
                        m.decode_step(t, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], o)
                    else:
                        m.full_read_decode(t, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], o)
                else:
                    m.state_update(t, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], o,
                                   flags=0 if mode == "sketch" else NO_SKETCH)
                launches += m.last_launch_count()
                if events is not None:
                    e1.record()
                    events.append(("decode" if t < L - 1 else "update", t, e0, e1))
        return launches

    def run_decode_only(self):
        """The L-1 decode steps of a window over every layer, back to back, no flush (the ring slots are simply
        rewritten with the same tokens on the next pass)."""
        L = self.w.buf_len
        for t in range(L - 1):
            for li, m in enumerate(self.layers):
                tok = self.inputs[li][t]
                m.decode_step(t, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], self.outs[li])
        return (L - 1) * self.n_layers

    def run_update_only(self):
        """One flush per layer, back to back (full ring: n_before = L-1 plus the token)."""
        L = self.w.buf_len
        for li, m in enumerate(self.layers):
            tok = self.inputs[li][L - 1]
            m.state_update(L - 1, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], self.outs[li])
        return self.n_layers

    # -- end-to-end: host buffers, copies inside the timed region ---------------------------------
    def setup_host(self):
        m = self.layers[0]
        self.host_window = []
        for tok in self.window0:
            hb = m.new_token_buffers(pinned_host=True)
            for k in ("q", "k", "v", "beta", "decay"):
                hb[k].copy_(tok[k])
            self.host_window.append(hb)
        self.staging = [m.new_token_buffers(pinned_host=False) for _ in range(2)]
        self.host_out = [m.new_token_buffers(pinned_host=True)["out"] for _ in range(2)]
        self.side_streams = [torch.cuda.Stream(device=self.device) for _ in range(2)]

    def run_window_host(self):
        """One window with host token tensors.  Layer-steps alternate between two streams (each with its own device
        staging and host output buffer) so that the upload of one layer-step overlaps the kernel and the download
        of the previous one; a layer always uses the same stream, so its own steps stay ordered."""
        from paper_2609_33051_b200 import binding
        L = self.w.buf_len
        h2d = d2h = 0
        cur = torch.cuda.current_stream()
        for s in self.side_streams:
            s.wait_stream(cur)
        for t in range(L):
            hb = self.host_window[t]
            for li, m in enumerate(self.layers):
                op = binding.OP_DECODE if t < L - 1 else binding.OP_UPDATE
                host = dict(hb)
                host["out"] = self.host_out[li & 1]
                m.step_host(op, t, host, self.staging[li & 1], stream=self.side_streams[li & 1])
                h2d += sum(hb[k].numel() * hb[k].element_size() for k in ("q", "k", "v", "beta", "decay"))
                d2h += host["out"].numel() * host["out"].element_size()
        for s in self.side_streams:
            cur.wait_stream(s)
        return h2d, d2h


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------
def oracle_window(w: synth.Workload, sample_heads: int, reps: int = 1):
    """Time the oracle, as it stands, on one window of `sample_heads` heads of the workload.
    Returns (seconds per window, head-steps per window, threads used)."""
    from oracle import sketchssm_oracle as orc
    total = w.batch * w.heads
    idx = np.sort(np.random.default_rng(1).choice(total, size=min(sample_heads, total), replace=False))
    bs, hs = idx // w.heads, idx % w.heads
    Om, C = fitted_basis(w.replace(heads=w.heads))
    Om_s, C_s = Om[hs].astype(np.float64), C[hs].astype(np.float64)
    S = synth.initial_state(w.replace(batch=min(w.batch, 8)), 0)
    bsel = bs % S.shape[0]
    S0 = S[bsel, hs].astype(np.float64)
    toks, qs = [], []
    for t in range(w.buf_len):
        x = synth.step_inputs(w, 0, t)
        toks.append(tuple(x[n][bs, hs].astype(np.float64) for n in ("k", "v", "beta", "decay")))
        qs.append(x["q"][bs, hs].astype(np.float64))
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        orc.run_schedule(w.kind, S0, Om_s, C_s, toks, qs, w.buf_len)
        times.append(time.perf_counter() - t0)
    return times, len(bs) * w.buf_len, 1


# ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_mamba2")
    ap.add_argument("--layers", type=int, default=8, help="layer copies in the stack (distinct memory)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch")
    ap.add_argument("--buf-len", type=int, default=0)
    ap.add_argument("--rank", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-launch-events", action="store_true", help="do not bracket every launch with events")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-full-read", action="store_true")
    ap.add_argument("--skip-graph", action="store_true")
    ap.add_argument("--tune", default="", help="comma list key=value passed to sketchssm_tune")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    w = synth.CONFIGS[args.workload]
    if args.batch or args.buf_len or args.rank:
        w = w.replace(batch=args.batch or w.batch, buf_len=args.buf_len or w.buf_len, rank=args.rank or w.rank)
    cfg = {"workload": f"{w.name}: {w.kind} B{w.batch} H{w.heads} K{w.dk} V{w.dv} r{w.rank} L{w.buf_len} "
                       f"{w.io} I/O, fp32 state/sketch", "layers": args.layers,
           "schedule": "per layer and window: L-1 decode_step + 1 state_update(+sketch)"}

    # ----------------------------------------------------------------------------------------
    if args.impl == "reference":
        if rank != 0:
            return
        sample = 64
        times, head_steps, cores = oracle_window(w, sample, reps=args.warmup + args.steps)
        timed = times[args.warmup:]
        sec = sum(timed) / len(timed)
        value = head_steps / sec / w.heads
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                                 "sample": f"{sample} (batch, head) pairs x one window of {w.buf_len} tokens per step; "
                                           f"rate scaled to a layer of {w.heads} heads"},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    # ----------------------------------------------------------------------------------------
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    from paper_2609_33051_b200 import build as _build
    if not os.path.exists(_build.LIB_PATH):
        _build.build()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    stack = Stack(w, args.layers, local_rank)
    for kv in filter(None, args.tune.split(",")):
        k, v = kv.split("=")
        for m in stack.layers:
            m.tune(k, int(v))
    L, B, H = w.buf_len, w.batch, w.heads
    tokens_per_step = B * L * args.layers
    cfg.update({"device_bytes": stack.device_bytes(), "l2": "inputs larger than L2: every layer has its own state, "
                "sketch, ring and token tensors; %.1f GB touched between re-uses" % (stack.device_bytes() / 1e9),
                "per_kernel_timing": "second timed pass of the same launches with CUDA events around every launch "
                                     "(bracketing costs a few % of step time, so the headline pass has none)"})

    def timed_region(fn, steps, warmup, sampler=None):
        for _ in range(warmup):
            fn()
        barrier()
        if sampler is not None:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = None
        for _ in range(steps):
            out = fn()
        e1.record()
        barrier()
        clocks = sampler.stop() if sampler is not None else None
        ms = max_over_ranks(e0.elapsed_time(e1), dist)
        return ms / steps, out, clocks

    # ---- device-resident timing (the headline value): no events between launches ----
    launches_per_step = [0]

    def step():
        launches_per_step[0] = stack.run_window("sketch", None)

    ms_step, _, clocks = timed_region(step, args.steps, args.warmup, ClockSampler(local_rank))
    for m in stack.layers:
        m.check_status()
    value = job_value(tokens_per_step, world, ms_step)

    # ---- the same step captured once in a CUDA graph and replayed (no host work between launches) ----
    graph = None
    if not args.skip_graph:
        try:
            g = torch.cuda.CUDAGraph()
            cap_stream = torch.cuda.Stream()
            cap_stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(g, stream=cap_stream):
                stack.run_window("sketch", None)
            torch.cuda.current_stream().wait_stream(cap_stream)
            ms_graph, _, _ = timed_region(g.replay, args.steps, args.warmup)
            for m in stack.layers:
                m.check_status()
            graph = {"value": job_value(tokens_per_step, world, ms_graph), "unit": UNIT, "ms_per_step": ms_graph,
                     "what": "one window over all layers captured in a CUDA graph (programmatic dependent launch edges "
                             "included) and replayed"}
        except Exception as exc:      # capture is a convenience measurement: report why it is missing
            graph = {"unavailable": f"{type(exc).__name__}: {exc}"[:200]}

    # ---- the same region again with every launch bracketed by events: per-kernel durations ----
    events = None if args.no_launch_events else []
    ms_step_instrumented = None
    if events is not None:
        ms_step_instrumented, _, _ = timed_region(lambda: stack.run_window("sketch", events),
                                                  max(3, args.steps // 2), 1)

    # ---- per-kernel durations and roofline of the dominant kernel ----
    peak, peak_kind = measured_peaks()
    kern = {}
    if events:
        agg = {"decode": [0.0, 0, 0], "update": [0.0, 0, 0]}            # ms, launches, bytes
        for kind, t, a, b in events:
            agg[kind][0] += a.elapsed_time(b)
            agg[kind][1] += 1
            agg[kind][2] += (traffic.decode_bytes(w.kind, B, H, w.dk, w.dv, w.rank, t, w.io) if kind == "decode"
                             else traffic.update_bytes(w.kind, B, H, w.dk, w.dv, w.rank, t, w.io))
        for kind, (ms, n, by) in agg.items():
            if n:
                kern[kind] = {"launches": n, "avg_us": 1e3 * ms / n, "share": ms / (agg["decode"][0] + agg["update"][0]),
                              "algorithmic_bytes_per_launch": by / n, "achieved_gbs": by / (ms * 1e-3) / 1e9}
    # Back-to-back runs of one kernel between two events: the average launch duration as the stream sees it.
    # An event between two launches removes the programmatic dependent launch overlap, so the bracketed figures
    # above are the conservative ones; these are what a window actually pays per launch.
    b2b = {}
    if not args.no_launch_events:
        reps = max(3, args.steps // 4)
        ms_d, _, _ = timed_region(stack.run_decode_only, reps, 2)
        n_d = (L - 1) * args.layers
        by_d = sum(traffic.decode_bytes(w.kind, B, H, w.dk, w.dv, w.rank, t, w.io) for t in range(L - 1)) / (L - 1)
        b2b["decode"] = {"avg_us": 1e3 * ms_d / n_d, "achieved_gbs": by_d / (ms_d / n_d * 1e-3) / 1e9}
        ms_u, _, _ = timed_region(stack.run_update_only, reps, 2)
        by_u = traffic.update_bytes(w.kind, B, H, w.dk, w.dv, w.rank, L - 1, w.io)
        b2b["update"] = {"avg_us": 1e3 * ms_u / args.layers, "achieved_gbs": by_u / (ms_u / args.layers * 1e-3) / 1e9}
        stack.run_window("sketch", None)     # leave every layer at the start of a window again
        for k in b2b:
            if k in kern:
                kern[k]["back_to_back_avg_us"] = b2b[k]["avg_us"]
                kern[k]["back_to_back_achieved_gbs"] = b2b[k]["achieved_gbs"]
    dominant = max(kern, key=lambda k: kern[k]["share"]) if kern else None
    roofline = None
    if dominant:
        kname = "decode_kernel" if dominant == "decode" else "update_kernel"
        ach = b2b.get(dominant, {}).get("achieved_gbs", kern[dominant]["achieved_gbs"])
        roofline = {"bound": "hbm", "kernel": kname, "achieved": ach, "peak": peak,
                    "unit": "GB/s", "frac": ach / peak, "peak_source": peak_kind,
                    "traffic": ncu_traffic(kname, w.name, kern[dominant]["algorithmic_bytes_per_launch"]),
                    "algorithmic_bytes_per_launch": kern[dominant]["algorithmic_bytes_per_launch"],
                    "duration": "average over a run of back-to-back launches between two CUDA events "
                                "(programmatic dependent launch overlaps heads and tails of consecutive launches; in "
                                "this run the n = 0 launches, 1 of L-1, also request their sketch rows before the "
                                "dependency wait, which after a flush in a window they do not)",
                    "achieved_bracketed": kern[dominant]["achieved_gbs"],
                    "frac_bracketed": kern[dominant]["achieved_gbs"] / peak,
                    "frac_of_8TBs_nominal": ach / 8000.0}

    # ---- in-library full-read baseline (buffered replay that reads all of S every step) ----
    full = None
    if not args.skip_full_read:
        ms_full, _, _ = timed_region(lambda: stack.run_window("full_read", None), max(3, args.steps // 4), 3)
        full = {"value": world * tokens_per_step / (ms_full * 1e-3), "unit": UNIT, "ms_per_step": ms_full,
                "what": "sketchssm_full_read_decode x (L-1) + sketchssm_state_update(NO_SKETCH) per layer and window",
                "sketch_speedup": ms_full / ms_step}
        # the execution without a buffer: full state read + write per token (what the paper calls the standard decode)
        ms_std, _, _ = timed_region(lambda: stack.run_window("standard", None), max(3, args.steps // 4), 3)
        full["standard"] = {"value": world * tokens_per_step / (ms_std * 1e-3), "unit": UNIT, "ms_per_step": ms_std,
                            "what": "sketchssm_state_update(n_before = 0, token, NO_SKETCH) at every step",
                            "sketch_speedup": ms_std / ms_step}
        stack.run_window("sketch", None)     # leave a fresh sketch behind

    # ---- end to end through the C ABI with host buffers ----
    e2e = None
    if not args.skip_e2e:
        stack.setup_host()
        bytes_io = [0, 0]

        def host_step():
            bytes_io[0], bytes_io[1] = stack.run_window_host()

        ms_e2e, _, _ = timed_region(host_step, args.e2e_steps, 3)
        e2e = {"value": world * tokens_per_step / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": bytes_io[0],
               "d2h_bytes_per_step": bytes_io[1], "ms_per_step": ms_e2e, "steps": args.e2e_steps,
               "what": "sketchssm_step_host per layer-step: pinned host q,k,v,beta,decay -> device, kernel, o -> host; "
                       "layer-steps alternate between two streams so uploads overlap kernels and downloads"}
    for m in stack.layers:
        m.check_status()

    # ---- CPU oracle on a bounded sample (rank 0, N = 1) ----
    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        probe, head_steps, cores = oracle_window(w, 512, reps=1)
        sample = int(min(w.batch * w.heads, max(512, 512 * 12.0 / max(probe[0], 1e-3))))
        times, head_steps, cores = oracle_window(w, sample, reps=1)
        cpu = {"value": head_steps / times[0] / H, "unit": UNIT, "cores": cores, "kind": "oracle",
               "seconds": times[0],
               "sample": f"{sample} (batch, head) pairs x one window of {L} tokens (L-1 decode steps + 1 state "
                         f"update), fp64 NumPy; rate scaled to a layer of {H} heads"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg, "clocks": clocks,
                "e2e": e2e, "gpu_launches": launches_per_step[0] * args.steps, "roofline": roofline,
                "kernels": kern, "ms_per_step_with_launch_events": ms_step_instrumented, "full_read_baseline": full, "graph_replay": graph, "cpu_baseline": cpu,
                "per_gpu_heads": B * H}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
