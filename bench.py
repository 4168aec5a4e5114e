#!/usr/bin/env python
"""Benchmark of the SketchSSM decode hot path on B200.

One *step* is one window of Algorithm 1 over a stack of layers: for every layer, L-1 non-flush decode
steps (sketchssm_decode_step) and one flush (sketchssm_state_update with the sketch refresh), over the
whole batch of the workload.  The metric is decode tokens/s per layer:  B * L * n_layers / step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME] [--no-sweep]

The default workload is the largest single-GPU point of the large-batch sweep (Mamba-2 stack of 48 layers,
batch 2048, L = 16, r = 16).  The 48 logical layers are mapped round-robin onto `n_phys` physical layer slots
(distinct state, sketch, ring and token tensors each), as many as fit the memory budget; `n_phys` is printed.
Unless --no-sweep is given, the same JSON line also carries, under "sweep", the Mamba-2, GDN and KDA layer
workloads and every other (batch, L, r) point of the sweep, each with its own clock record, and under
"sustained" a seconds-long repetition of the headline step with per-step times binned by SM clock.

Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed on a bounded sample of the
same workload instead.  Under torchrun (N > 1) every rank runs the same per-GPU workload (weak scaling,
no data-path collective: heads are independent); the time is the max over ranks.  `--gpus N` without a
torchrun environment re-launches itself under torch.distributed.run with N ranks.
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

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_33051_b200 import synth, traffic  # noqa: E402

METRIC = "decode tokens/s per layer"
UNIT = "tokens/s/layer"
NOMINAL_HBM_GBS = 8000.0
INPUT_BATCH = 64            # token inputs are generated for this many batch entries and repeated over the batch
LOGICAL_LAYERS = 48         # depth of the large-batch sweep's stack
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/:
# kernel -> (captured bytes, algorithmic bytes of the captured launches).  The captures are of the Mamba-2 layer
# (batch 256); per-head traffic does not depend on the batch, so the bench line scales the captured figure to its own
# launch by the algorithmic bytes.
NCU_TRAFFIC_CAPTURES = {
    ("decode_kernel", "mamba2"): (117.46e6, float(traffic.decode_bytes("mamba2", 256, 64, 128, 64, 16, 5, "bf16"))),
    ("update_tc_ws_mamba2_kernel", "mamba2"): (1194.16e6, float(traffic.update_bytes("mamba2", 256, 64, 128, 64, 16, 15, "bf16"))),
}


def ncu_traffic(kernel: str, kind: str, algorithmic_bytes_per_launch: float):
    cap = NCU_TRAFFIC_CAPTURES.get((kernel, kind))
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


def physical_layers(per_layer_bytes: int, budget_bytes: int, logical: int) -> int:
    """Physical layer slots the logical layers are mapped onto round-robin: as many as fit the budget."""
    return int(max(1, min(logical, budget_bytes // max(per_layer_bytes, 1))))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def update_kernel_name(w: synth.Workload) -> str:
    """The flush kernel the library's default dispatch runs for a workload (the names ncu lists)."""
    if w.io == "bf16" and w.dk == 128:
        if w.kind == "mamba2":
            return "update_tc_ws_mamba2_kernel" if w.rank <= 32 else "update_tc_mamba2_kernel"
        if w.kind == "gdn" and w.dv == 128 and w.rank <= 16:
            return "update_tc_ws_gdn_kernel"
        if w.kind == "kda" and w.dv == 128 and w.rank <= 16:
            return "update_tc_ws_kda_kernel"
    return "update_kernel"


# ---------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, device_index: int, period_s: float = 0.01):
        self.samples, self.stamps, self.reasons = [], [], set()
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
                self.stamps.append(time.perf_counter())
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
        return self

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
_BASIS_CACHE, _INPUT_CACHE = {}, {}


def fitted_basis(w: synth.Workload):
    """Omega [H,K,r], C [H,r,K] float32 from the workload's calibration queries (E_0 = I)."""
    key = (w.seed, w.kind, w.heads, w.dk, w.rank, w.basis)
    if key not in _BASIS_CACHE:
        _BASIS_CACHE[key] = _fit_basis(w)
    return _BASIS_CACHE[key]


def step_inputs_cached(wi: synth.Workload, t: int):
    """synth.step_inputs of layer 0 (they do not depend on the window length or the rank: sweep points share them)."""
    key = (wi.seed, wi.kind, wi.batch, wi.heads, wi.dk, wi.dv, wi.io, t)
    if key not in _INPUT_CACHE:
        _INPUT_CACHE[key] = synth.step_inputs(wi, 0, t)
    return _INPUT_CACHE[key]


def _fit_basis(w: synth.Workload):
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


def input_workload(w: synth.Workload) -> synth.Workload:
    """The workload the token inputs are generated for: the first INPUT_BATCH batch entries (repeated over the batch)."""
    return w if w.batch <= INPUT_BATCH or w.batch % INPUT_BATCH else w.replace(batch=INPUT_BATCH)


def layer_bytes(w: synth.Workload, own_inputs: bool = True) -> int:
    """Device bytes of one physical layer slot (state, sketch, ring and, if it has its own, one window of tokens)."""
    bh = w.batch * w.heads
    per = bh * (w.dk * w.dv * 4 + w.rank * w.dv * 4 + w.buf_len * traffic.slot_bytes(w.kind, w.dk, w.dv, w.io))
    per += bh * (w.dk + w.buf_len) * 4                       # work
    if own_inputs:
        per += w.buf_len * bh * traffic.token_bytes(w.kind, w.dk, w.dv, w.io)
    return per + bh * w.dv * 4                               # output


class Stack:
    """`logical` layers of one workload on one GPU, mapped round-robin onto `n_phys` physical layer slots, with one
    window of device-resident inputs per slot."""

    def __init__(self, w: synth.Workload, n_phys: int, logical: int, device: int, coef=None, sketch="f32", erase=False):
        """coef: None (fixed offline map) or "pivot" / "ridge" (state-dependent map rebuilt by every flush);
        sketch: storage type of U and C; erase: decode through projected erase vectors (GDN / KDA)."""
        from paper_2609_33051_b200.binding import SketchSSM
        self.w, self.n_phys, self.logical, self.device = w, n_phys, logical, device
        self.coef, self.sketch, self.erase = coef, sketch, erase
        dev = torch.device("cuda", device)
        Om, C = fitted_basis(w)
        wi = input_workload(w)
        reps = w.batch // wi.batch
        dec_io = w.io if w.kind == "kda" else "f32"
        window = []
        for t in range(w.buf_len):
            x = step_inputs_cached(wi, t)
            tok = dict(q=synth.to_torch(x["q"], w.io, dev), k=synth.to_torch(x["k"], w.io, dev),
                       v=synth.to_torch(x["v"], w.io, dev), beta=synth.to_torch(x["beta"], "f32", dev),
                       decay=synth.to_torch(x["decay"], dec_io, dev))
            if reps > 1:
                tok = {k: v.repeat(reps, *([1] * (v.dim() - 1))).contiguous() for k, v in tok.items()}
            window.append(tok)
        self.host_window = None
        self.layers, self.inputs, self.outs = [], [], []
        gen = torch.Generator(device=dev)
        Om_t, C_t = torch.from_numpy(Om), torch.from_numpy(C)
        for li in range(n_phys):
            m = SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, out="f32", device=device,
                          coef_per_seq=coef is not None, coef_pivots=4 if coef == "pivot" else 0, sketch=sketch,
                          erase_factors=erase)
            gen.manual_seed(w.seed * 1000 + li)
            m.state.normal_(0.0, w.state_std, generator=gen)          # S_init ~ N(0, 0.02^2), drawn on the device
            m.omega.copy_(Om_t)
            if coef is None:
                m.coef.copy_(C_t)
            m.state_update(0)
            self.layers.append(m)
            # every slot gets its own copy of the window so that no input is served from L2 across layers
            self.inputs.append(window if li == 0 else [{k: v.clone() for k, v in tok.items()} for tok in window])
            self.outs.append(m.new_output())
        self.window0 = window
        torch.cuda.synchronize(dev)

    def close(self):
        for m in self.layers:
            m.close()
        self.layers, self.inputs, self.outs, self.window0 = [], [], [], None
        self.host_window = None
        torch.cuda.empty_cache()

    def device_bytes(self) -> int:
        m = self.layers[0]
        per = m.state.numel() * 4 + m.sketch.numel() * 4 + m.ring.numel()
        per += sum(v.numel() * v.element_size() for tok in self.inputs[0] for v in tok.values())
        return per * self.n_phys

    def run_window(self, mode: str = "sketch", events=None):
        """One step: L tokens through every logical layer.  mode: "sketch" (decode_step + state_update),
        "full_read" (full_read_decode + state_update without the sketch write) or "standard" (no buffering: the
        state is read, updated with the one token and written back at every step; the flush kernel with an empty
        ring and no sketch).  `events`, if given, receives (kind, n_before, start_event, end_event) per launch."""
        from paper_2609_33051_b200.binding import NO_SKETCH
        L = self.w.buf_len
        launches = 0
        for t in range(L):
            for l in range(self.logical):
                li = l % self.n_phys
                m, tok, o = self.layers[li], self.inputs[li][t], self.outs[li]
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

    def run_decode_only(self, mode: str = "sketch"):
        """The L-1 decode steps of a window over every logical layer, back to back, no flush (the ring slots are
        simply rewritten with the same tokens on the next pass)."""
        L = self.w.buf_len
        for t in range(L - 1):
            for l in range(self.logical):
                li = l % self.n_phys
                m, tok = self.layers[li], self.inputs[li][t]
                if mode == "sketch":
                    m.decode_step(t, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], self.outs[li])
                else:
                    m.full_read_decode(t, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], self.outs[li])
        return (L - 1) * self.logical

    def run_update_only(self, flags: int = 0):
        """One flush per logical layer, back to back (full ring: n_before = L-1 plus the token)."""
        L = self.w.buf_len
        for l in range(self.logical):
            li = l % self.n_phys
            m, tok = self.layers[li], self.inputs[li][L - 1]
            m.state_update(L - 1, tok["q"], tok["k"], tok["v"], tok["beta"], tok["decay"], self.outs[li], flags=flags)
        return self.logical

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
        of the previous one; a physical layer always uses the same stream, so its own steps stay ordered."""
        from paper_2609_33051_b200 import binding
        L = self.w.buf_len
        h2d = d2h = 0
        cur = torch.cuda.current_stream()
        for s in self.side_streams:
            s.wait_stream(cur)
        for t in range(L):
            hb = self.host_window[t]
            for l in range(self.logical):
                li = l % self.n_phys
                m = self.layers[li]
                op = binding.OP_DECODE if t < L - 1 else binding.OP_UPDATE
                host = dict(hb)
                host["out"] = self.host_out[li & 1]
                m.step_host(op, t, host, self.staging[li & 1], stream=self.side_streams[li & 1])
                h2d += sum(hb[k].numel() * hb[k].element_size() for k in ("q", "k", "v", "beta", "decay"))
                d2h += host["out"].numel() * host["out"].element_size()
        for s in self.side_streams:
            cur.wait_stream(s)
        return h2d, d2h


def make_stack(w: synth.Workload, budget_gb: float, logical: int, device: int, coef=None, sketch="f32", erase=False) -> Stack:
    per = layer_bytes(w) + (w.batch * w.heads * w.rank * w.dk * (2 if sketch == "bf16" else 4) if coef else 0)
    per += w.batch * w.heads * w.buf_len * w.rank * 4 if erase else 0
    n_phys = physical_layers(per, int(budget_gb * 1e9), logical)
    return Stack(w, n_phys, logical, device, coef=coef, sketch=sketch, erase=erase)


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------
CPU_SAMPLE_BATCH = 32       # batch entries of the sample the CPU oracle is timed on (all heads of each)


def oracle_sample(w: synth.Workload):
    """The bounded sample both CPU legs time: every head of the first CPU_SAMPLE_BATCH batch entries, one window."""
    wi = w if w.batch <= CPU_SAMPLE_BATCH else w.replace(batch=CPU_SAMPLE_BATCH)
    return wi, f"{wi.batch * wi.heads} (batch, head) pairs (the first {wi.batch} batch entries x {wi.heads} heads) x one " \
               f"window of {w.buf_len} tokens (L-1 decode steps + 1 state update), fp64 NumPy, one core; rate scaled to " \
               f"a layer of {w.heads} heads"


def oracle_window(w: synth.Workload, reps: int = 1):
    """Time the oracle, as it stands, on one window of the sample.  Returns (seconds per rep, head-steps per window, threads)."""
    from oracle import sketchssm_oracle as orc
    wi, _ = oracle_sample(w)
    Om, C = fitted_basis(wi)
    Om_s, C_s = Om.astype(np.float64)[None], C.astype(np.float64)[None]
    S0 = synth.initial_state(wi, 0).astype(np.float64)
    toks, qs = [], []
    for t in range(w.buf_len):
        x = step_inputs_cached(wi, t)
        toks.append(tuple(x[n].astype(np.float64) for n in ("k", "v", "beta", "decay")))
        qs.append(x["q"].astype(np.float64))
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        orc.run_schedule(w.kind, S0, Om_s, C_s, toks, qs, w.buf_len)
        times.append(time.perf_counter() - t0)
    return times, wi.batch * wi.heads * w.buf_len, 1


# ---------------------------------------------------------------------------------------------
# timing
# ---------------------------------------------------------------------------------------------
class Timer:
    def __init__(self, dist, device_index):
        self.dist, self.device_index = dist, device_index

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()

    def region(self, fn, steps, warmup, sample_clocks=False):
        """W untimed calls, then K timed calls bracketed by barrier + synchronize; device time by CUDA events on the
        launching stream, max over ranks.  Returns (ms per call, last result, clock record or None)."""
        for _ in range(warmup):
            fn()
        self.barrier()
        sampler = ClockSampler(self.device_index).start() if sample_clocks else None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = None
        for _ in range(steps):
            out = fn()
        e1.record()
        self.barrier()
        clocks = sampler.stop() if sampler is not None else None
        ms = max_over_ranks(e0.elapsed_time(e1), self.dist)
        return ms / steps, out, clocks


def kernel_figures(w, stack, timer, ms_window, reps, peak):
    """Back-to-back launch durations of the two kernels, the in-window decode duration derived from the window time,
    and the bandwidth fractions.  `ms_window` is the time of one window over all logical layers."""
    L, B, H = w.buf_len, w.batch, w.heads
    n_log = stack.logical
    tkw = dict(sketch_bytes=2 if stack.sketch == "bf16" else 4, coef_per_seq=stack.coef is not None)
    dkw = dict(tkw, erase_factors=stack.erase)
    ms_d, _, _ = timer.region(stack.run_decode_only, reps, 1)
    us_dec_b2b = 1e3 * ms_d / ((L - 1) * n_log)
    ms_u, _, _ = timer.region(stack.run_update_only, reps, 1)
    us_upd = 1e3 * ms_u / n_log
    stack.run_window("sketch", None)     # leave every layer at the start of a window again
    by_d = sum(traffic.decode_bytes(w.kind, B, H, w.dk, w.dv, w.rank, t, w.io, **dkw) for t in range(L - 1)) / (L - 1)
    by_u = traffic.update_bytes(w.kind, B, H, w.dk, w.dv, w.rank, L - 1, w.io, **tkw)
    # what a decode launch costs inside the window: the window minus the flush, over its L-1 decode launches
    us_dec_win = max((1e3 * ms_window / n_log - us_upd) / (L - 1), 1e-3)
    gbs = lambda by, us: by / (us * 1e-6) / 1e9
    return {
        "decode": {"kernel": "decode_kernel", "algorithmic_bytes_per_launch": by_d,
                   "in_window_us": us_dec_win, "in_window_gbs": gbs(by_d, us_dec_win),
                   "frac_of_measured": gbs(by_d, us_dec_win) / peak, "frac_of_8TBs_nominal": gbs(by_d, us_dec_win) / NOMINAL_HBM_GBS,
                   "back_to_back_us": us_dec_b2b, "back_to_back_gbs": gbs(by_d, us_dec_b2b),
                   "back_to_back_frac_of_measured": gbs(by_d, us_dec_b2b) / peak},
        "update": {"kernel": update_kernel_name(w), "algorithmic_bytes_per_launch": by_u,
                   "back_to_back_us": us_upd, "back_to_back_gbs": gbs(by_u, us_upd),
                   "frac_of_measured": gbs(by_u, us_upd) / peak, "frac_of_8TBs_nominal": gbs(by_u, us_upd) / NOMINAL_HBM_GBS},
        "decode_share_of_window": (L - 1) * us_dec_win / (1e3 * ms_window / n_log),
    }


def measure_point(w, budget_gb, logical, device, timer, peak, min_seconds=0.25, coef=None, sketch="f32", erase=False):
    """One sweep record: the sketch window, the full-read window, per-kernel figures, byte accounting, clocks."""
    stack = make_stack(w, budget_gb, logical, device, coef=coef, sketch=sketch, erase=erase)
    try:
        L, B, H = w.buf_len, w.batch, w.heads
        tokens = B * L * logical
        t0 = time.perf_counter()
        stack.run_window("sketch", None)
        torch.cuda.synchronize()
        est = max(time.perf_counter() - t0, 1e-4)
        steps = int(min(50, max(2, min_seconds / est)))
        sampler = ClockSampler(device).start()
        ms, _, _ = timer.region(lambda: stack.run_window("sketch", None), steps, 3)
        figs = kernel_figures(w, stack, timer, ms, max(2, steps // 2), peak)
        ms_full, _, _ = timer.region(lambda: stack.run_window("full_read", None), max(2, steps // 3), 3)
        stack.run_window("sketch", None)
        clocks = sampler.stop()
        for m in stack.layers:
            m.check_status()
        mean_n = (L - 2) / 2.0
        tkw = dict(sketch_bytes=2 if sketch == "bf16" else 4, coef_per_seq=coef is not None)
        dec_b = traffic.decode_bytes(w.kind, 1, 1, w.dk, w.dv, w.rank, 0, w.io, erase_factors=erase, **tkw)
        if coef is None:
            dec_b -= w.rank * w.dk * tkw["sketch_bytes"]          # the shared map is read once per launch, not per head
        from paper_2609_33051_b200.binding import NO_SKETCH
        ms_u0, _, _ = timer.region(lambda: stack.run_update_only(NO_SKETCH), max(2, steps // 2), 1)
        stack.run_window("sketch", None)
        full_b = traffic.decode_bytes(w.kind, 1, 1, w.dk, w.dv, w.rank, 0, w.io, full_read=True)
        slot = traffic.slot_bytes(w.kind, w.dk, w.dv, w.io)
        return {
            "workload": f"{w.name}: {w.kind} B{B} H{H} K{w.dk} V{w.dv} r{w.rank} L{L}", "logical_layers": logical,
            "coefficient_map": {None: "fixed offline map [H][r][K]", "pivot": "state-dependent, P = 4 approximation, lambda 0.1, "
                                "rebuilt by every flush [B][H][r][K]", "ridge": "state-dependent, exact ridge solve, lambda 0.1"}[coef],
            "sketch_storage": sketch,
            "erase_factors": bool(erase),
            "flush_without_sketch_us": 1e3 * ms_u0 / logical,
            "sketch_and_map_overhead_on_flush": figs["update"]["back_to_back_us"] / (1e3 * ms_u0 / logical) - 1.0,
            "n_phys": stack.n_phys, "device_bytes": stack.device_bytes(), "steps": steps,
            "value": tokens / (ms * 1e-3), "unit": UNIT, "ms_per_window_all_layers": ms,
            "decode_in_window_us": figs["decode"]["in_window_us"],
            "decode_frac_of_measured": figs["decode"]["frac_of_measured"],
            "decode_frac_of_8TBs_nominal": figs["decode"]["frac_of_8TBs_nominal"],
            "decode_back_to_back_us": figs["decode"]["back_to_back_us"],
            "decode_back_to_back_frac_of_measured": figs["decode"]["back_to_back_frac_of_measured"],
            "update_kernel": figs["update"]["kernel"], "update_us": figs["update"]["back_to_back_us"],
            "update_frac_of_measured": figs["update"]["frac_of_measured"],
            "update_frac_of_8TBs_nominal": figs["update"]["frac_of_8TBs_nominal"],
            "full_read": {"value": tokens / (ms_full * 1e-3), "unit": UNIT, "sketch_speedup": ms_full / ms},
            "decode_bytes_per_token_head": dec_b + mean_n * (slot + (w.rank * 4 if erase else 0)), "full_read_bytes_per_token_head": full_b + mean_n * slot,
            "state_read_ratio_dk_over_r": w.dk / w.rank,
            "clocks": clocks,
        }
    finally:
        stack.close()


def sustained_leg(stack, timer, device, seconds, tokens_per_step):
    """The headline step repeated for `seconds`, every step timed by its own pair of events, with the SM clock sampled
    alongside; steps are binned by the median clock seen while they ran (time x MHz shows what scales with the clock)."""
    stack.run_window("sketch", None)
    timer.barrier()
    sampler = ClockSampler(device, period_s=0.005).start()
    evs, stamps = [], []
    t_start = time.perf_counter()
    while time.perf_counter() - t_start < seconds or len(evs) < 3:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0 = time.perf_counter()
        e0.record()
        stack.run_window("sketch", None)
        e1.record()
        e1.synchronize()
        stamps.append((h0, time.perf_counter()))
        evs.append((e0, e1))
    timer.barrier()
    clocks = sampler.stop()
    ms = [a.elapsed_time(b) for a, b in evs]
    per_step_mhz = []
    for (h0, h1) in stamps:
        inside = [c for c, ts in zip(sampler.samples, sampler.stamps) if h0 <= ts <= h1]
        per_step_mhz.append(statistics.median(inside) if inside else None)
    bins = {}
    for t_ms, mhz in zip(ms, per_step_mhz):
        if mhz is not None:
            bins.setdefault(int(round(mhz / 50.0) * 50), []).append(t_ms)
    total_ms = sum(ms)
    return {"seconds": total_ms * 1e-3, "steps": len(ms), "value": tokens_per_step * len(ms) / (total_ms * 1e-3), "unit": UNIT,
            "ms_per_step_first": ms[0], "ms_per_step_median": statistics.median(ms), "ms_per_step_last": ms[-1],
            "by_sm_mhz": {str(k): {"steps": len(v), "ms_per_step": statistics.mean(v), "ms_x_mhz": statistics.mean(v) * k}
                          for k, v in sorted(bins.items())},
            "clocks": clocks}


# ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5_B2048_L16_r16",
                    help="c5_B<batch>_L<L>_r<r> (a point of the 48-layer Mamba-2 sweep) or c2_mamba2 / c3_gdn / c4_kda")
    ap.add_argument("--layers", type=int, default=0, help="logical layers in the stack (default 48 for sweep points, "
                                                          "else as many distinct copies as fit the budget, at most 8)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (small cases for profiler captures)")
    ap.add_argument("--budget-gb", type=float, default=100.0, help="device memory for the headline stack's layer slots")
    ap.add_argument("--sweep-budget-gb", type=float, default=40.0, help="device memory per sweep point")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustained-seconds", type=float, default=3.0)
    ap.add_argument("--no-sweep", action="store_true", help="headline workload only")
    ap.add_argument("--no-launch-events", action="store_true", help="do not bracket every launch with events")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-full-read", action="store_true")
    ap.add_argument("--skip-graph", action="store_true")
    ap.add_argument("--tune", default="", help="comma list key=value passed to sketchssm_tune")
    ap.add_argument("--coef", default="fixed", choices=["fixed", "pivot", "ridge"], help="coefficient map of the headline stack")
    ap.add_argument("--sketch", default="f32", choices=["f32", "bf16"], help="storage type of U and C of the headline stack")
    ap.add_argument("--erase-factors", action="store_true", help="GDN / KDA workloads: decode through projected erase vectors (Eq. 44-45)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.workload.startswith("c5_B"):
        bb, ll, rr = (int(x[1:]) for x in args.workload.split("_")[1:4])
        w = synth.sweep_point(bb, ll, rr)
        logical = args.layers or LOGICAL_LAYERS
    else:
        w = synth.CONFIGS[args.workload]
        logical = args.layers or min(8, physical_layers(layer_bytes(w), int(args.budget_gb * 1e9), 8))
    if args.batch:
        w = w.replace(batch=args.batch)
        logical = args.layers or logical
    cfg = {"workload": f"{w.name}: {w.kind} B{w.batch} H{w.heads} K{w.dk} V{w.dv} r{w.rank} L{w.buf_len} "
                       f"{w.io} I/O, fp32 state/sketch", "layers": logical,
           "schedule": "per layer and window: L-1 decode_step + 1 state_update(+sketch)"}

    # ----------------------------------------------------------------------------------------
    if args.impl == "reference":
        if rank != 0:
            return
        _, sample_text = oracle_sample(w)
        times, head_steps, cores = oracle_window(w, reps=args.warmup + args.steps)
        timed = times[args.warmup:]
        sec = sum(timed) / len(timed)
        value = head_steps / sec / w.heads
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample_text},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    # ----------------------------------------------------------------------------------------
    if world == 1 and args.gpus > 1:
        # asked for N GPUs outside torchrun: start the N ranks ourselves (or refuse), never measure one GPU as N
        have = torch.cuda.device_count()
        if have < args.gpus:
            sys.exit(f"bench.py: --gpus {args.gpus} asked for but {have} CUDA device(s) visible")
        port = 29500 + (os.getpid() % 2000)
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
        sys.exit(subprocess.call(cmd))

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    from paper_2609_33051_b200 import build as _build
    if not os.path.exists(_build.LIB_PATH):
        _build.build()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    timer = Timer(dist, local_rank)
    peak, peak_kind = measured_peaks()

    stack = make_stack(w, args.budget_gb, logical, local_rank, coef=None if args.coef == "fixed" else args.coef, sketch=args.sketch,
                       erase=args.erase_factors)
    for kv in filter(None, args.tune.split(",")):
        k, v = kv.split("=")
        for m in stack.layers:
            m.tune(k, int(v))
    L, B, H = w.buf_len, w.batch, w.heads
    tokens_per_step = B * L * logical
    details = {"n_phys": stack.n_phys, "logical_layers": logical, "device_bytes": stack.device_bytes(),
               "layer_mapping": "logical layer l runs on physical slot l mod n_phys (distinct state, sketch, ring, token "
                                "and output tensors per slot)",
               "l2": "inputs larger than L2: %.1f GB of slot data touched between re-uses of a slot" % (stack.device_bytes() / 1e9),
               "inputs": f"token inputs generated for {input_workload(w).batch} batch entries and repeated over the batch; "
                         "initial states drawn on the device, N(0, 0.02^2), distinct per entry and slot",
               "per_kernel_timing": "kernels[..].back_to_back_us: runs of one kernel between two CUDA events; "
                                    "kernels.decode.in_window_us: (window time per layer - flush) / (L-1); bracketed_us: "
                                    "every launch between its own pair of events (removes the launch overlap)"}

    # ---- device-resident timing (the headline value): no events between launches ----
    launches_per_step = [0]

    def step():
        launches_per_step[0] = stack.run_window("sketch", None)

    ms_step, _, clocks = timer.region(step, args.steps, args.warmup, sample_clocks=True)
    for m in stack.layers:
        m.check_status()
    value = job_value(tokens_per_step, world, ms_step)

    # ---- per-kernel durations and the roofline of the dominant kernel ----
    kern = kernel_figures(w, stack, timer, ms_step, max(2, args.steps // 4), peak)
    ms_step_instrumented = None
    if not args.no_launch_events:
        events = []
        ms_step_instrumented, _, _ = timer.region(lambda: stack.run_window("sketch", events), 2, 1)
        agg = {"decode": [0.0, 0], "update": [0.0, 0]}
        for kind, t, a, b in events:
            agg[kind][0] += a.elapsed_time(b)
            agg[kind][1] += 1
        tot = agg["decode"][0] + agg["update"][0]
        for kind, (ms, n) in agg.items():
            if n:
                kern[kind]["bracketed_us"] = 1e3 * ms / n
                kern[kind]["bracketed_share"] = ms / tot
    dominant = "decode" if kern["decode_share_of_window"] >= 0.5 else "update"
    kd = kern[dominant]
    ach = kd["in_window_gbs"] if dominant == "decode" else kd["back_to_back_gbs"]
    roofline = {"bound": "hbm", "kernel": kd["kernel"], "achieved": ach, "peak": peak, "unit": "GB/s",
                "frac": ach / peak, "peak_source": peak_kind,
                "traffic": ncu_traffic(kd["kernel"], w.kind, kd["algorithmic_bytes_per_launch"]),
                "algorithmic_bytes_per_launch": kd["algorithmic_bytes_per_launch"],
                "share_of_window": kern["decode_share_of_window"] if dominant == "decode" else 1.0 - kern["decode_share_of_window"],
                "duration": ("in-window launch duration: (window time per layer - flush duration) / (L-1 decode launches), "
                             "from the headline timed region" if dominant == "decode" else
                             "average over a run of back-to-back launches between two CUDA events"),
                "achieved_back_to_back": kd["back_to_back_gbs"], "frac_back_to_back": kd["back_to_back_gbs"] / peak,
                "frac_of_8TBs_nominal": ach / NOMINAL_HBM_GBS}

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
            ms_graph, _, _ = timer.region(g.replay, max(3, args.steps // 2), 3)
            for m in stack.layers:
                m.check_status()
            graph = {"value": job_value(tokens_per_step, world, ms_graph), "unit": UNIT, "ms_per_step": ms_graph,
                     "what": "one window over all layers captured in a CUDA graph (programmatic dependent launch edges "
                             "included) and replayed"}
            del g
        except Exception as exc:      # capture is a convenience measurement: report why it is missing
            graph = {"unavailable": f"{type(exc).__name__}: {exc}"[:200]}

    # ---- sustained: the headline step for seconds, binned by clock ----
    sustained = None
    if args.sustained_seconds > 0:
        sustained = sustained_leg(stack, timer, local_rank, args.sustained_seconds, world * tokens_per_step)

    # ---- in-library full-read baseline (buffered replay that reads all of S every step) ----
    full = None
    if not args.skip_full_read:
        n_b = max(2, args.steps // 6)
        ms_full, _, _ = timer.region(lambda: stack.run_window("full_read", None), n_b, 3)
        full = {"value": world * tokens_per_step / (ms_full * 1e-3), "unit": UNIT, "ms_per_step": ms_full,
                "what": "sketchssm_full_read_decode x (L-1) + sketchssm_state_update(NO_SKETCH) per layer and window",
                "sketch_speedup": ms_full / ms_step}
        # the same flush without the sketch write and the exact-output column: the sketch's cost on the flush
        from paper_2609_33051_b200.binding import NO_SKETCH
        ms_u0, _, _ = timer.region(lambda: stack.run_update_only(NO_SKETCH), n_b, 2)
        full["flush_without_sketch_us"] = 1e3 * ms_u0 / logical
        full["sketch_write_overhead"] = kern["update"]["back_to_back_us"] / (1e3 * ms_u0 / logical) - 1.0
        # the execution without a buffer: full state read + write per token (what the paper calls the standard decode)
        ms_std, _, _ = timer.region(lambda: stack.run_window("standard", None), n_b, 3)
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

        ms_e2e, _, _ = timer.region(host_step, args.e2e_steps, 3)
        e2e = {"value": world * tokens_per_step / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": bytes_io[0],
               "d2h_bytes_per_step": bytes_io[1], "ms_per_step": ms_e2e, "steps": args.e2e_steps,
               "what": "sketchssm_step_host per layer-step: pinned host q,k,v,beta,decay -> device, kernel, o -> host; "
                       "layer-steps alternate between two streams so uploads overlap kernels and downloads"}
    for m in stack.layers:
        m.check_status()
    stack.close()
    del stack

    # ---- the other workloads: Mamba-2 / GDN / KDA layers and every other point of the sweep ----
    sweep = None
    if not args.no_sweep and world == 1:
        sweep = []
        for name in ("c2_mamba2", "c3_gdn", "c4_kda"):
            ww = synth.CONFIGS[name]
            sweep.append(measure_point(ww, args.sweep_budget_gb, 8, local_rank, timer, peak))
        for bb in synth.SWEEP_BATCH:
            for ll in synth.SWEEP_BUF_LEN:
                for rr in synth.SWEEP_RANK:
                    ww = synth.sweep_point(bb, ll, rr)
                    if ww.name == w.name:
                        continue
                    sweep.append(measure_point(ww, args.sweep_budget_gb, LOGICAL_LAYERS, local_rank, timer, peak))

    # ---- the headline workload in the paper's own configuration of the method: state-dependent coefficient map (P = 4),
    # and bfloat16 storage of the sketch; and the KDA layer with the tensor-core flush ----
    variants = None
    if not args.no_sweep and world == 1:
        variants = [measure_point(w, args.sweep_budget_gb, logical, local_rank, timer, peak, coef="pivot"),
                    measure_point(w, args.sweep_budget_gb, logical, local_rank, timer, peak, sketch="bf16"),
                    measure_point(w, args.sweep_budget_gb, logical, local_rank, timer, peak, coef="pivot", sketch="bf16"),
                    measure_point(synth.CONFIGS["c3_gdn"], args.sweep_budget_gb, 8, local_rank, timer, peak, coef="pivot"),
                    measure_point(synth.CONFIGS["c3_gdn"], args.sweep_budget_gb, 8, local_rank, timer, peak, erase=True),
                    measure_point(synth.CONFIGS["c4_kda"], args.sweep_budget_gb, 8, local_rank, timer, peak, erase=True),
                    measure_point(synth.CONFIGS["c3_gdn"], args.sweep_budget_gb, 8, local_rank, timer, peak, coef="pivot",
                                  sketch="bf16", erase=True)]

    # ---- CPU oracle on a bounded sample (rank 0, N = 1) ----
    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        _, sample_text = oracle_sample(w)
        times, head_steps, cores = oracle_window(w, reps=3)
        sec = statistics.median(times)
        cpu = {"value": head_steps / sec / H, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": sum(times),
               "sample": sample_text + "; median of 3 repetitions"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg, "details": details,
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step[0] * args.steps, "roofline": roofline,
                "kernels": kern, "ms_per_step_with_launch_events": ms_step_instrumented, "full_read_baseline": full,
                "graph_replay": graph, "sustained": sustained, "cpu_baseline": cpu, "per_gpu_heads": B * H,
                "sweep": sweep, "variants": variants}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
