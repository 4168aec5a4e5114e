"""Shared test harness: drives the CUDA library and the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import sketchssm_oracle as orc
from paper_2609_33051_b200 import synth


def basis_for(w: synth.Workload, layer: int = 0):
    """Omega [H,K,r] and C [H,r,K] (float32) for a workload: the seeded QR basis with C = Omega^T, or the
    oracle's offline fit (Appendix A.1, Eq. 10) on the workload's calibration queries with E_0 = I."""
    if w.basis == "qr":
        Om = synth.qr_basis(w, layer)
        return Om, np.ascontiguousarray(np.swapaxes(Om, 1, 2))
    Om = np.empty((w.heads, w.dk, w.rank), np.float32)
    C = np.empty((w.heads, w.rank, w.dk), np.float32)
    E0 = np.eye(w.dk)
    for h in range(w.heads):
        Q = synth.calibration_queries(w, layer, h)
        Omega, _lam = orc.fit_sketching_matrix(Q, E0, w.rank)
        Om[h] = Omega.astype(np.float32)
        C[h] = orc.offline_coefficient_map(Om[h].astype(np.float64), E0).astype(np.float32)
    return Om, C


def token_tensors(w: synth.Workload, x: dict, device):
    """Device tensors of one step's inputs in the C ABI's dtypes."""
    dec_io = w.io if w.kind == "kda" else "f32"
    return dict(
        q=synth.to_torch(x["q"], w.io, device), k=synth.to_torch(x["k"], w.io, device),
        v=synth.to_torch(x["v"], w.io, device), beta=synth.to_torch(x["beta"], "f32", device),
        decay=synth.to_torch(x["decay"], dec_io, device))


def oracle_token(x: dict, bs, hs):
    """(k, v, beta, decay) of the selected heads as float64 arrays [N, ...]."""
    return (x["k"][bs, hs].astype(np.float64), x["v"][bs, hs].astype(np.float64),
            x["beta"][bs, hs].astype(np.float64), x["decay"][bs, hs].astype(np.float64))


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |got - ref| / max |ref| over all elements (the parity norm of the workloads)."""
    denom = float(np.abs(ref).max())
    return float(np.abs(got.astype(np.float64) - ref).max()) / (denom if denom > 0 else 1.0)


def select_heads(w: synth.Workload, max_heads: int, seed: int = 0):
    """Deterministic sample of (b, h) pairs; everything if the workload is small."""
    total = w.batch * w.heads
    if total <= max_heads:
        idx = np.arange(total)
    else:
        rng = np.random.default_rng(seed)
        idx = np.sort(rng.choice(total, size=max_heads, replace=False))
        idx[0], idx[-1] = 0, total - 1            # always include the corners
    return idx // w.heads, idx % w.heads
