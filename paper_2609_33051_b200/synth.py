"""Seeded synthetic inputs for the SketchSSM decode path.

This module only draws random numbers and shapes them into the tensors the
decode path consumes (queries, keys, values, gates, initial states, calibration
queries).  It contains none of the method's arithmetic: no recurrence, no
sketch, no coefficient map.  Both the CUDA library's tests/benchmarks and the
CPU oracle's tests take their inputs from here so that they see identical bits.

Every array is produced in float64, shaped, and then rounded ONCE to the I/O
precision of the workload (float32 or bfloat16).  The rounded values are
returned in float32 containers: widening them to float64 (oracle) or narrowing
them to bfloat16 (GPU) is exact, so both consumers see the same numbers.

Workloads mirror the five decode regimes this repository is measured on:
a tiny gated-delta-rule layer, a Mamba-2 layer, a GDN layer, a KDA layer and a
multi-layer Mamba-2 sweep.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch

MAMBA2, GDN, KDA = "mamba2", "gdn", "kda"
KINDS = (MAMBA2, GDN, KDA)

BASE_SEED = 33051

# field ids used to key the counter-based generator
_F_Q, _F_K, _F_V, _F_BETA, _F_DECAY, _F_STATE, _F_ALOG, _F_OMEGA, _F_CALIB_BASIS, _F_CALIB_G, _F_CALIB_E = range(11)


@dataclass(frozen=True)
class Workload:
    """Shape and distribution recipe of one synthetic decode workload."""

    name: str
    kind: str          # "mamba2" | "gdn" | "kda"
    batch: int
    heads: int
    dk: int            # K: key/query channels (Mamba-2: state dim N)
    dv: int            # V: value channels     (Mamba-2: head dim P)
    rank: int          # r (paper G): sketch rank
    buf_len: int       # L (paper W): window / ring capacity
    steps: int         # decode steps of a full run
    io: str            # "f32" | "bf16": precision of q, k, v, beta, KDA gates
    seed: int
    layers: int = 1
    basis: str = "pca"  # "qr": Omega = Q factor of a Gaussian, C = Omega^T; "pca": fitted from calibration queries
    calib_n: int = 4096
    calib_rank: int = 24
    calib_noise: float = 0.05
    state_std: float = 0.02

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, Workload] = {
    # config 1: tiny GDN layer, fp32 throughout, orthonormal random basis
    "c1_gdn_tiny": Workload("c1_gdn_tiny", GDN, 4, 4, 64, 64, 8, 8, 64, "f32", BASE_SEED + 1, basis="qr"),
    # config 2: Mamba-2-style layer (state 128x64 per head)
    "c2_mamba2": Workload("c2_mamba2", MAMBA2, 256, 64, 128, 64, 16, 16, 256, "bf16", BASE_SEED + 2),
    # config 3: GDN layer
    "c3_gdn": Workload("c3_gdn", GDN, 512, 32, 128, 128, 16, 16, 256, "bf16", BASE_SEED + 3),
    # config 4: KDA layer
    "c4_kda": Workload("c4_kda", KDA, 512, 32, 128, 128, 16, 32, 256, "bf16", BASE_SEED + 4),
    # config 5: one point of the 48-layer Mamba-2 sweep; use sweep_point() for the others
    "c5_mamba2_stack": Workload("c5_mamba2_stack", MAMBA2, 256, 64, 128, 64, 16, 16, 256, "bf16", BASE_SEED + 5, layers=48),
}

SWEEP_BATCH = (64, 256, 1024, 2048)
SWEEP_BUF_LEN = (4, 16, 64)
SWEEP_RANK = (8, 16, 32)


def sweep_point(batch: int, buf_len: int, rank: int) -> Workload:
    """One (batch, L, r) point of the config-5 sweep."""
    return CONFIGS["c5_mamba2_stack"].replace(
        name=f"c5_mamba2_B{batch}_L{buf_len}_r{rank}", batch=batch, buf_len=buf_len, rank=rank)


def _gen(w: Workload, field: int, layer: int = 0, step: int = 0, extra: int = 0) -> np.random.Generator:
    ss = np.random.SeedSequence([w.seed, field, layer, step, extra])
    return np.random.Generator(np.random.Philox(ss))


def round_io(x: np.ndarray, io: str) -> np.ndarray:
    """Round float64 values to the I/O precision; result is float32 holding representable values."""
    x32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    if io == "f32":
        return x32
    if io == "bf16":
        t = torch.from_numpy(np.ascontiguousarray(x32)).to(torch.bfloat16).to(torch.float32)
        return t.numpy()
    raise ValueError(f"unknown io precision {io!r}")


def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def _softplus(x):
    return np.logaddexp(0.0, x)


def initial_state(w: Workload, layer: int = 0) -> np.ndarray:
    """S_init ~ N(0, state_std^2), shape [B, H, K, V], float32."""
    g = _gen(w, _F_STATE, layer)
    out = g.standard_normal((w.batch, w.heads, w.dk, w.dv), dtype=np.float32)
    out *= np.float32(w.state_std)
    return out


def a_log(w: Workload, layer: int = 0) -> np.ndarray:
    """Mamba-2 per-head A_log ~ U(0, 2.7), float32 [H]."""
    g = _gen(w, _F_ALOG, layer)
    return g.uniform(0.0, 2.7, size=(w.heads,)).astype(np.float32)


def step_inputs(w: Workload, layer: int, step: int) -> Dict[str, np.ndarray]:
    """Inputs of one decode step for every (batch, head).

    Returns float32 arrays holding values representable in the workload's I/O
    precision:
      q, k : [B, H, K]   (GDN/KDA: L2-normalised per head before rounding)
      v    : [B, H, V]
      beta : [B, H]      write gate (Mamba-2: the step size Delta_t, float32)
      decay: [B, H]      scalar decay (Mamba-2 a_t, GDN alpha_t; float32), or
             [B, H, K]   KDA per-channel decay g_t in (0, 1)
    """
    B, H, K, V = w.batch, w.heads, w.dk, w.dv
    q = _gen(w, _F_Q, layer, step).standard_normal((B, H, K))
    k = _gen(w, _F_K, layer, step).standard_normal((B, H, K))
    v = _gen(w, _F_V, layer, step).standard_normal((B, H, V))
    zb = _gen(w, _F_BETA, layer, step).standard_normal((B, H))
    if w.kind in (GDN, KDA):
        q = q / np.linalg.norm(q, axis=-1, keepdims=True)
        k = k / np.linalg.norm(k, axis=-1, keepdims=True)
        beta = round_io(_sigmoid(zb), w.io)
    else:
        beta = _softplus(zb).astype(np.float32)                      # Delta_t, fp32
    if w.kind == MAMBA2:
        al = a_log(w, layer).astype(np.float64)[None, :]
        decay = np.exp(-beta.astype(np.float64) * np.exp(al)).astype(np.float32)
    elif w.kind == GDN:
        zd = _gen(w, _F_DECAY, layer, step).standard_normal((B, H))
        decay = np.exp(-_softplus(zd)).astype(np.float32)
    else:
        zd = 2.0 + _gen(w, _F_DECAY, layer, step).standard_normal((B, H, K))
        decay = round_io(_sigmoid(zd), w.io)
    return {
        "q": round_io(q, w.io), "k": round_io(k, w.io), "v": round_io(v, w.io),
        "beta": np.ascontiguousarray(beta, dtype=np.float32),
        "decay": np.ascontiguousarray(decay, dtype=np.float32),
    }


def _orthonormal(g: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    qmat, rmat = np.linalg.qr(g.standard_normal((rows, cols)))
    return qmat * np.sign(np.diag(rmat))[None, :]


def qr_basis(w: Workload, layer: int = 0) -> np.ndarray:
    """Omega [H, K, r]: per head the orthonormal Q factor of a seeded Gaussian (float32)."""
    out = np.empty((w.heads, w.dk, w.rank), dtype=np.float32)
    for h in range(w.heads):
        out[h] = _orthonormal(_gen(w, _F_OMEGA, layer, 0, h), w.dk, w.rank).astype(np.float32)
    return out


def calibration_queries(w: Workload, layer: int, head: int, n: Optional[int] = None) -> np.ndarray:
    """Calibration effective queries of one head, [n, K] float64.

    Each sample is A g + noise * eps with A an orthonormal K x calib_rank matrix
    (fixed per head), g ~ N(0, I) and eps ~ N(0, I_K).
    """
    n = w.calib_n if n is None else n
    A = _orthonormal(_gen(w, _F_CALIB_BASIS, layer, 0, head), w.dk, w.calib_rank)
    g = _gen(w, _F_CALIB_G, layer, 0, head).standard_normal((n, w.calib_rank))
    e = _gen(w, _F_CALIB_E, layer, 0, head).standard_normal((n, w.dk))
    return g @ A.T + w.calib_noise * e


def to_torch(x: np.ndarray, io: str, device="cpu") -> torch.Tensor:
    """Exact narrowing of a round_io() result to a torch tensor of the I/O dtype."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    if io == "bf16":
        t = t.to(torch.bfloat16)
    return t.to(device)
