"""Algorithmic HBM bytes of the three hot-path kernels (what the method must move, per launch).

fp32 state and sketch; q/k/v and the ring's k/v (and KDA gates) in the I/O dtype; fp32 scalar gates.
The per-head basis Omega and coefficient map C are shared by the whole batch and counted once per launch.
"""
from __future__ import annotations


def _io(io: str) -> int:
    return 2 if io == "bf16" else 4


def slot_bytes(kind: str, K: int, V: int, io: str) -> int:
    """Bytes of one ring slot: k, v, beta and the decay (scalar, or K-vector for KDA)."""
    e = _io(io)
    return K * e + V * e + 4 + (K * e if kind == "kda" else 4)


def token_bytes(kind: str, K: int, V: int, io: str) -> int:
    """Bytes of one step's token inputs per head: q plus one slot's worth."""
    return K * _io(io) + slot_bytes(kind, K, V, io)


def decode_bytes(kind, B, H, K, V, r, n_before, io="bf16", out_bytes=4, full_read=False, append=True,
                 sketch_bytes=4, coef_per_seq=False, erase_factors=False) -> int:
    """decode_step / full_read_decode launch at ring fill n_before.  sketch_bytes: storage of U and C (4 or 2);
    coef_per_seq: every head reads its own coefficient map instead of the one shared by the batch;
    erase_factors: the projected erase vectors f_s (r floats per buffered token) are read, and the token's is written."""
    per_head = (K * V * 4 if full_read else r * V * sketch_bytes)   # S or U
    per_head += n_before * slot_bytes(kind, K, V, io)               # ring read
    per_head += token_bytes(kind, K, V, io)                         # q, k, v, gates of the token
    per_head += slot_bytes(kind, K, V, io) if append else 0         # append write
    per_head += V * out_bytes                                       # o
    shared = 0
    if not full_read:
        if coef_per_seq:
            per_head += r * K * sketch_bytes                        # the head's own C
        else:
            shared = H * r * K * sketch_bytes                       # C, once per launch
        if erase_factors and kind != "mamba2":
            per_head += (n_before + (1 if append else 0)) * r * sketch_bytes   # f_s of the buffered tokens in, f_t out
    return B * H * per_head + shared


def update_bytes(kind, B, H, K, V, r, n_before, io="bf16", out_bytes=4, has_token=True, sketch=True,
                 with_output=True, sketch_bytes=4, coef_per_seq=False) -> int:
    """state_update launch replaying n_before buffered tokens (+ the current one).  With coef_per_seq the write of the
    per-head coefficient map is counted (what the method must move); the second read of the state that this
    implementation's separate coefficient kernel performs is not algorithmic and shows up as a lower fraction."""
    n_tot = n_before + (1 if has_token else 0)
    per_head = K * V * 4 * (2 if n_tot > 0 else 1)                  # S read (+ write)
    per_head += n_before * slot_bytes(kind, K, V, io)
    per_head += slot_bytes(kind, K, V, io) if has_token else 0
    per_head += (K * _io(io) + V * out_bytes) if with_output else 0  # q in, o out
    per_head += r * V * sketch_bytes if sketch else 0               # U write
    per_head += r * K * sketch_bytes if (sketch and coef_per_seq) else 0   # C write
    shared = H * K * r * 4 if sketch else 0                         # Omega
    return B * H * per_head + shared
