"""The decode entry point for callers that cannot allocate (sketchssm_decode_step_static).

Some users of this library run where no device memory can be obtained at call time: inside an engine whose
pool was divided up at start-up, as a plug-in that is only handed tensors, or in a region where an allocation
would stall the device.  For them the library carries a fixed 4 MiB device array and this entry point uses it
for the hand-off between its two kernels.  The test drives it through the C ABI and checks it against the
regular decode step on identical state, twice in a row with different tokens and ring fills, so that anything
the first call leaves behind in the shared array would show up in the second.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_33051_b200 import binding, build, synth
from tests import harness

TOL = 2e-5      # same fp32 arithmetic on the same bits; only the summation order differs between the two paths


def _layer(w):
    Om, C = harness.basis_for(w)
    m = binding.SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, device=0)
    m.state.copy_(torch.from_numpy(synth.initial_state(w)))
    m.omega.copy_(torch.from_numpy(Om))
    m.coef.copy_(torch.from_numpy(C))
    m.state_update(0)
    return m


@pytest.mark.gpu
@pytest.mark.parametrize("kind", synth.KINDS)
def test_static_decode_matches_regular_decode_on_two_calls_in_a_row(kind):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    dev = torch.device("cuda", 0)
    w = synth.Workload("t", kind, 8, 4, 128, 64 if kind == "mamba2" else 128, 16, 16, 0, "bf16", 2024, basis="qr")
    m = _layer(w)
    toks = [harness.token_tensors(w, synth.step_inputs(w, 0, t), dev) for t in range(6)]
    args = lambda t: (toks[t]["q"], toks[t]["k"], toks[t]["v"], toks[t]["beta"], toks[t]["decay"])
    ref, got = m.new_output(), m.new_output()
    for t in range(3):                                   # three buffered tokens through the regular path
        m.decode_step(t, *args(t), ref)
    # the caller's scratch must never be touched by the static call: fill it with a sentinel and compare afterwards
    # (the regular decode step runs as one kernel and leaves it alone too)
    sentinel = torch.arange(m.work.numel(), dtype=torch.float32, device=dev) * 0.5 - 7.0
    m.work.copy_(sentinel)
    # call 1: token 3 at ring fill 3, not appended by the reference, appended by the static call
    m.decode_step(3, *args(3), ref, flags=binding.NO_APPEND)
    m.decode_step_static(3, *args(3), got)
    assert m.last_launch_count() == 2
    assert harness.rel_err(got.cpu().numpy(), ref.cpu().numpy().astype(np.float64)) <= TOL
    # call 2, immediately after: another token, one more slot in the ring (appended by call 1)
    m.decode_step(4, *args(4), ref, flags=binding.NO_APPEND)
    m.decode_step_static(4, *args(4), got, flags=binding.NO_APPEND)
    assert harness.rel_err(got.cpu().numpy(), ref.cpu().numpy().astype(np.float64)) <= TOL
    # the ring the static call appended to is the ring the regular path would have produced
    rk, rv, rb, rd = m.ring_views()
    assert torch.equal(rk[:, :, 3], toks[3]["k"]) and torch.equal(rv[:, :, 3], toks[3]["v"])
    assert torch.equal(rb[:, :, 3], toks[3]["beta"]) and torch.equal(rd[:, :, 3], toks[3]["decay"])
    assert torch.equal(m.work, sentinel), "sketchssm_decode_step_static wrote to the caller's work buffer"
    # and against the oracle directly: the step at ring fill 4 over the five tokens now known to the ring
    from oracle import sketchssm_oracle as orc
    Om, C = harness.basis_for(w)
    S0 = synth.initial_state(w).astype(np.float64)
    U = orc.sketch_of(S0, Om.astype(np.float64)[None])
    xs = [synth.step_inputs(w, 0, t) for t in range(5)]
    ring = [tuple(x[n].astype(np.float64) for n in ("k", "v", "beta", "decay")) for x in xs]
    want = orc.decode_step(kind, U, C.astype(np.float64)[None], ring, xs[4]["q"].astype(np.float64))
    assert harness.rel_err(got.cpu().numpy(), want) <= 5e-5
    m.check_status()


def test_static_decode_rejects_what_does_not_fit_its_array():
    """Host-side check, no GPU needed: batch * heads * (dk + buf_len) floats must fit in 4 MiB."""
    build.build()
    lib = binding.load_library()
    cfg = binding.Config(kind=0, batch=256, heads=64, dk=128, dv=64, rank=16, buf_len=16, io_dtype=1, out_dtype=0, device=0)
    ctx = ctypes.c_void_p()
    assert lib.sketchssm_create(ctypes.byref(cfg), ctypes.byref(ctx)) == 0
    d = ctypes.c_void_p(0x1000)
    assert lib.sketchssm_decode_step_static(ctx, 0, d, d, d, d, d, d, 0, None) == -3           # not bound
    bufs = binding.Buffers(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000)
    assert lib.sketchssm_bind(ctx, ctypes.byref(bufs)) == 0
    assert 256 * 64 * (128 + 16) * 4 > 4 << 20
    assert lib.sketchssm_decode_step_static(ctx, 0, d, d, d, d, d, d, 0, None) == -2           # too large: clear error
    assert lib.sketchssm_decode_step_static(ctx, 16, d, d, d, d, d, d, 0, None) == -1          # n_before out of range
    assert lib.sketchssm_decode_step_static(ctx, 0, None, d, d, d, d, d, 0, None) == -1
    lib.sketchssm_destroy(ctx)
