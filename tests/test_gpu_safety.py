"""Checks that stand in for a memory sanitizer and a fault injector, in forms that cannot fault a GPU.

(a) Guard regions: every buffer the library is handed (state, sketch, ring, basis, coefficient map, status, work,
    token tensors, output) sits inside a larger allocation with a byte pattern before and after it; after a window
    of calls the patterns must be intact, so no kernel wrote outside a caller buffer.
(b) Poisoned inputs: a token whose q, k and v are NaN in one (batch, head) must not change any other head: outputs,
    state and sketch of all other heads are bit-identical to a clean run.  (One documented exception: the Mamba-2
    tensor-core flush with 64 value channels contracts two batch entries of the same head index in one 128-lane
    tile, and a NaN key times the other entry's zero weights is NaN, so the tile partner is excluded there.)
(c) A bounded device wait that runs out: the self-test entry point makes one warp wait on a barrier phase that
    nothing completes; the call returns, the status word reports the time-out with the place that was passed in, and
    after the caller clears the status block the next calls give correct results.
"""
import numpy as np
import pytest
import torch

from paper_2609_33051_b200 import binding, synth
from tests import harness
from tests.test_gpu_parity import FP32_GUARD, run_schedule

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on each side; a multiple of 256 keeps the inner buffer aligned
PATTERN = 0xA5


class Guarded:
    """A device buffer of `nbytes` between two guard regions filled with a byte pattern."""

    def __init__(self, nbytes, dev):
        self.nbytes = nbytes
        self.raw = torch.full((GUARD + ((nbytes + 255) // 256) * 256 + GUARD,), PATTERN, dtype=torch.uint8, device=dev)
        self.inner = self.raw[GUARD:GUARD + nbytes]
        self.inner.zero_()

    def view(self, dtype, *shape):
        return self.inner.view(dtype).view(*shape)

    def intact(self):
        tail = self.raw[GUARD + self.nbytes:]
        return bool((self.raw[:GUARD] == PATTERN).all().item()) and bool((tail == PATTERN).all().item())


def guarded_layer(w, dev):
    """A SketchSSM whose seven bound buffers all live between guard regions; returns (layer, {name: Guarded})."""
    m = binding.SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, device=0, allocate=False)
    sz = m.sizes
    g = {"state": Guarded(sz.state_bytes, dev), "sketch": Guarded(sz.sketch_bytes, dev), "ring": Guarded(sz.ring_bytes, dev),
         "omega": Guarded(sz.omega_bytes, dev), "coef": Guarded(sz.coef_bytes, dev), "status": Guarded(sz.status_bytes, dev),
         "work": Guarded(sz.work_bytes, dev)}
    f32 = torch.float32
    m.state = g["state"].view(f32, w.batch, w.heads, w.dk, w.dv)
    m.sketch = g["sketch"].view(f32, w.batch, w.heads, w.rank, w.dv)
    m.ring = g["ring"].inner
    m.omega = g["omega"].view(f32, w.heads, w.dk, w.rank)
    m.coef = g["coef"].view(f32, w.heads, w.rank, w.dk)
    m.status = g["status"].view(torch.int32, sz.status_bytes // 4)
    m.work = g["work"].view(f32, sz.work_bytes // 4)
    m.bind()
    return m, g


def guarded_tokens(w, x, dev):
    """One step's token tensors and an output tensor, each between guard regions."""
    plain = harness.token_tensors(w, x, dev)
    out, guards = {}, []
    for name, t in plain.items():
        gb = Guarded(t.numel() * t.element_size(), dev)
        gv = gb.view(t.dtype, *t.shape)
        gv.copy_(t)
        out[name] = gv
        guards.append((name, gb))
    go = Guarded(w.batch * w.heads * w.dv * 4, dev)
    out["out"] = go.view(torch.float32, w.batch, w.heads, w.dv)
    guards.append(("out", go))
    return out, guards


@pytest.mark.parametrize("kind", synth.KINDS)
@pytest.mark.parametrize("batch,heads,dv,rank,buf_len", [(6, 3, None, 16, 16), (37, 5, None, 8, 12)])
@pytest.mark.parametrize("decode_impl", [1, 0])
def test_no_kernel_writes_outside_a_caller_buffer(kind, batch, heads, dv, rank, buf_len, decode_impl):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    dev = torch.device("cuda", 0)
    dv = dv or (64 if kind == "mamba2" else 128)
    w = synth.Workload("t", kind, batch, heads, 128, dv, rank, buf_len, 0, "bf16", 61, basis="qr")
    m, g = guarded_layer(w, dev)
    m.tune("decode_impl", decode_impl)
    Om, C = harness.basis_for(w)
    m.state.copy_(torch.from_numpy(synth.initial_state(w)))
    m.omega.copy_(torch.from_numpy(Om))
    m.coef.copy_(torch.from_numpy(C))
    m.state_update(0)
    token_guards = []
    for t in range(buf_len + 2):                      # one full window (decode steps, flush) and the start of the next
        tt, tg = guarded_tokens(w, synth.step_inputs(w, 0, t), dev)
        token_guards += tg
        n = t % buf_len
        if n < buf_len - 1:
            m.decode_step(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], tt["out"])
            m.full_read_decode(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], tt["out"], flags=binding.NO_APPEND)
        else:
            m.state_update(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], tt["out"])
    torch.cuda.synchronize()
    m.check_status()
    for name, gb in list(g.items()) + token_guards:
        assert gb.intact(), f"guard region around `{name}` was overwritten"
    # and the run itself was a correct one: the scheduler counters behind the status ints are back to zero
    assert int(m.status.abs().sum().item()) == 0


@pytest.mark.parametrize("kind,coef,sketch,erase,ranks", [
    ("mamba2", "pivot", "bf16", False, False), ("gdn", "pivot", "f32", True, True), ("kda", None, "bf16", True, False),
    ("gdn", "ridge", "bf16", False, True), ("kda", "pivot", "f32", False, False)])
def test_no_kernel_writes_outside_a_caller_buffer_in_the_optional_modes(kind, coef, sketch, erase, ranks):
    """The same check for the buffers and kernels of the optional modes: per-head coefficient maps (written by the map
    kernel, fp32 or bfloat16), bfloat16 sketch storage, the erase vectors, a per-head rank table, and calls with
    per-sequence phases (decode kernel of the general kind, CUDA-core flush, map kernel in one call)."""
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    dev = torch.device("cuda", 0)
    dv = 64 if kind == "mamba2" else 128
    L = 8
    w = synth.Workload("t", kind, 7, 3, 128, dv, 8, L, 0, "bf16", 67, basis="qr")
    m = binding.SketchSSM(kind, w.batch, w.heads, w.dk, w.dv, w.rank, L, io="bf16", device=0, allocate=False,
                          coef_per_seq=coef is not None, coef_pivots=4 if coef == "pivot" else 0, sketch=sketch,
                          erase_factors=erase)
    sz = m.sizes
    names = ["state", "sketch", "ring", "omega", "coef", "status", "work"] + (["erase"] if erase else [])
    g = {n: Guarded(getattr(sz, n + "_bytes"), dev) for n in names}
    f32, st = torch.float32, binding.TORCH_DTYPE[sketch]
    m.state = g["state"].view(f32, w.batch, w.heads, w.dk, w.dv)
    m.sketch = g["sketch"].view(st, w.batch, w.heads, w.rank, w.dv)
    m.ring = g["ring"].inner
    m.omega = g["omega"].view(f32, w.heads, w.dk, w.rank)
    m.coef = g["coef"].view(st, *((w.batch,) if coef else ()), w.heads, w.rank, w.dk)
    m.status = g["status"].view(torch.int32, sz.status_bytes // 4)
    m.work = g["work"].view(f32, sz.work_bytes // 4)
    if erase:
        m.erase = g["erase"].view(st, w.batch, w.heads, L, w.rank)
    if ranks:
        g["head_rank"] = Guarded(w.heads * 4, dev)
        m.head_rank = g["head_rank"].view(torch.int32, w.heads)
        m.head_rank.copy_(torch.tensor([8, 0, 4], dtype=torch.int32))
    m.bind()
    Om, C = harness.basis_for(w)
    m.state.copy_(torch.from_numpy(synth.initial_state(w)))
    m.omega.copy_(torch.from_numpy(Om))
    if coef is None:
        m.coef.copy_(torch.from_numpy(C))
    m.state_update(0)
    token_guards = []
    for t in range(L + 2):                            # a lock-step window, then the start of the next
        tt, tg = guarded_tokens(w, synth.step_inputs(w, 0, t), dev)
        token_guards += tg
        n = t % L
        if n < L - 1:
            m.decode_step(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], tt["out"])
        else:
            m.state_update(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], tt["out"])
    # calls with per-sequence phases: every sequence flushes once at its own ring fill (the lock-step steps left 2 tokens)
    fill = [2] * w.batch
    for t in range(L + 2, 2 * L + 2):
        tt, tg = guarded_tokens(w, synth.step_inputs(w, 0, t), dev)
        token_guards += tg
        phase = []
        for b in range(w.batch):
            if fill[b] == L - 1 or fill[b] == 2 + b % 4 + 1:
                phase.append(-(fill[b] + 1)); fill[b] = 0
            else:
                phase.append(fill[b]); fill[b] += 1
        gp = Guarded(w.batch * 4, dev)
        ph = gp.view(torch.int32, w.batch)
        ph.copy_(torch.tensor(phase, dtype=torch.int32))
        token_guards.append(("phase", gp))
        m.step_mixed(ph, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], tt["out"])
    torch.cuda.synchronize()
    m.check_status()
    for name, gb in list(g.items()) + token_guards:
        assert gb.intact(), f"guard region around `{name}` was overwritten"
    assert bool(torch.isfinite(m.state).all().item()) and bool(torch.isfinite(m.sketch.float()).all().item())


def _window(w, dev, poison_at=None, poison_bh=(1, 1), tune=None):
    """Two windows on a fresh layer; optionally one step's q, k, v of one (batch, head) are NaN.  Returns the outputs of
    every step, the final state and the final sketch (device tensors)."""
    m = binding.SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, device=0)
    for key, val in (tune or {}).items():
        m.tune(key, val)
    Om, C = harness.basis_for(w)
    m.state.copy_(torch.from_numpy(synth.initial_state(w)))
    m.omega.copy_(torch.from_numpy(Om))
    m.coef.copy_(torch.from_numpy(C))
    m.state_update(0)
    outs = []
    for t in range(2 * w.buf_len):
        tt = harness.token_tensors(w, synth.step_inputs(w, 0, t), dev)
        if t == poison_at:
            b, h = poison_bh
            for name in ("q", "k", "v"):
                tt[name][b, h] = float("nan")
        o = m.new_output()
        n = t % w.buf_len
        if n < w.buf_len - 1:
            m.decode_step(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
        else:
            m.state_update(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
        outs.append(o)
    torch.cuda.synchronize()
    m.check_status()
    return outs, m.state.clone(), m.sketch.clone()


@pytest.mark.parametrize("kind,dv", [("mamba2", 64), ("mamba2", 128), ("gdn", 128), ("kda", 128)])
@pytest.mark.parametrize("poison_at", [2, 7])          # a decode step; the flush step of the first window (L = 8)
def test_a_nan_token_stays_in_its_head(kind, dv, poison_at):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    dev = torch.device("cuda", 0)
    w = synth.Workload("t", kind, 6, 3, 128, dv, 16, 8, 0, "bf16", 67, basis="qr")
    pb, ph = 3, 1
    clean = _window(w, dev)
    dirty = _window(w, dev, poison_at=poison_at, poison_bh=(pb, ph))
    keep = torch.ones(w.batch, w.heads, dtype=torch.bool, device=dev)
    keep[pb, ph] = False
    if kind == "mamba2" and dv == 64:
        keep[pb ^ 1, ph] = False        # tile partner of the tensor-core flush (see the module docstring)
    for oc, od in zip(clean[0], dirty[0]):
        assert torch.equal(oc[keep], od[keep])
    assert torch.equal(clean[1][keep], dirty[1][keep])
    assert torch.equal(clean[2][keep], dirty[2][keep])
    # the poisoned head itself did see the NaN (the test would be vacuous otherwise)
    assert torch.isnan(dirty[1][pb, ph]).any()
    # with the CUDA-core flush no head shares a tile with another: nothing but the poisoned head changes
    if kind == "mamba2" and dv == 64:
        clean1 = _window(w, dev, tune={"update_impl": 1})
        dirty1 = _window(w, dev, poison_at=poison_at, poison_bh=(pb, ph), tune={"update_impl": 1})
        keep[pb ^ 1, ph] = True
        assert torch.equal(clean1[1][keep], dirty1[1][keep]) and torch.equal(clean1[2][keep], dirty1[2][keep])


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    w = synth.Workload("t", "gdn", 4, 2, 128, 128, 16, 8, 0, "bf16", 71, basis="qr")
    m = binding.SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, device=0)
    rc, detail = m.read_status()
    assert rc == 0 and detail == [0, 0, 0, 0]
    m.selftest_wait_timeout(poll_limit=2048, where=1234)
    rc, detail = m.read_status()
    assert rc == -5 and detail[0] == 4 and detail[1] == 1234          # SKETCHSSM_DEVICE_TIMEOUT, the probe's wait, its place
    with pytest.raises(binding.SketchSSMError):
        m.check_status()
    # the first fault is kept: a second time-out elsewhere does not overwrite it
    m.selftest_wait_timeout(poll_limit=512, where=77)
    rc, detail = m.read_status()
    assert rc == -5 and detail[1] == 1234
    # the caller clears the status block; the GPU context is intact and the library computes correctly again
    m.status.zero_()
    torch.cuda.synchronize()
    assert m.read_status()[0] == 0
    m.close()
    errs = run_schedule(w, w.buf_len + 3, max_heads=10**9)
    assert errs["out"] <= FP32_GUARD and errs["S"] <= FP32_GUARD and errs["U"] <= FP32_GUARD
