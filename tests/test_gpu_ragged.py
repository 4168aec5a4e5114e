"""Runtime consequences of the paper's deployment beyond one lock-step rank for all heads:

- a per-head rank table with dense-fallback heads (Appendix E: offline rank allocation gives every head its own sketch
  rank, and heads whose budget reaches the full state keep the exact read), served inside one decode launch;
- per-sequence window phases (continuous batching): in one call some sequences take a non-flush decode step at their
  own ring fill while others take the flush step, possibly before their ring is full;
- the value width 80 of the second Mamba-2 head shape in the paper's traffic tables (K = 128, V = 80).

Each is compared with the oracle element by element; the oracle is driven per head / per sequence with the same
truncated basis, the same phases and the same tokens.
"""
import numpy as np
import pytest
import torch

from oracle import sketchssm_oracle as orc
from paper_2609_33051_b200 import binding, synth
from tests import harness
from tests.test_gpu_parity import FP32_GUARD, check, make_layer, run_schedule

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch.device("cuda", 0)


@pytest.mark.parametrize("kind,dv,erase", [("mamba2", 64, False), ("gdn", 128, False), ("kda", 128, False), ("mamba2", 80, False),
                                            ("gdn", 128, True), ("kda", 128, True)])
@pytest.mark.parametrize("coef", [None, "pivot"])
def test_per_head_ranks_and_dense_fallback_heads(kind, dv, coef, erase):
    """Heads of one layer with ranks (8, 3, 0, 5, 1, 8): rank-g heads use the first g columns of Omega (and the first g rows
    of C, or their own state-dependent map of that rank); rank 0 reads the full state exactly.  Two windows."""
    dev = _dev()
    ranks = np.array([8, 3, 0, 5, 1, 8], dtype=np.int32)
    w = synth.Workload("t", kind, 5, len(ranks), 128, dv, 8, 8, 0, "bf16", 131, basis="qr")
    m, S0, Om, C, _ = make_layer(w, coef=coef, erase=erase)
    m.head_rank = torch.from_numpy(ranks).to(dev)
    m.bind()
    m.state_update(0)
    S = S0.astype(np.float64)                                    # [B, H, K, V]
    Om64, C64 = Om.astype(np.float64), C.astype(np.float64)

    def maps(Snow):
        """per-head (U, C) of the head's own rank"""
        out = {}
        for h, g in enumerate(ranks):
            if g == 0:
                continue
            U = orc.sketch_of(Snow[:, h], Om64[h][None, :, :g])
            if coef is None:
                Cm = np.broadcast_to(C64[h, :g], (w.batch, g, w.dk))
            else:
                Cm = orc.coefficient_maps(Snow[:, h], np.broadcast_to(Om64[h, :, :g], (w.batch, w.dk, g)), coef, 0.1, 4)
            out[h] = (U, Cm)
        return out

    UC = maps(S)
    ring, worst = [], 0.0
    o = m.new_output()
    for t in range(2 * w.buf_len + 3):
        x = synth.step_inputs(w, 0, t)
        tt = harness.token_tensors(w, x, dev)
        n = t % w.buf_len
        ring.append(tuple(x[f].astype(np.float64) for f in ("k", "v", "beta", "decay")))
        q = x["q"].astype(np.float64)
        ref = np.empty((w.batch, w.heads, w.dv))
        if n < w.buf_len - 1:
            m.decode_step(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
            for h, g in enumerate(ranks):
                toks_h = [tuple(a[:, h] for a in tok) for tok in ring]
                if g == 0:
                    ref[:, h] = orc.full_read_decode(kind, S[:, h], toks_h, q[:, h])
                else:
                    ref[:, h] = orc.decode_step(kind, UC[h][0], UC[h][1], toks_h, q[:, h])
        else:
            m.state_update(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
            S, _, ref = orc.state_update(kind, S, ring, np.broadcast_to(Om64, (w.batch,) + Om64.shape), q)
            UC = maps(S)
            ring = []
        worst = max(worst, harness.rel_err(o.cpu().numpy(), ref))
    m.check_status()
    assert worst <= (2e-4 if coef else FP32_GUARD), worst
    assert harness.rel_err(m.state.cpu().numpy(), S) <= FP32_GUARD


@pytest.mark.parametrize("kind,dv,coef,erase", [("mamba2", 64, None, False), ("gdn", 128, None, False), ("kda", 128, None, False),
                                                 ("mamba2", 80, None, False), ("gdn", 128, "pivot", False),
                                                 ("mamba2", 64, "ridge", False), ("gdn", 128, None, True),
                                                 ("kda", 128, "pivot", True)])
def test_sequences_at_different_window_phases_in_one_call(kind, dv, coef, erase):
    """Sequence b takes its first flush when b mod L tokens are buffered and then one every L tokens, so every call mixes
    decode steps at different ring fills with flush steps.  The oracle follows every sequence with its own ring."""
    dev = _dev()
    L = 8
    w = synth.Workload("t", kind, 11, 3, 128, dv, 8, L, 0, "bf16", 137, basis="qr")
    m, S0, Om, C, _ = make_layer(w, coef=coef, erase=erase)
    m.state_update(0)
    Om64 = Om.astype(np.float64)
    S = [S0[b].astype(np.float64) for b in range(w.batch)]                       # per sequence: [H, K, V]
    U = [orc.sketch_of(S[b], Om64) for b in range(w.batch)]
    Cm = [C.astype(np.float64) if coef is None else orc.coefficient_maps(S[b], Om64, coef, 0.1, 4) for b in range(w.batch)]
    rings = [[] for _ in range(w.batch)]
    first = [b % L for b in range(w.batch)]                                      # ring fill at which the first flush comes
    flushed = [False] * w.batch
    o = m.new_output()
    worst, n_flush, n_decode = 0.0, 0, 0
    for t in range(3 * L + 2):
        x = synth.step_inputs(w, 0, t)
        tt = harness.token_tensors(w, x, dev)
        phase = np.empty(w.batch, np.int32)
        ref = np.empty((w.batch, w.heads, w.dv))
        for b in range(w.batch):
            n = len(rings[b])
            tok = tuple(x[f][b].astype(np.float64) for f in ("k", "v", "beta", "decay"))
            q = x["q"][b].astype(np.float64)
            rings[b].append(tok)
            do_flush = n == L - 1 or (not flushed[b] and n == first[b])
            if do_flush:
                phase[b] = -(n + 1)
                S[b], U[b], ref[b] = orc.state_update(kind, S[b], rings[b], Om64, q)
                if coef is not None:
                    Cm[b] = orc.coefficient_maps(S[b], Om64, coef, 0.1, 4)
                rings[b] = []
                flushed[b] = True
                n_flush += 1
            else:
                phase[b] = n
                ref[b] = orc.decode_step(kind, U[b], Cm[b], rings[b], q)
                n_decode += 1
        m.step_mixed(torch.from_numpy(phase).to(dev), tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
        torch.cuda.synchronize()
        got = o.cpu().numpy()
        assert np.all(np.isfinite(got))
        worst = max(worst, harness.rel_err(got, ref))
    m.check_status()
    assert n_flush >= 3 * w.batch and n_decode > n_flush                          # the calls really were mixed
    assert worst <= (2e-4 if coef else FP32_GUARD), worst
    assert harness.rel_err(m.state.cpu().numpy(), np.stack(S)) <= FP32_GUARD
    assert harness.rel_err(m.sketch.cpu().numpy().transpose(0, 1, 3, 2), np.stack(U)) <= FP32_GUARD


def test_mixed_step_with_uniform_phases_equals_the_lock_step_calls():
    """All sequences at the same phase: sketchssm_step_mixed must reproduce decode_step / state_update."""
    dev = _dev()
    w = synth.Workload("t", "gdn", 6, 2, 128, 128, 16, 8, 0, "bf16", 139, basis="qr")
    ma, *_ = make_layer(w)
    mb, *_ = make_layer(w)
    ma.tune("update_impl", 1); mb.tune("update_impl", 1)       # the mixed step flushes on CUDA cores: compare like with like
    ma.state_update(0); mb.state_update(0)
    oa, ob = ma.new_output(), mb.new_output()
    for t in range(2 * w.buf_len):
        tt = harness.token_tensors(w, synth.step_inputs(w, 0, t), dev)
        n = t % w.buf_len
        args = (tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"])
        if n < w.buf_len - 1:
            ma.decode_step(n, *args, oa)
            ph = torch.full((w.batch,), n, dtype=torch.int32, device=dev)
        else:
            ma.state_update(n, *args, oa)
            ph = torch.full((w.batch,), -(n + 1), dtype=torch.int32, device=dev)
        mb.step_mixed(ph, *args, ob)
        assert torch.equal(oa, ob), t
    assert torch.equal(ma.state, mb.state) and torch.equal(ma.sketch, mb.sketch) and torch.equal(ma.ring, mb.ring)


@pytest.mark.parametrize("kind", synth.KINDS)
@pytest.mark.parametrize("io", ["bf16", "f32"])
def test_value_width_80(kind, io):
    """K = 128, V = 80 (20 lanes of 4 value elements in the decode kernel, one 80-column tile in the flush kernel)."""
    w = synth.Workload("t", kind, 7, 3, 128, 80, 16, 8, 0, io, 141, basis="qr")
    guard = 1e-5 if io == "f32" else FP32_GUARD
    check(run_schedule(w, 2 * w.buf_len + 3, max_heads=10**9), io, guard=guard)
    check(run_schedule(w, w.buf_len + 3, max_heads=10**9, mode="full_read"), io, guard=guard)
    errs = run_schedule(w, w.buf_len + 3, max_heads=10**9, coef="pivot")
    assert errs["out"] <= 2e-4 and errs["C"] <= 1e-3, errs
