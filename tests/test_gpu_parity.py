"""Parity of the CUDA library (through the C ABI) with the CPU oracle, element by element.

Norm: per decode step, max |o_gpu - o_oracle| over max |o_oracle| across all compared (b, h, v);
the same for the final state S and sketch U.  Bars: 1e-5 for float32 I/O, 2e-3 for bfloat16 I/O
(float32 state and accumulation in both cases).
"""
import numpy as np
import pytest
import torch

from oracle import sketchssm_oracle as orc
from paper_2609_33051_b200 import synth
from tests import harness

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}
# the kernels accumulate in float32 on the same input bits, so the observed error sits far below the
# bf16 bar; a regression guard at this level catches wrong-but-small mistakes the bar would hide
FP32_GUARD = 5e-5


def _device():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch.device("cuda", 0)


def make_layer(w, layer=0, out="f32", coef=None, lam=0.1, pivots=4, sketch="f32", erase=False):
    """coef: None (fixed offline map, an input), "pivot" or "ridge" (state-dependent map, rebuilt by every flush).
    sketch: storage type of U and C ("bf16": the fixed map is rounded to bfloat16 before either side sees it).
    erase: the decode step forms c_t from projected erase vectors (Eq. 44-45) instead of the swept query."""
    from paper_2609_33051_b200.binding import SketchSSM
    dev = _device()
    Om, C = harness.basis_for(w, layer)
    m = SketchSSM(w.kind, w.batch, w.heads, w.dk, w.dv, w.rank, w.buf_len, io=w.io, out=out, device=0,
                  coef_per_seq=coef is not None, coef_pivots=pivots if coef == "pivot" else 0, ridge_lambda=lam, sketch=sketch,
                  erase_factors=erase)
    if sketch == "bf16":
        C = synth.round_io(C, "bf16")
    S0 = synth.initial_state(w, layer)
    m.state.copy_(torch.from_numpy(S0))
    m.omega.copy_(torch.from_numpy(Om))
    if coef is None:
        m.coef.copy_(torch.from_numpy(C))            # (exact narrowing when the map is stored as bfloat16)
    return m, S0, Om, C, dev


def run_schedule(w, steps, max_heads=64, mode="sketch", tune=None, out="f32", input_batch=None, per_element=None,
                 coef=None, lam=0.1, pivots=4, sketch="f32", erase=False):
    """Algorithm 1 on GPU and oracle; returns the worst per-step relative error and the final-state errors.

    input_batch: generate the token inputs for this many batch entries and repeat them over the batch (the initial
    states stay distinct per entry, so every entry still follows its own trajectory); keeps the host-side input
    generation of the largest batches short.  per_element: optional callable(got, ref) run on every step's outputs.
    errs["windows"] lists the worst output error of each window, so drift across flushes is visible.
    coef: None, or "pivot" / "ridge": the state-dependent coefficient map, which both sides rebuild from the state at
    the initial sketch construction and at every flush (errs["C"]: the final maps).
    erase: decode through the projected erase vectors; errs["f"] compares the vector every decode step stores with the
    oracle's f_s of that token (Eq. 45)."""
    m, S0, Om, C, dev = make_layer(w, out=out, coef=coef, lam=lam, pivots=pivots, sketch=sketch, erase=erase)
    if erase:
        m.erase.fill_(float("nan"))                     # the buffer needs no initialisation: stale contents must not matter
        errs_f = 0.0
    stored = (lambda u: orc.round_bf16(u)) if sketch == "bf16" else (lambda u: u)      # the oracle rounds U where the flush stores it
    for key, val in (tune or {}).items():
        m.tune(key, val)
    bs, hs = harness.select_heads(w, max_heads)
    wi = w if not input_batch or input_batch >= w.batch else w.replace(batch=input_batch)
    reps = w.batch // wi.batch
    assert reps * wi.batch == w.batch
    bsi = bs % wi.batch
    m.state_update(0)                                   # initial sketch from the prefilled state
    S = S0[bs, hs].astype(np.float64)
    Om_s, C_s = Om[hs].astype(np.float64), C[hs].astype(np.float64)
    U = stored(orc.sketch_of(S, Om_s))
    errs = {"u0": harness.rel_err(m.sketch.float().cpu().numpy()[bs, hs].transpose(0, 2, 1), U)}
    def maps(Snow, Unow):
        """the state-dependent maps as the library stores them: from the state and, with bfloat16 storage, from the
        rounded sketch, then rounded themselves"""
        if sketch == "bf16":
            return stored(orc.coefficient_maps(Snow, Om_s, coef, lam, pivots, U=Unow))
        return orc.coefficient_maps(Snow, Om_s, coef, lam, pivots)
    if coef is not None:
        C_s = maps(S, U)
        errs["c0"] = harness.rel_err(m.coef.float().cpu().numpy()[bs, hs], C_s)
    worst = 0.0
    windows = []
    ring = []
    o_dev = m.new_output()
    L = w.buf_len
    bs_t, hs_t = torch.from_numpy(bs).to(dev), torch.from_numpy(hs).to(dev)
    for t in range(steps):
        x = synth.step_inputs(wi, 0, t)
        tt = harness.token_tensors(wi, x, dev)
        if reps > 1:
            tt = {k: v.repeat(reps, *([1] * (v.dim() - 1))).contiguous() for k, v in tt.items()}
        n = t % L
        ring.append(harness.oracle_token(x, bsi, hs))
        q = x["q"][bsi, hs].astype(np.float64)
        if n < L - 1:
            if mode == "sketch":
                m.decode_step(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o_dev)
                # (erase vectors stored as bfloat16 are rounded where they are stored, on both sides)
                f_store = orc.round_bf16 if (erase and sketch == "bf16") else None
                ref = orc.decode_step(w.kind, U, C_s, ring, q, erase_store=f_store)
                if erase:
                    f_ref = orc.projected_erase_vectors(w.kind, ring, C_s, store=f_store)[0][-1]
                    errs_f = max(errs_f, harness.rel_err(m.erase[bs_t, hs_t, n].float().cpu().numpy(), f_ref))
            else:
                m.full_read_decode(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o_dev)
                ref = orc.full_read_decode(w.kind, S, ring, q)
        else:
            m.state_update(n, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o_dev)
            S, U, ref = orc.state_update(w.kind, S, ring, Om_s, q)
            U = stored(U)
            if coef is not None:
                C_s = maps(S, U)
            ring = []
        # the two-kernel decode launches twice; a GDN flush of more than 16 tokens is one launch per block of 16
        assert 1 <= m.last_launch_count() <= max(2, (w.buf_len + 15) // 16) + (1 if coef else 0)
        got = o_dev[bs_t, hs_t].float().cpu().numpy()
        assert np.all(np.isfinite(got))
        if per_element is not None:
            per_element(got, ref)
        e = harness.rel_err(got, ref)
        worst = max(worst, e)
        if n == 0:
            windows.append(0.0)
        windows[-1] = max(windows[-1], e)
    m.check_status()
    errs["out"] = worst
    errs["S"] = harness.rel_err(m.state[bs_t, hs_t].cpu().numpy(), S)
    errs["U"] = harness.rel_err(m.sketch[bs_t, hs_t].float().cpu().numpy().transpose(0, 2, 1), U)
    if sketch == "bf16":         # how many stored sketch elements differ from the oracle's rounding (a value next to a rounding
        got_u = m.sketch[bs_t, hs_t].float().cpu().numpy().transpose(0, 2, 1)         # boundary may fall on the other side)
        errs["u_mismatch"] = float(np.mean(got_u != U))
    if coef is not None:
        errs["C"] = harness.rel_err(m.coef[bs_t, hs_t].float().cpu().numpy(), C_s)
    if erase:
        errs["f"] = errs_f
    errs["windows"] = windows
    return errs


def check(errs, io, guard=FP32_GUARD):
    for key, e in errs.items():
        if key in ("windows", "u_mismatch"):
            continue
        assert e <= TOL[io], (key, e, errs)
        assert e <= guard, (key, e, errs)


# ---------------------------------------------------------------------------------------------
# config 1 in full, and reduced-batch versions of configs 2-4 (all heads compared)
# ---------------------------------------------------------------------------------------------

def test_config1_gdn_tiny_full_run():
    w = synth.CONFIGS["c1_gdn_tiny"]
    errs = run_schedule(w, w.steps, max_heads=10**9)
    check(errs, "f32", guard=1e-5)


@pytest.mark.parametrize("name,batch,steps", [("c2_mamba2", 6, 40), ("c3_gdn", 5, 40), ("c4_kda", 3, 70)])
def test_configs_2_to_4_reduced_batch(name, batch, steps):
    w = synth.CONFIGS[name].replace(batch=batch, heads=4)
    check(run_schedule(w, steps, max_heads=10**9), w.io)


@pytest.mark.parametrize("name", ["c2_mamba2", "c3_gdn", "c4_kda"])
def test_full_read_decode_reduced_batch(name):
    w = synth.CONFIGS[name].replace(batch=5, heads=3)
    check(run_schedule(w, w.buf_len + 5, max_heads=10**9, mode="full_read"), w.io)


# ---------------------------------------------------------------------------------------------
# shapes, ranks, window lengths, launch tunings
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kind", synth.KINDS)
@pytest.mark.parametrize("dk,dv", [(64, 64), (64, 128), (128, 64), (128, 128)])
@pytest.mark.parametrize("io", ["f32", "bf16"])
def test_shapes_and_dtypes(kind, dk, dv, io):
    w = synth.Workload("t", kind, 3, 2, dk, dv, 8, 8, 20, io, 4242, basis="qr")
    check(run_schedule(w, 20, max_heads=10**9), io, guard=1e-5 if io == "f32" else FP32_GUARD)
    check(run_schedule(w, 11, max_heads=10**9, mode="full_read"), io, guard=1e-5 if io == "f32" else FP32_GUARD)


@pytest.mark.parametrize("kind", synth.KINDS)
@pytest.mark.parametrize("rank,buf_len", [(1, 4), (5, 12), (32, 64), (64, 8)])
def test_ranks_and_window_lengths(kind, rank, buf_len):
    w = synth.Workload("t", kind, 2, 3, 128, 64, rank, buf_len, 0, "bf16", 99, basis="qr")
    check(run_schedule(w, buf_len + 3, max_heads=10**9), "bf16")


@pytest.mark.parametrize("kind", synth.KINDS)
@pytest.mark.parametrize("tune", [{"decode_impl": 1, "decode_stages": 1, "decode_batches_per_cta": 1},
                                  {"decode_impl": 1, "decode_stages": 2, "decode_batches_per_cta": 7},
                                  {"decode_impl": 0, "decode_stages": 2, "decode_warps_per_cta": 2},
                                  {"decode_impl": 0, "decode_stages": 1, "decode_max_warps_per_sm": 4},
                                  {"update_impl": 1}])
def test_launch_tunings_and_ragged_batches(kind, tune):
    w = synth.Workload("t", kind, 37, 3, 128, 128, 16, 16, 0, "bf16", 7, basis="qr")
    check(run_schedule(w, 20, max_heads=10**9, tune=tune), "bf16")
    check(run_schedule(w, 18, max_heads=10**9, mode="full_read", tune=tune), "bf16")


@pytest.mark.parametrize("dv,rank,buf_len", [(64, 16, 16), (128, 40, 48), (64, 5, 64)])
def test_mamba2_tensor_core_variants(dv, rank, buf_len):
    """The Mamba-2 flush on CUDA cores and as the single-group tcgen05 kernel (ranks above 32 use it by default)."""
    w = synth.Workload("t", "mamba2", 6, 3, 128, dv, rank, buf_len, 0, "bf16", 77, basis="qr")
    check(run_schedule(w, buf_len + 5, max_heads=10**9, tune={"update_impl": 1}), "bf16")
    check(run_schedule(w, buf_len + 5, max_heads=10**9, tune={"update_impl": 3}), "bf16")     # single-group tcgen05 kernel


@pytest.mark.parametrize("tune", [{}, {"decode_max_warps_per_sm": 8}, {"pdl": 0}])
@pytest.mark.parametrize("dv,batch,heads,buf_len,rank", [(64, 64, 24, 16, 16), (128, 40, 20, 8, 16), (64, 64, 24, 16, 32),
                                                         (128, 24, 10, 12, 24), (64, 48, 12, 40, 8)])
def test_mamba2_update_several_tiles_per_cta(tune, dv, batch, heads, buf_len, rank):
    """Warp-specialised tcgen05 update with every CTA walking several tiles (double-buffered accumulators, operand
    sets and W buffers; head index changes inside a CTA's range), over two windows."""
    w = synth.Workload("t", "mamba2", batch, heads, 128, dv, rank, buf_len, 0, "bf16", 79, basis="qr")
    check(run_schedule(w, 2 * buf_len + 2, max_heads=96, tune=tune), "bf16")


@pytest.mark.parametrize("tune", [{}, {"decode_max_warps_per_sm": 10}, {"pdl": 0}])
@pytest.mark.parametrize("batch,heads,rank,buf_len", [(5, 3, 16, 16), (40, 20, 16, 16), (33, 7, 8, 12), (6, 2, 5, 4),
                                                      (12, 4, 16, 32), (7, 3, 12, 40), (5, 2, 16, 64)])
def test_gdn_warp_specialised_update(tune, batch, heads, rank, buf_len):
    """Warp-specialised tcgen05 flush of the gated delta rule (two passes over the state, interleaved across tiles,
    tiles claimed at run time; windows of more than 16 tokens replayed in blocks of 16) against the oracle's
    token-by-token replay, over two windows."""
    w = synth.Workload("t", "gdn", batch, heads, 128, 128, rank, buf_len, 0, "bf16", 93, basis="qr")
    check(run_schedule(w, 2 * buf_len + 3, max_heads=96, tune=tune), "bf16")


@pytest.mark.parametrize("tune", [{}, {"decode_stages": 2}, {"pdl": 0}])
@pytest.mark.parametrize("batch,heads,rank,buf_len", [(5, 3, 16, 32), (40, 20, 16, 16), (33, 7, 8, 12), (6, 2, 5, 4),
                                                      (12, 4, 16, 32), (7, 3, 12, 40), (5, 2, 16, 64), (150, 3, 16, 32)])
def test_kda_warp_specialised_update(tune, batch, heads, rank, buf_len):
    """Warp-specialised tcgen05 flush of the delta rule with per-channel decay (WY form with vector decays, up to 32 tokens
    per pass, tiles claimed at run time, one CTA per SM so the largest case gives every CTA several tiles) against the
    oracle's token-by-token replay, over two windows."""
    w = synth.Workload("t", "kda", batch, heads, 128, 128, rank, buf_len, 0, "bf16", 95, basis="qr")
    check(run_schedule(w, 2 * buf_len + 3, max_heads=96, tune=tune), "bf16")


@pytest.mark.parametrize("kind,dv,buf_len,fills", [("mamba2", 64, 32, (0, 1, 15, 16, 17, 31)), ("mamba2", 128, 64, (16, 32, 47, 48, 63)),
                                                    ("gdn", 128, 16, (0, 1, 7, 15)), ("gdn", 128, 32, (3, 15, 16, 31)),
                                                    ("gdn", 128, 64, (17, 32, 33, 48, 63)),
                                                    ("kda", 128, 32, (0, 1, 7, 15, 16, 17, 31)), ("kda", 128, 64, (31, 32, 33, 47, 63))])
def test_flush_at_any_ring_fill(kind, dv, buf_len, fills):
    """state_update with n_before tokens in the ring plus the current token, for fills around the tensor-core kernels'
    block boundaries (16 tokens per block) and beyond their domains, and a replay without a current token."""
    dev = _device()
    w = synth.Workload("t", kind, 6, 3, 128, dv, 16, buf_len, 0, "bf16", 23, basis="qr")
    bs, hs = harness.select_heads(w, 10**9)
    toks = [synth.step_inputs(w, 0, t) for t in range(buf_len)]
    for n_before in fills:
        for with_token in ((True, False) if n_before > 0 else (True,)):
            m, S0, Om, C, _ = make_layer(w)
            m.state_update(0)
            o = m.new_output()
            S = S0[bs, hs].astype(np.float64)
            Om_s = Om[hs].astype(np.float64)
            ring = []
            for t in range(n_before):
                tt = harness.token_tensors(w, toks[t], dev)
                m.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
                ring.append(harness.oracle_token(toks[t], bs, hs))
            x = toks[n_before if with_token else n_before - 1]
            tt = harness.token_tensors(w, x, dev)
            q = x["q"][bs, hs].astype(np.float64)
            if with_token:
                ring.append(harness.oracle_token(x, bs, hs))
                m.state_update(n_before, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
                S_ref, U_ref, o_ref = orc.state_update(w.kind, S, ring, Om_s, q)
                got_o = o.float().cpu().numpy()[bs, hs]
                assert harness.rel_err(got_o, o_ref) <= TOL["bf16"], (n_before, with_token)
            else:
                m.state_update(n_before)
                S_ref, U_ref, _ = orc.state_update(w.kind, S, ring, Om_s, q)
            m.check_status()
            assert harness.rel_err(m.state.cpu().numpy()[bs, hs], S_ref) <= FP32_GUARD, (n_before, with_token)
            assert harness.rel_err(m.sketch.cpu().numpy()[bs, hs].transpose(0, 2, 1), U_ref) <= FP32_GUARD, (n_before, with_token)


def test_bf16_output_mode():
    """A bf16-stored output carries its own rounding on top of the arithmetic error; checked element by element:
    |o_gpu - o_ref| <= 2e-3 * max|o_ref| + 2^-8 |o_ref_i| for every output element of every step."""
    w = synth.Workload("t", "gdn", 4, 2, 128, 128, 16, 8, 0, "bf16", 5, basis="qr")

    def per_element(got, ref):
        bound = 2e-3 * np.abs(ref).max() + 2.0 ** -8 * np.abs(ref)
        assert np.all(np.abs(got.astype(np.float64) - ref) <= bound)

    errs = run_schedule(w, 12, max_heads=10**9, out="bf16", per_element=per_element)
    assert errs["S"] <= FP32_GUARD and errs["U"] <= FP32_GUARD


@pytest.mark.parametrize("kind,dv", [("mamba2", 64), ("gdn", 128), ("kda", 128), ("mamba2", 80)])
def test_bf16_sketch_storage(kind, dv):
    """U and C stored as bfloat16 (the paper's storage): the oracle rounds U at the same point, after the flush has formed
    it.  The stored sketch agrees with the oracle's to one bfloat16 spacing everywhere and bit for bit almost everywhere
    (an fp32 value next to a rounding boundary may fall on the other side of it); outputs keep the 2e-3 bar plus the half
    spacing 2^-9 such an element can contribute."""
    w = synth.Workload("t", kind, 6, 3, 128, dv, 16, 8, 0, "bf16", 151, basis="qr")
    errs = run_schedule(w, 2 * w.buf_len + 3, max_heads=10**9, sketch="bf16")
    assert errs["out"] <= 2e-3 + 2.0 ** -9, errs
    assert errs["S"] <= FP32_GUARD, errs
    assert errs["U"] <= 2.0 ** -7 and errs["u0"] <= 2.0 ** -7 and errs["u_mismatch"] <= 2e-2, errs
    # the mode halves the sketch and map bytes
    from paper_2609_33051_b200.binding import SketchSSM
    m = SketchSSM(kind, 2, 2, 128, dv, 16, 8, device=0, sketch="bf16")
    assert m.sizes.sketch_bytes == 2 * 2 * 16 * dv * 2 and m.sizes.coef_bytes == 2 * 16 * 128 * 2
    m = SketchSSM(kind, 2, 2, 128, dv, 16, 8, device=0, sketch="bf16", coef_per_seq=True)
    assert m.sizes.coef_bytes == 2 * 2 * 16 * 128 * 2


# ---------------------------------------------------------------------------------------------
# special cases the method has
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kind", synth.KINDS)
def test_identity_basis_gives_exact_read(kind):
    """r = K, Omega = I, C = I: the sketch path equals the full-read path and the recurrence itself."""
    from paper_2609_33051_b200.binding import SketchSSM
    dev = _device()
    w = synth.Workload("t", kind, 3, 2, 64, 64, 64, 8, 0, "f32", 31)
    m = SketchSSM(kind, w.batch, w.heads, 64, 64, 64, 8, io="f32", device=0)
    S0 = synth.initial_state(w)
    eye = np.broadcast_to(np.eye(64, dtype=np.float32), (w.heads, 64, 64)).copy()
    m.state.copy_(torch.from_numpy(S0)); m.omega.copy_(torch.from_numpy(eye)); m.coef.copy_(torch.from_numpy(eye))
    m.state_update(0)
    np.testing.assert_allclose(m.sketch.cpu().numpy(), S0, rtol=0, atol=1e-7)   # U[g, v] = S[g, v]
    S = S0.astype(np.float64)
    o1, o2 = m.new_output(), m.new_output()
    for t in range(7):
        x = synth.step_inputs(w, 0, t)
        tt = harness.token_tensors(w, x, dev)
        m.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o1, flags=1)   # NO_APPEND
        m.full_read_decode(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o2)
        S = orc.transition(kind, S, x["k"], x["v"], x["beta"], x["decay"])
        ref = orc.exact_read(S, x["q"])
        assert harness.rel_err(o1.cpu().numpy(), ref) <= 1e-5
        assert harness.rel_err(o2.cpu().numpy(), ref) <= 1e-5
    m.check_status()


@pytest.mark.parametrize("kind", synth.KINDS)
def test_replay_equals_single_token_updates_and_flags(kind):
    """Replaying L buffered tokens equals L updates of one token; NO_SKETCH leaves U alone;
    a replay without a current token (n_before = L) works; the ring holds what was appended."""
    from paper_2609_33051_b200.binding import SketchSSM, NO_SKETCH
    dev = _device()
    w = synth.Workload("t", kind, 4, 3, 128, 64, 8, 8, 0, "bf16", 17, basis="qr")
    ma, S0, Om, C, _ = make_layer(w)
    mb, *_ = make_layer(w)
    ma.state_update(0); mb.state_update(0)
    o = ma.new_output()
    toks = [harness.token_tensors(w, synth.step_inputs(w, 0, t), dev) for t in range(w.buf_len)]
    for t, tt in enumerate(toks):                      # a: buffer all L tokens (decode steps), replay at once
        ma.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o) if t < w.buf_len - 1 else None
    # ring contents are exactly what was appended
    rk, rv, rb, rd = ma.ring_views()
    for t in range(w.buf_len - 1):
        assert torch.equal(rk[:, :, t], toks[t]["k"]) and torch.equal(rv[:, :, t], toks[t]["v"])
        assert torch.equal(rb[:, :, t], toks[t]["beta"]) and torch.equal(rd[:, :, t], toks[t]["decay"])
    last = toks[-1]
    sketch_before = ma.sketch.clone()
    ma.state_update(w.buf_len - 1, last["q"], last["k"], last["v"], last["beta"], last["decay"], o, flags=NO_SKETCH)
    assert torch.equal(ma.sketch, sketch_before)
    ma.state_update(0)                                  # now refresh the sketch from the updated state
    ob = mb.new_output()
    for tt in toks:                                     # b: one-token updates ("standard" execution)
        mb.state_update(0, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], ob)
    assert harness.rel_err(ma.state.cpu().numpy(), mb.state.cpu().numpy().astype(np.float64)) <= 2e-5
    assert harness.rel_err(ma.sketch.cpu().numpy(), mb.sketch.cpu().numpy().astype(np.float64)) <= 2e-5
    assert harness.rel_err(o.cpu().numpy(), ob.cpu().numpy().astype(np.float64)) <= 2e-5
    # c: replay a full ring without a current token
    mc, *_ = make_layer(w)
    mc.state_update(0)
    w2 = w.replace(buf_len=8)
    for t, tt in enumerate(toks[:-1]):
        mc.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
    # append the last one by a decode step with n_before = L-1, then replay with n_before = L and no token
    mc.decode_step(w.buf_len - 1, last["q"], last["k"], last["v"], last["beta"], last["decay"], o)
    mc.state_update(w.buf_len)
    assert harness.rel_err(mc.state.cpu().numpy(), mb.state.cpu().numpy().astype(np.float64)) <= 2e-5
    for m in (ma, mb, mc):
        m.check_status()


@pytest.mark.parametrize("kind", synth.KINDS)
def test_empty_buffer_output_is_U_C_q(kind):
    """A token with beta = 0 and unit decay contributes nothing: o = U C q_t."""
    dev = _device()
    w = synth.Workload("t", kind, 3, 2, 128, 128, 16, 8, 0, "f32", 23, basis="qr")
    m, S0, Om, C, _ = make_layer(w)
    m.state_update(0)
    x = synth.step_inputs(w, 0, 0)
    x["beta"] = np.zeros_like(x["beta"]); x["decay"] = np.ones_like(x["decay"])
    tt = harness.token_tensors(w, x, dev)
    o = m.new_output()
    m.decode_step(0, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
    U = orc.sketch_of(S0.astype(np.float64), Om.astype(np.float64)[None])
    ref = np.einsum("bhvg,bhg->bhv", U, np.einsum("hgk,bhk->bhg", C.astype(np.float64), x["q"].astype(np.float64)))
    assert harness.rel_err(o.cpu().numpy(), ref) <= 1e-5
    m.check_status()


def test_checkpoint_resume_mid_window():
    """(S, ring, n) is the whole recurrent truth: restoring them and rebuilding U continues identically."""
    dev = _device()
    w = synth.Workload("t", "kda", 3, 2, 128, 128, 16, 8, 0, "bf16", 29, basis="qr")
    ma, *_ = make_layer(w)
    ma.state_update(0)
    oa, ob = ma.new_output(), ma.new_output()
    toks = [harness.token_tensors(w, synth.step_inputs(w, 0, t), dev) for t in range(8)]
    for t in range(3):
        tt = toks[t]
        ma.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], oa)
    mb, *_ = make_layer(w)
    mb.state.copy_(ma.state); mb.ring.copy_(ma.ring)
    mb.state_update(0)                                   # rebuild U from the restored state
    for t in range(3, 8):
        tt = toks[t]
        for m, o in ((ma, oa), (mb, ob)):
            if t < 7:
                m.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
            else:
                m.state_update(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
        assert torch.equal(oa, ob)
    assert torch.equal(ma.state, mb.state) and torch.equal(ma.sketch, mb.sketch)


def test_repeat_runs_are_bitwise_identical():
    w = synth.CONFIGS["c3_gdn"].replace(batch=9, heads=2)
    outs = []
    for _ in range(2):
        m, *_ = make_layer(w)
        dev = _device()
        m.state_update(0)
        o = m.new_output()
        for t in range(16):
            tt = harness.token_tensors(w, synth.step_inputs(w, 0, t), dev)
            if t < 15:
                m.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
            else:
                m.state_update(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], o)
        outs.append((o.clone(), m.state.clone(), m.sketch.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_window_replays_from_a_cuda_graph():
    """Every call only enqueues work on the given stream, so a window can be captured in a CUDA graph; replaying it
    reproduces the eager results bit for bit (the update kernels' run-time tile scheduler leaves its counters zero)."""
    dev = _device()
    w = synth.Workload("t", "mamba2", 8, 4, 128, 64, 16, 8, 0, "bf16", 31, basis="qr")
    toks = [harness.token_tensors(w, synth.step_inputs(w, 0, t), dev) for t in range(w.buf_len)]

    def window(m, outs):
        for t, tt in enumerate(toks):
            if t < w.buf_len - 1:
                m.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], outs[t])
            else:
                m.state_update(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], outs[t])

    me, *_ = make_layer(w)
    mg, *_ = make_layer(w)
    me.state_update(0); mg.state_update(0)
    oe = [me.new_output() for _ in toks]
    og = [mg.new_output() for _ in toks]
    window(mg, og)                                  # warm-up outside capture (first-call set-up), then restore
    torch.cuda.synchronize()
    mg.state.copy_(me.state); mg.sketch.copy_(me.sketch)
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=s):
        window(mg, og)
    torch.cuda.current_stream().wait_stream(s)
    for rep in range(2):                            # two windows eagerly and from the graph
        window(me, oe)
        g.replay()
        torch.cuda.synchronize()
        for a, b in zip(oe, og):
            assert torch.equal(a, b)
        assert torch.equal(me.state, mg.state) and torch.equal(me.sketch, mg.sketch)
    me.check_status(); mg.check_status()


@pytest.mark.parametrize("kind,dv", [("mamba2", 64), ("gdn", 128)])
def test_decode_after_update_sees_the_new_sketch_with_dependent_launch(kind, dv):
    """With programmatic dependent launch a decode step requests sketch rows before it waits for its predecessor in
    the stream, unless that predecessor is a state update of its own context (the only writer of the sketch).  Windows
    run back to back without synchronisation, and a decode step issued directly after a flush, give bit-identical
    results with dependent launch on and off."""
    dev = _device()
    w = synth.Workload("t", kind, 64, 8, 128, dv, 16, 8, 0, "bf16", 37, basis="qr")
    toks = [harness.token_tensors(w, synth.step_inputs(w, 0, t), dev) for t in range(w.buf_len)]
    results = []
    for pdl in (1, 0):
        m, *_ = make_layer(w)
        m.tune("pdl", pdl)
        m.state_update(0)
        outs = [m.new_output() for _ in range(3 * w.buf_len + 1)]
        i = 0
        for rep in range(3):
            for t, tt in enumerate(toks):
                if t < w.buf_len - 1:
                    m.decode_step(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], outs[i])
                else:
                    m.state_update(t, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], outs[i])
                i += 1
        # directly after the flush: a decode step over the first three (still stored) ring slots, nothing appended
        tt = toks[3]
        m.decode_step(3, tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"], outs[i], flags=1)
        torch.cuda.synchronize()
        m.check_status()
        results.append(([o.clone() for o in outs], m.state.clone(), m.sketch.clone()))
    (oa, sa, ua), (ob, sb, ub) = results
    for a, b in zip(oa, ob):
        assert torch.equal(a, b)
    assert torch.equal(sa, sb) and torch.equal(ua, ub)
