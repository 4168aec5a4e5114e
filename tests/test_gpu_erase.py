"""Decode through projected erase vectors (Appendix C.2, Eq. 44-45) for the delta-rule kinds.

With `erase_factors` the decode step keeps f_s = C pi_s in R^r for every buffered token and forms
c_t = C (d_[t] * q_t) - sum_s f_s <l_s(t), q_t> instead of applying C to the swept effective query.  The identity is exact
for the map in force during the window, so the outputs are compared with the same oracle steps as the default path, and
every stored f_s with the oracle's recurrence (which is pinned to C times the erase factors of the WY form).
"""
import numpy as np
import pytest
import torch

from paper_2609_33051_b200 import binding, synth
from tests import harness
from tests.test_gpu_parity import FP32_GUARD, check, make_layer, run_schedule

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kind", ("gdn", "kda"))
@pytest.mark.parametrize("io", ("bf16", "f32"))
@pytest.mark.parametrize("dk,dv,rank,L", [(128, 128, 16, 16), (128, 128, 8, 32), (64, 64, 12, 8), (128, 64, 32, 8)])
def test_erase_factor_decode_matches_the_oracle(kind, io, dk, dv, rank, L):
    w = synth.Workload("t", kind, 7, 5, dk, dv, rank, L, 0, io, 211, basis="qr")
    errs = run_schedule(w, 2 * L + 3, max_heads=10**9, erase=True)
    check(errs, io)
    assert "f" in errs and errs["f"] <= FP32_GUARD, errs


@pytest.mark.parametrize("kind", ("gdn", "kda"))
@pytest.mark.parametrize("coef", ("pivot", "ridge"))
def test_erase_factors_with_the_state_dependent_map(kind, coef):
    # the map changes at every flush; inside a window it is fixed, and the erase vectors start afresh with the ring
    w = synth.Workload("t", kind, 6, 3, 128, 128, 8, 8, 0, "bf16", 223, basis="qr")
    errs = run_schedule(w, 3 * w.buf_len, max_heads=10**9, coef=coef, erase=True)
    for key in ("out", "f"):
        assert errs[key] <= 2e-4, errs
    assert errs["S"] <= FP32_GUARD and errs["U"] <= FP32_GUARD, errs


@pytest.mark.parametrize("kind", ("gdn", "kda"))
def test_erase_factors_with_bfloat16_sketch_storage(kind):
    # U, the fixed map and the erase vectors stored as bfloat16, the paper's storage (the oracle rounds U where the flush
    # stores it and every erase vector where the decode step stores it; both sides get the map already rounded).  A stored
    # value next to a rounding boundary may fall on the other side of it: the vectors are held to 2^-7 of their largest
    # element, the outputs to the bar of the bfloat16 sketch test
    w = synth.Workload("t", kind, 6, 4, 128, 128, 16, 16, 0, "bf16", 229, basis="qr")
    errs = run_schedule(w, 2 * w.buf_len + 2, max_heads=10**9, sketch="bf16", erase=True)
    assert errs["out"] <= 2e-3 + 2.0 ** -9 and errs["f"] <= 2.0 ** -7 and errs["S"] <= FP32_GUARD, errs
    m = binding.SketchSSM(kind, 2, 2, 128, 128, 16, 16, sketch="bf16", erase_factors=True, allocate=False)
    assert m.sizes.erase_bytes == 2 * 2 * 16 * 16 * 2
    with pytest.raises(binding.SketchSSMError):          # bfloat16 rows travel in 16-byte units: rank % 8 = 0
        binding.SketchSSM(kind, 2, 2, 128, 128, 12, 16, sketch="bf16", erase_factors=True, allocate=False)


@pytest.mark.parametrize("kind", ("gdn", "kda"))
def test_the_papers_storage_and_map_together_with_erase_vectors(kind):
    # state-dependent map (P = 4), bfloat16 U / C / f_s: every piece of the paper's decode configuration at once
    w = synth.Workload("t", kind, 5, 3, 128, 128, 16, 8, 0, "bf16", 233, basis="qr")
    errs = run_schedule(w, 3 * w.buf_len, max_heads=10**9, coef="pivot", sketch="bf16", erase=True)
    assert errs["out"] <= 2e-3 + 2.0 ** -9 and errs["S"] <= FP32_GUARD, errs
    assert max(errs["U"], errs["C"], errs["c0"], errs["f"]) <= 2.0 ** -7, errs


def test_erase_factors_give_the_same_outputs_as_the_swept_query():
    # same layer, same tokens, with and without the projected vectors: equal up to rounding order
    dev = torch.device("cuda", 0)
    w = synth.Workload("t", "kda", 9, 4, 128, 128, 16, 16, 0, "bf16", 227, basis="qr")
    ma, *_ = make_layer(w)
    mb, *_ = make_layer(w, erase=True)
    ma.state_update(0); mb.state_update(0)
    oa, ob = ma.new_output(), mb.new_output()
    worst = 0.0
    for t in range(2 * w.buf_len):
        tt = harness.token_tensors(w, synth.step_inputs(w, 0, t), dev)
        n = t % w.buf_len
        args = (tt["q"], tt["k"], tt["v"], tt["beta"], tt["decay"])
        if n < w.buf_len - 1:
            ma.decode_step(n, *args, oa); mb.decode_step(n, *args, ob)
        else:
            ma.state_update(n, *args, oa); mb.state_update(n, *args, ob)
        worst = max(worst, harness.rel_err(ob.cpu().numpy(), oa.cpu().numpy().astype(np.float64)))
    ma.check_status(); mb.check_status()
    assert worst <= FP32_GUARD, worst
    assert torch.equal(ma.state, mb.state)


def test_erase_factors_are_refused_where_they_do_not_apply():
    with pytest.raises(binding.SketchSSMError):          # Mamba-2 has no erase term
        binding.SketchSSM("mamba2", 2, 2, 128, 64, 16, 16, erase_factors=True, allocate=False)
    with pytest.raises(binding.SketchSSMError):          # rank must be a multiple of 4
        binding.SketchSSM("gdn", 2, 2, 128, 128, 6, 16, erase_factors=True, allocate=False)
    with pytest.raises(binding.SketchSSMError):          # windows of at most 32 tokens
        binding.SketchSSM("gdn", 2, 2, 128, 128, 16, 64, erase_factors=True, allocate=False)
    m = binding.SketchSSM("gdn", 2, 2, 128, 128, 16, 16, erase_factors=True)
    tt = [torch.zeros(2, 2, 128, dtype=torch.bfloat16, device="cuda") for _ in range(3)] + \
         [torch.zeros(2, 2, device="cuda") for _ in range(2)]
    m.tune("decode_impl", 0)                             # the two-kernel decode does not know the vectors
    with pytest.raises(binding.SketchSSMError):
        m.decode_step(0, *tt, m.new_output())
