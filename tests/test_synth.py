"""Checks of the seeded input generator: determinism, shapes, value ranges, I/O precision."""
import numpy as np
import pytest
import torch

from paper_2609_33051_b200 import synth


def small(kind, io="bf16"):
    return synth.Workload("t", kind, 3, 2, 32, 16, 4, 4, 8, io, 77)


@pytest.mark.parametrize("kind", synth.KINDS)
def test_step_inputs_are_deterministic_and_shaped(kind):
    w = small(kind)
    a, b = synth.step_inputs(w, 0, 5), synth.step_inputs(w, 0, 5)
    for key in a:
        np.testing.assert_array_equal(a[key], b[key])
        assert a[key].dtype == np.float32
    assert a["q"].shape == (3, 2, 32) and a["v"].shape == (3, 2, 16) and a["beta"].shape == (3, 2)
    assert a["decay"].shape == ((3, 2, 32) if kind == "kda" else (3, 2))
    c = synth.step_inputs(w, 0, 6)
    assert not np.array_equal(a["q"], c["q"])
    assert not np.array_equal(a["q"], synth.step_inputs(w, 1, 5)["q"])
    assert np.all(a["decay"] > 0) and np.all(a["decay"] < 1)
    assert np.all(a["beta"] > 0)
    if kind != "mamba2":
        assert np.all(a["beta"] < 1)
        np.testing.assert_allclose(np.linalg.norm(a["k"], axis=-1), 1.0, atol=1e-2)


def test_bf16_values_are_exactly_representable():
    w = small("kda")
    x = synth.step_inputs(w, 0, 0)
    for key in ("q", "k", "v", "beta", "decay"):
        t = torch.from_numpy(x[key])
        assert torch.equal(t.to(torch.bfloat16).to(torch.float32), t), key
    w32 = small("gdn", "f32")
    q = synth.step_inputs(w32, 0, 0)["q"]
    assert not torch.equal(torch.from_numpy(q).to(torch.bfloat16).to(torch.float32), torch.from_numpy(q))


def test_mamba2_decay_follows_its_recipe():
    w = small("mamba2")
    x = synth.step_inputs(w, 0, 3)
    al = synth.a_log(w, 0)
    assert np.all(al >= 0) and np.all(al <= 2.7)
    ref = np.exp(-x["beta"].astype(np.float64) * np.exp(al.astype(np.float64))[None, :])
    np.testing.assert_allclose(x["decay"], ref.astype(np.float32), rtol=1e-6)


def test_qr_basis_is_orthonormal_and_calibration_queries_are_low_rank_plus_noise():
    w = synth.CONFIGS["c1_gdn_tiny"]
    Om = synth.qr_basis(w)
    assert Om.shape == (4, 64, 8)
    for h in range(4):
        np.testing.assert_allclose(Om[h].T @ Om[h], np.eye(8), atol=1e-5)
    w2 = small("gdn").replace(calib_n=512, calib_rank=5)
    Q = synth.calibration_queries(w2, 0, 1)
    assert Q.shape == (512, 32)
    s = np.linalg.svd(Q, compute_uv=False)
    assert s[4] > 5 * s[5]            # rank-5 signal well above the 0.05 noise floor


def test_state_init_scale_and_configs():
    w = small("gdn")
    S = synth.initial_state(w)
    assert S.shape == (3, 2, 32, 16) and abs(S.std() - 0.02) < 0.003
    c = synth.CONFIGS
    assert (c["c2_mamba2"].batch, c["c2_mamba2"].heads, c["c2_mamba2"].dk, c["c2_mamba2"].dv) == (256, 64, 128, 64)
    assert (c["c4_kda"].buf_len, c["c4_kda"].rank) == (32, 16)
    p = synth.sweep_point(2048, 64, 32)
    assert (p.batch, p.buf_len, p.rank, p.layers, p.kind) == (2048, 64, 32, 48, "mamba2")
