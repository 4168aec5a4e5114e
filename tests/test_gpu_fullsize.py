"""Parity at the workloads' full sizes and full lengths, in the launch configuration the benchmark times.

The whole batch runs on the GPU; the oracle follows a deterministic sample of (batch, head) pairs (heads are
independent, so sampled parity is exact parity for those heads), including the corners of the batch.  Same norm and
bars as tests/test_gpu_parity.py.  Configs 2-4 run all 256 decode steps (16 or 8 windows), so the error that the
tensor-core flushes feed back through the state is measured over the whole run; the worst output error per window is
printed (pytest -s) and must stay under the bar in every window.
"""
import pytest

from paper_2609_33051_b200 import synth
from tests.test_gpu_parity import FP32_GUARD, TOL, check, run_schedule

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c2_mamba2", "c3_gdn", "c4_kda"])
def test_configs_2_to_4_full_batch_full_length(name):
    w = synth.CONFIGS[name]
    errs = run_schedule(w, w.steps, max_heads=48)
    wins = errs["windows"]
    assert len(wins) == w.steps // w.buf_len
    print(f"\n{name}: worst output error after window " +
          ", ".join(f"{i}: {wins[i - 1]:.2e}" for i in (1, 2, 4, 8, 16) if i <= len(wins)) +
          f"; final S {errs['S']:.2e}, U {errs['U']:.2e}")
    check(errs, w.io)
    assert max(wins) <= FP32_GUARD
    # no systematic growth: the last window is no worse than a few times the first
    assert wins[-1] <= max(4.0 * wins[0], 2e-5), wins


@pytest.mark.parametrize("name", ["c2_mamba2", "c3_gdn", "c4_kda"])
def test_full_read_decode_full_batch_sampled_heads(name):
    w = synth.CONFIGS[name]
    check(run_schedule(w, w.buf_len + 3, max_heads=32, mode="full_read"), w.io)


# the eight corners of the sweep (batch 64 / 2048, L 4 / 64, r 8 / 32), one batch-1024 point, and the two points the
# benchmark reports as its headline and as the paper's regime
@pytest.mark.parametrize("batch,buf_len,rank", [(64, 4, 8), (64, 4, 32), (64, 64, 8), (64, 64, 32),
                                                (2048, 4, 8), (2048, 4, 32), (2048, 64, 8), (2048, 64, 32),
                                                (1024, 16, 16), (2048, 16, 16), (256, 64, 32)])
def test_config5_sweep_points_sampled_heads(batch, buf_len, rank):
    w = synth.sweep_point(batch, buf_len, rank)
    # more than one window; token inputs of the largest batches are generated for 256 entries and repeated
    check(run_schedule(w, buf_len + 3, max_heads=32, input_batch=256), w.io)


def test_two_kernel_decode_full_batch():
    w = synth.CONFIGS["c3_gdn"]
    check(run_schedule(w, 20, max_heads=32, tune={"decode_impl": 0}), w.io)
