"""Parity at the workloads' full sizes, in the launch configuration the benchmark times.

The whole batch runs on the GPU; the oracle follows a deterministic sample of (batch, head) pairs (heads are
independent, so sampled parity is exact parity for those heads) through more than one window, including the
corners of the batch.  Same norm and bars as tests/test_gpu_parity.py.
"""
import pytest

from paper_2609_33051_b200 import synth
from tests.test_gpu_parity import check, run_schedule

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,steps", [("c2_mamba2", 35), ("c3_gdn", 35), ("c4_kda", 67)])
def test_configs_2_to_4_full_batch_sampled_heads(name, steps):
    w = synth.CONFIGS[name]
    check(run_schedule(w, steps, max_heads=48), w.io)


@pytest.mark.parametrize("name", ["c2_mamba2", "c3_gdn"])
def test_full_read_decode_full_batch_sampled_heads(name):
    w = synth.CONFIGS[name]
    check(run_schedule(w, w.buf_len + 3, max_heads=32, mode="full_read"), w.io)


@pytest.mark.parametrize("batch,buf_len,rank", [(64, 4, 8), (256, 64, 32), (2048, 16, 16)])
def test_config5_sweep_points_sampled_heads(batch, buf_len, rank):
    w = synth.sweep_point(batch, buf_len, rank)
    check(run_schedule(w, buf_len + 3, max_heads=32), w.io)


@pytest.mark.parametrize("impl", [0, 2])
def test_alternative_decode_kernels_full_batch(impl):
    w = synth.CONFIGS["c3_gdn"]
    check(run_schedule(w, 20, max_heads=32, tune={"decode_impl": impl}), w.io)
