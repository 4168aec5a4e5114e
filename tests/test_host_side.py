"""CPU tests of the host-side pieces: the product's offline calibration against the oracle's fit, the byte
accounting, and the benchmark's rank sharding under torch.distributed (gloo, world size 2)."""
import os
import subprocess
import sys

import numpy as np
import torch

from oracle import sketchssm_oracle as orc
from paper_2609_33051_b200 import calibrate, synth, traffic

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_product_calibration_matches_oracle_fit():
    w = synth.CONFIGS["c2_mamba2"].replace(calib_n=1024)
    Q = synth.calibration_queries(w, 0, 3)
    Om_p, C_p = calibrate.fit_head(torch.from_numpy(Q), w.rank)
    Om_o, lam = orc.fit_sketching_matrix(Q, np.eye(w.dk), w.rank)
    C_o = orc.offline_coefficient_map(Om_o, np.eye(w.dk))
    np.testing.assert_allclose(Om_p.numpy(), Om_o, atol=1e-8)      # same sign convention, distinct eigenvalues
    np.testing.assert_allclose(C_p.numpy(), C_o, atol=1e-8)
    # and with a non-identity metric
    rng = np.random.default_rng(0)
    A = rng.standard_normal((w.dk, w.dk))
    E0 = A @ A.T / w.dk + 0.5 * np.eye(w.dk)
    Om_p, C_p = calibrate.fit_head(torch.from_numpy(Q), 5, torch.from_numpy(E0))
    Om_o, _ = orc.fit_sketching_matrix(Q, E0, 5)
    np.testing.assert_allclose(Om_p.numpy(), Om_o, atol=1e-7)
    np.testing.assert_allclose(C_p.numpy(), orc.offline_coefficient_map(Om_o, E0), atol=1e-7)


def test_algorithmic_byte_accounting():
    # Mamba-2 layer, bf16 I/O: slot = 128*2 + 64*2 + 8 = 392 B, token = 256 + 392 = 648 B
    assert traffic.slot_bytes("mamba2", 128, 64, "bf16") == 392
    assert traffic.slot_bytes("gdn", 128, 128, "bf16") == 520
    assert traffic.slot_bytes("kda", 128, 128, "bf16") == 772
    assert traffic.token_bytes("mamba2", 128, 64, "bf16") == 648
    per_head = 16 * 64 * 4 + 7 * 392 + 648 + 392 + 64 * 4
    assert traffic.decode_bytes("mamba2", 256, 64, 128, 64, 16, 7) == 256 * 64 * per_head + 64 * 16 * 128 * 4
    full = 128 * 64 * 4 + 7 * 392 + 648 + 392 + 64 * 4
    assert traffic.decode_bytes("mamba2", 256, 64, 128, 64, 16, 7, full_read=True) == 256 * 64 * full
    upd = 2 * 128 * 64 * 4 + 15 * 392 + 392 + 256 + 256 + 16 * 64 * 4
    assert traffic.update_bytes("mamba2", 256, 64, 128, 64, 16, 15) == 256 * 64 * upd + 64 * 128 * 16 * 4
    # the sketch read is K/r times smaller than the state read
    assert (128 * 64 * 4) // (16 * 64 * 4) == 8


_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
# every rank times its own shard; the job time is the max over ranks, the job value the sum of tokens over that time
ms_local = 10.0 + 5.0 * rank
ms = bench.max_over_ranks(ms_local, dist, device="cpu")
value = bench.job_value(tokens_per_rank=1000, world=2, ms_step=ms)
shard = bench.rank_shard(total_batch=9, rank=rank, world=2)
if rank == 0:
    print(json.dumps(dict(ms=ms, value=value, shard=list(shard))))
else:
    print(json.dumps(dict(shard=list(shard))))
dist.destroy_process_group()
"""


def test_rank_sharding_and_max_over_ranks_timing_with_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT, port=29641))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)
             for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    import json
    r0 = json.loads(outs[0][0].strip().splitlines()[-1])
    r1 = json.loads(outs[1][0].strip().splitlines()[-1])
    assert r0["ms"] == 15.0                       # max over ranks
    assert abs(r0["value"] - 2 * 1000 / 15e-3) < 1e-6
    assert r0["shard"] == [0, 4] and r1["shard"] == [4, 9]     # disjoint cover of the batch, no exchange needed


def test_logical_layers_map_onto_the_physical_slots_that_fit():
    """The 48-layer stack of the large-batch sweep does not fit at batch 2048: the benchmark maps the logical layers
    round-robin onto as many physical slots as its memory budget holds."""
    import bench
    w = synth.sweep_point(2048, 16, 16)
    per = bench.layer_bytes(w)
    assert per > 2048 * 64 * 128 * 64 * 4                       # at least the state: 4 GiB per layer
    assert 48 * per > 180e9                                     # 48 distinct layers exceed the GPU's memory
    n = bench.physical_layers(per, int(100e9), 48)
    assert 1 <= n < 48 and n * per <= 100e9 < (n + 1) * per
    assert bench.physical_layers(bench.layer_bytes(synth.sweep_point(64, 4, 8)), int(40e9), 48) == 48
    assert bench.physical_layers(10**12, 10**9, 48) == 1        # never fewer than one slot
    assert [l % n for l in range(48)].count(0) == -(-48 // n)   # slot 0 serves ceil(48 / n) logical layers
    assert bench.update_kernel_name(w) == "update_tc_ws_mamba2_kernel"
    assert bench.update_kernel_name(synth.CONFIGS["c4_kda"]) == "update_tc_ws_kda_kernel"
    assert bench.update_kernel_name(synth.CONFIGS["c1_gdn_tiny"]) == "update_kernel"
