"""The C-ABI library loads without a GPU, exports every declared symbol, and its host-side logic
(validation, sizes, layout) behaves as the header says.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2609_33051_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sketchssm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sketchssm_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(binding.EXPORTED)
    for n in names:
        assert hasattr(lib, n), n
    assert lib.sketchssm_version().decode().startswith("sketchssm-b200")


def make(lib, **kw):
    base = dict(kind=1, batch=4, heads=2, dk=128, dv=128, rank=16, buf_len=16, io_dtype=1, out_dtype=0, device=0)
    base.update(kw)
    cfg = binding.Config(**base)
    ctx = ctypes.c_void_p()
    rc = lib.sketchssm_create(ctypes.byref(cfg), ctypes.byref(ctx))
    return rc, ctx


def test_create_validates_configuration(lib):
    rc, ctx = make(lib)
    assert rc == 0 and ctx.value
    assert lib.sketchssm_destroy(ctx) == 0
    assert make(lib, kind=3)[0] == -1
    assert make(lib, batch=0)[0] == -1
    assert make(lib, io_dtype=2)[0] == -1
    assert make(lib, dk=96)[0] == -2
    assert make(lib, dv=96)[0] == -2
    assert make(lib, dv=80)[0] == 0              # K = 128, V = 80: the second Mamba-2 head shape
    assert make(lib, dk=64, dv=80)[0] == -2
    assert make(lib, rank=65)[0] == -2
    assert make(lib, rank=0)[0] == -1
    assert make(lib, buf_len=6)[0] == -2
    assert make(lib, buf_len=68)[0] == -2
    assert lib.sketchssm_create(None, None) == -1
    assert lib.sketchssm_destroy(None) == -1
    # state-dependent coefficient map: needs a positive ridge, at most 8 pivots (0 = exact ridge solve)
    assert make(lib, coef_per_seq=1, coef_pivots=4, ridge_lambda=0.1)[0] == 0
    assert make(lib, coef_per_seq=1, coef_pivots=0, ridge_lambda=0.1)[0] == 0
    assert make(lib, coef_per_seq=1, coef_pivots=4, ridge_lambda=0.0)[0] == -1
    assert make(lib, coef_per_seq=1, coef_pivots=-1, ridge_lambda=0.1)[0] == -1
    assert make(lib, coef_per_seq=1, coef_pivots=9, ridge_lambda=0.1)[0] == -2
    assert make(lib, coef_per_seq=2)[0] == -1
    rc, ctx = make(lib, coef_per_seq=1, coef_pivots=4, ridge_lambda=0.1, batch=3, heads=5, rank=8)
    s = binding.Sizes()
    assert rc == 0 and lib.sketchssm_query_sizes(ctx, ctypes.byref(s)) == 0
    assert s.coef_bytes == 3 * 5 * 8 * 128 * 4                  # one map per (batch, head)
    assert s.erase_bytes == 0
    lib.sketchssm_destroy(ctx)
    # projected erase vectors: delta-rule kinds only, rank a multiple of 4, windows of at most 32 tokens, and room for two
    # coefficient vectors in the scratch (2 * round_up(rank, 8) <= dk)
    assert make(lib, erase_factors=1)[0] == 0
    assert make(lib, erase_factors=2)[0] == -1
    assert make(lib, kind=0, dv=64, erase_factors=1)[0] == -1
    assert make(lib, rank=6, erase_factors=1)[0] == -2
    assert make(lib, buf_len=64, erase_factors=1)[0] == -2
    assert make(lib, dk=64, dv=64, rank=36, erase_factors=1)[0] == -2
    rc, ctx = make(lib, erase_factors=1, batch=3, heads=5, rank=8, buf_len=8)
    assert rc == 0 and lib.sketchssm_query_sizes(ctx, ctypes.byref(s)) == 0
    assert s.erase_bytes == 3 * 5 * 8 * 8 * 4
    b = binding.Buffers(*([1 << 20] * 7), None, None)             # (addresses are only checked, never dereferenced, by bind)
    assert lib.sketchssm_bind(ctx, ctypes.byref(b)) == -1         # the erase buffer is required
    b.erase = 1 << 20
    assert lib.sketchssm_bind(ctx, ctypes.byref(b)) == 0
    lib.sketchssm_destroy(ctx)


@pytest.mark.parametrize("kind,io,K,V,L,expect_head", [
    (0, 1, 128, 64, 16, 16 * 128 * 2 + 16 * 64 * 2 + 64 + 64),        # Mamba-2 bf16
    (1, 1, 128, 128, 16, 16 * 128 * 2 * 2 + 64 + 64),                  # GDN bf16
    (2, 1, 128, 128, 32, 32 * 128 * 2 * 3 + 128),                      # KDA bf16: k, v, g vectors + beta
    (1, 0, 64, 64, 8, 8 * 64 * 4 * 2 + 32 + 32),                       # GDN fp32
])
def test_sizes_and_ring_layout(lib, kind, io, K, V, L, expect_head):
    rc, ctx = make(lib, kind=kind, io_dtype=io, dk=K, dv=V, buf_len=L, batch=3, heads=5, rank=8)
    assert rc == 0
    s = binding.Sizes()
    assert lib.sketchssm_query_sizes(ctx, ctypes.byref(s)) == 0
    assert s.state_bytes == 15 * K * V * 4
    assert s.sketch_bytes == 15 * 8 * V * 4
    assert s.omega_bytes == 5 * K * 8 * 4 and s.coef_bytes == 5 * 8 * K * 4
    assert s.ring_head_bytes == expect_head and s.ring_bytes == 15 * expect_head
    esz = 2 if io else 4
    assert s.ring_v_offset == L * K * esz
    assert s.ring_beta_offset == s.ring_v_offset + L * V * esz
    assert s.ring_decay_offset == s.ring_beta_offset + L * 4
    assert s.alignment == 16 and s.status_bytes == ((4 + 4 + 5) * 4 + 15) // 16 * 16
    assert s.work_bytes == 15 * (K + L) * 4
    for off in (s.ring_head_bytes, s.ring_v_offset, s.ring_beta_offset, s.ring_decay_offset):
        assert off % 16 == 0
    lib.sketchssm_destroy(ctx)


def test_calls_are_rejected_before_bind_and_on_bad_arguments(lib):
    rc, ctx = make(lib)
    dummy = ctypes.c_void_p(0x1000)
    assert lib.sketchssm_decode_step(ctx, 0, dummy, dummy, dummy, dummy, dummy, dummy, 0, None) == -3
    assert lib.sketchssm_state_update(ctx, 0, None, None, None, None, None, None, 0, None) == -3
    assert lib.sketchssm_read_status(ctx, None, None) == -3
    bufs = binding.Buffers(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0, 0x7000)
    assert lib.sketchssm_bind(ctx, ctypes.byref(bufs)) == -1            # null status
    bufs = binding.Buffers(0x1000, 0x2000, 0x3008, 0x4000, 0x5000, 0x6000, 0x7000)
    assert lib.sketchssm_bind(ctx, ctypes.byref(bufs)) == -1            # misaligned ring
    bufs = binding.Buffers(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000)
    assert lib.sketchssm_bind(ctx, ctypes.byref(bufs)) == 0
    # argument checks happen on the host before any CUDA call
    assert lib.sketchssm_decode_step(ctx, 16, dummy, dummy, dummy, dummy, dummy, dummy, 0, None) == -1   # n_before > L-1
    assert lib.sketchssm_decode_step(ctx, -1, dummy, dummy, dummy, dummy, dummy, dummy, 0, None) == -1
    assert lib.sketchssm_decode_step(ctx, 0, None, dummy, dummy, dummy, dummy, dummy, 0, None) == -1
    assert lib.sketchssm_decode_step(ctx, 0, ctypes.c_void_p(0x1004), dummy, dummy, dummy, dummy, dummy, 0, None) == -1
    assert lib.sketchssm_decode_step(ctx, 0, dummy, dummy, dummy, dummy, dummy, dummy, 2, None) == -1   # unknown flag
    assert lib.sketchssm_full_read_decode(ctx, 99, dummy, dummy, dummy, dummy, dummy, dummy, 0, None) == -1
    assert lib.sketchssm_state_update(ctx, 16, dummy, dummy, dummy, dummy, dummy, dummy, 0, None) == -1  # L+1 tokens
    assert lib.sketchssm_state_update(ctx, 3, dummy, dummy, dummy, None, dummy, dummy, 0, None) == -1   # partial token
    assert lib.sketchssm_state_update(ctx, 3, dummy, None, None, None, None, None, 0, None) == -1       # q without out
    assert lib.sketchssm_state_update(ctx, 0, None, None, None, None, None, None, 1, None) == 0         # nothing to do
    assert lib.sketchssm_tune(ctx, b"decode_stages", 2) == 0
    assert lib.sketchssm_tune(ctx, b"no_such_key", 2) == -1
    assert lib.sketchssm_status_string(-5).decode() == "bounded device wait ran out"
    lib.sketchssm_destroy(ctx)


def test_product_path_has_no_cpu_fallback_and_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_33051_b200")
    for dirpath, _dirs, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|sketchssm_oracle|oracle[/.]", text, flags=re.M), f
    with pytest.raises(FileNotFoundError):
        binding.load_library("/nonexistent/libsketchssm.so")
