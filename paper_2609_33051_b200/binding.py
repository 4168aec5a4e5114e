"""ctypes binding of libsketchssm.so: argument marshalling only.

Every step of the decode path runs in the CUDA library; this module converts
torch tensors to raw device pointers, forwards the calls with the same names as
the C ABI and raises on a non-zero status.  There is no fallback: if the shared
library is missing or CUDA is unavailable the calls fail.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

KIND = {"mamba2": 0, "gdn": 1, "kda": 2}
DTYPE = {"f32": 0, "bf16": 1}
TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}
NO_SKETCH = 0x1
NO_APPEND = 0x1

EXPORTED = (
    "sketchssm_create", "sketchssm_destroy", "sketchssm_query_sizes", "sketchssm_bind",
    "sketchssm_state_update", "sketchssm_decode_step", "sketchssm_full_read_decode",
    "sketchssm_read_status", "sketchssm_last_launch_count", "sketchssm_tune",
    "sketchssm_status_string", "sketchssm_version", "sketchssm_last_cuda_error", "sketchssm_step_host",
    "sketchssm_decode_step_static", "sketchssm_selftest_wait_timeout", "sketchssm_step_mixed",
)
OP_DECODE, OP_FULL_READ, OP_UPDATE = 0, 1, 2


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("kind", "batch", "heads", "dk", "dv", "rank", "buf_len", "io_dtype", "out_dtype", "device",
                 "coef_per_seq", "coef_pivots")] + [("ridge_lambda", ctypes.c_float), ("sketch_dtype", ctypes.c_int32),
                                                            ("erase_factors", ctypes.c_int32)]


class Sizes(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in
                ("state_bytes", "sketch_bytes", "ring_bytes", "omega_bytes", "coef_bytes", "status_bytes",
                 "work_bytes", "ring_head_bytes", "ring_v_offset", "ring_beta_offset", "ring_decay_offset", "alignment",
                 "erase_bytes")]


class Buffers(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("state", "sketch", "ring", "omega", "coef", "status", "work", "head_rank",
                                                "erase")]


class Staging(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("q", "k", "v", "beta", "decay", "out")]


class SketchSSMError(RuntimeError):
    def __init__(self, fn: str, status: int, text: str):
        super().__init__(f"{fn} failed: {text} ({status})")
        self.status = status


_LIB = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load libsketchssm.so (built in-tree by build.py) and declare the prototypes."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2609_33051_b200.build` (needs nvcc)")
    lib = ctypes.CDLL(path)
    vp, i32, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32
    lib.sketchssm_create.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(vp)]
    lib.sketchssm_destroy.argtypes = [vp]
    lib.sketchssm_query_sizes.argtypes = [vp, ctypes.POINTER(Sizes)]
    lib.sketchssm_bind.argtypes = [vp, ctypes.POINTER(Buffers)]
    for name in ("sketchssm_state_update", "sketchssm_decode_step", "sketchssm_full_read_decode",
                 "sketchssm_decode_step_static"):
        getattr(lib, name).argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, u32, vp]
    lib.sketchssm_step_mixed.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, u32, vp]
    lib.sketchssm_step_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, ctypes.POINTER(Staging), u32, vp]
    lib.sketchssm_selftest_wait_timeout.argtypes = [vp, i32, i32, vp]
    lib.sketchssm_read_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32 * 4), vp]
    lib.sketchssm_last_launch_count.argtypes = [vp]
    lib.sketchssm_tune.argtypes = [vp, ctypes.c_char_p, i32]
    lib.sketchssm_status_string.argtypes = [i32]
    lib.sketchssm_status_string.restype = ctypes.c_char_p
    lib.sketchssm_version.restype = ctypes.c_char_p
    lib.sketchssm_last_cuda_error.argtypes = [vp]
    lib.sketchssm_last_cuda_error.restype = ctypes.c_char_p
    for name in EXPORTED:
        if name not in ("sketchssm_status_string", "sketchssm_version", "sketchssm_last_cuda_error"):
            getattr(lib, name).restype = ctypes.c_int
    if path == _build.LIB_PATH:
        _LIB = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


class SketchSSM:
    """One layer's decode state on one GPU: owns the torch buffers, forwards to the C ABI.

    Tensors (all on `device`): state [B,H,K,V] f32, sketch [B,H,r,V] f32, ring (bytes),
    omega [H,K,r] f32, coef [H,r,K] f32 (or [B,H,r,K] with coef_per_seq: the state-dependent map that every
    state update rebuilds).  Token arguments follow the C header:
    q,k [B,H,K] io; v [B,H,V] io; beta [B,H] f32; decay [B,H] f32 or [B,H,K] io (KDA).
    With erase_factors (GDN / KDA) the decode step forms c_t from projected erase vectors kept in `erase` [B,H,L,r] f32.
    """

    def __init__(self, kind: str, batch: int, heads: int, dk: int, dv: int, rank: int, buf_len: int,
                 io: str = "bf16", out: str = "f32", device: int = 0, allocate: bool = True,
                 coef_per_seq: bool = False, coef_pivots: int = 4, ridge_lambda: float = 0.1, sketch: str = "f32",
                 erase_factors: bool = False):
        self.lib = load_library()
        self.kind, self.io, self.out = kind, io, out
        self.B, self.H, self.K, self.V, self.R, self.L = batch, heads, dk, dv, rank, buf_len
        self.device = torch.device("cuda", device)
        self.coef_per_seq = bool(coef_per_seq)
        self.cfg = Config(KIND[kind], batch, heads, dk, dv, rank, buf_len, DTYPE[io], DTYPE[out], device,
                          int(self.coef_per_seq), coef_pivots, ridge_lambda, DTYPE[sketch], int(bool(erase_factors)))
        self.erase_factors = bool(erase_factors)
        self.sketch_dtype = sketch
        self._ctx = ctypes.c_void_p()
        self._check("sketchssm_create", self.lib.sketchssm_create(ctypes.byref(self.cfg), ctypes.byref(self._ctx)))
        self.sizes = Sizes()
        self._check("sketchssm_query_sizes", self.lib.sketchssm_query_sizes(self._ctx, ctypes.byref(self.sizes)))
        self.state = self.sketch = self.ring = self.omega = self.coef = self.status = self.work = self.erase = None
        self.head_rank = None        # optional int32 [H] device tensor: per-head sketch rank (0 = full-state read); set, then bind()
        if allocate:
            self.allocate()

    # -- memory -----------------------------------------------------------------------------
    def allocate(self):
        d = self.device
        self.state = torch.zeros(self.B, self.H, self.K, self.V, dtype=torch.float32, device=d)
        self.sketch = torch.zeros(self.B, self.H, self.R, self.V, dtype=TORCH_DTYPE[self.sketch_dtype], device=d)
        self.ring = torch.zeros(self.sizes.ring_bytes, dtype=torch.uint8, device=d)
        self.omega = torch.zeros(self.H, self.K, self.R, dtype=torch.float32, device=d)
        self.coef = torch.zeros(*((self.B,) if self.coef_per_seq else ()), self.H, self.R, self.K,
                                dtype=TORCH_DTYPE[self.sketch_dtype], device=d)
        self.status = torch.zeros(self.sizes.status_bytes // 4, dtype=torch.int32, device=d)
        self.work = torch.zeros(self.sizes.work_bytes // 4, dtype=torch.float32, device=d)
        if self.erase_factors:
            self.erase = torch.zeros(self.B, self.H, self.L, self.R, dtype=TORCH_DTYPE[self.sketch_dtype], device=d)
        self.bind()

    def bind(self):
        assert self.state.numel() * 4 == self.sizes.state_bytes
        assert self.sketch.numel() * self.sketch.element_size() == self.sizes.sketch_bytes
        assert self.ring.numel() == self.sizes.ring_bytes
        b = Buffers(self.state.data_ptr(), self.sketch.data_ptr(), self.ring.data_ptr(),
                    self.omega.data_ptr(), self.coef.data_ptr(), self.status.data_ptr(), self.work.data_ptr(),
                    self.head_rank.data_ptr() if self.head_rank is not None else None,
                    self.erase.data_ptr() if self.erase is not None else None)
        self._check("sketchssm_bind", self.lib.sketchssm_bind(self._ctx, ctypes.byref(b)))

    def close(self):
        if self._ctx:
            self.lib.sketchssm_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers ------------------------------------------------------------------------------
    def _check(self, fn: str, rc: int):
        if rc != 0:
            text = self.lib.sketchssm_status_string(rc).decode()
            if rc == -4 and self._ctx:
                text += ": " + self.lib.sketchssm_last_cuda_error(self._ctx).decode()
            raise SketchSSMError(fn, rc, text)

    @staticmethod
    def _stream(stream) -> ctypes.c_void_p:
        s = torch.cuda.current_stream() if stream is None else stream
        return ctypes.c_void_p(s.cuda_stream)

    def new_output(self) -> torch.Tensor:
        return torch.empty(self.B, self.H, self.V, dtype=TORCH_DTYPE[self.out], device=self.device)

    def ring_views(self):
        """Typed views of the ring: k [B,H,L,K], v [B,H,L,V], beta [B,H,L], decay [B,H,L] or [B,H,L,K]."""
        hb = self.sizes.ring_head_bytes
        raw = self.ring.view(self.B, self.H, hb)
        iod = TORCH_DTYPE[self.io]
        k = raw[..., : self.sizes.ring_v_offset].view(iod).view(self.B, self.H, self.L, self.K)
        v = raw[..., self.sizes.ring_v_offset: self.sizes.ring_beta_offset].view(iod).view(self.B, self.H, self.L, self.V)
        beta = raw[..., self.sizes.ring_beta_offset: self.sizes.ring_decay_offset].view(torch.float32)
        dec = raw[..., self.sizes.ring_decay_offset:]
        dec = dec.view(iod).view(self.B, self.H, self.L, self.K) if self.kind == "kda" else dec.view(torch.float32)
        return k, v, beta, dec

    # -- the C ABI calls --------------------------------------------------------------------
    def state_update(self, n_before: int, q=None, k=None, v=None, beta=None, decay=None, out=None,
                     flags: int = 0, stream=None):
        rc = self.lib.sketchssm_state_update(self._ctx, n_before, _ptr(q), _ptr(k), _ptr(v), _ptr(beta),
                                             _ptr(decay), _ptr(out), flags, self._stream(stream))
        self._check("sketchssm_state_update", rc)
        return out

    def decode_step(self, n_before: int, q, k, v, beta, decay, out, flags: int = 0, stream=None):
        rc = self.lib.sketchssm_decode_step(self._ctx, n_before, _ptr(q), _ptr(k), _ptr(v), _ptr(beta),
                                            _ptr(decay), _ptr(out), flags, self._stream(stream))
        self._check("sketchssm_decode_step", rc)
        return out

    def decode_step_static(self, n_before: int, q, k, v, beta, decay, out, flags: int = 0, stream=None):
        """sketchssm_decode_step_static: the decode step for callers that can neither allocate nor supply
        scratch; its kernel-to-kernel hand-off uses the library's fixed 4 MiB device array."""
        rc = self.lib.sketchssm_decode_step_static(self._ctx, n_before, _ptr(q), _ptr(k), _ptr(v), _ptr(beta),
                                                   _ptr(decay), _ptr(out), flags, self._stream(stream))
        self._check("sketchssm_decode_step_static", rc)
        return out

    def step_mixed(self, phase: torch.Tensor, q, k, v, beta, decay, out, stream=None):
        """sketchssm_step_mixed: one step for sequences at different window phases; phase is an int32 [B] device tensor
        (n >= 0: decode step at ring fill n; -(n + 1): flush with n buffered tokens plus the current one)."""
        assert phase.dtype == torch.int32 and phase.is_cuda and phase.numel() == self.B
        rc = self.lib.sketchssm_step_mixed(self._ctx, _ptr(phase), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(decay),
                                           _ptr(out), 0, self._stream(stream))
        self._check("sketchssm_step_mixed", rc)
        return out

    def full_read_decode(self, n_before: int, q, k, v, beta, decay, out, flags: int = 0, stream=None):
        rc = self.lib.sketchssm_full_read_decode(self._ctx, n_before, _ptr(q), _ptr(k), _ptr(v), _ptr(beta),
                                                 _ptr(decay), _ptr(out), flags, self._stream(stream))
        self._check("sketchssm_full_read_decode", rc)
        return out

    def new_token_buffers(self, pinned_host: bool = False):
        """Empty q, k, v, beta, decay, out tensors of the C ABI's shapes: on the device, or page-locked host."""
        iod = TORCH_DTYPE[self.io]
        kw = dict(device="cpu", pin_memory=True) if pinned_host else dict(device=self.device)
        dec = (torch.empty(self.B, self.H, self.K, dtype=iod, **kw) if self.kind == "kda"
               else torch.empty(self.B, self.H, dtype=torch.float32, **kw))
        return dict(q=torch.empty(self.B, self.H, self.K, dtype=iod, **kw),
                    k=torch.empty(self.B, self.H, self.K, dtype=iod, **kw),
                    v=torch.empty(self.B, self.H, self.V, dtype=iod, **kw),
                    beta=torch.empty(self.B, self.H, dtype=torch.float32, **kw), decay=dec,
                    out=torch.empty(self.B, self.H, self.V, dtype=TORCH_DTYPE[self.out], **kw))

    def step_host(self, op: int, n_before: int, host: dict, staging: dict, flags: int = 0, stream=None):
        """sketchssm_step_host: host token tensors in, host output out, copies and kernel on one stream."""
        st = Staging(*[staging[n].data_ptr() for n in ("q", "k", "v", "beta", "decay", "out")])
        rc = self.lib.sketchssm_step_host(self._ctx, op, n_before, _ptr(host["q"]), _ptr(host["k"]), _ptr(host["v"]),
                                          _ptr(host["beta"]), _ptr(host["decay"]), _ptr(host["out"]),
                                          ctypes.byref(st), flags, self._stream(stream))
        self._check("sketchssm_step_host", rc)
        return host["out"]

    def selftest_wait_timeout(self, poll_limit: int = 2048, where: int = 99, stream=None):
        """sketchssm_selftest_wait_timeout: one warp whose bounded wait runs out and reports through the status block."""
        self._check("sketchssm_selftest_wait_timeout",
                    self.lib.sketchssm_selftest_wait_timeout(self._ctx, poll_limit, where, self._stream(stream)))

    def read_status(self, stream=None):
        detail = (ctypes.c_int32 * 4)()
        rc = self.lib.sketchssm_read_status(self._ctx, ctypes.byref(detail), self._stream(stream))
        return rc, list(detail)

    def check_status(self, stream=None):
        rc, detail = self.read_status(stream)
        if rc != 0:
            raise SketchSSMError("sketchssm_read_status", rc,
                                 self.lib.sketchssm_status_string(rc).decode() + f" detail={detail}")

    def last_launch_count(self) -> int:
        return self.lib.sketchssm_last_launch_count(self._ctx)

    def tune(self, key: str, value: int):
        self._check("sketchssm_tune", self.lib.sketchssm_tune(self._ctx, key.encode(), value))
