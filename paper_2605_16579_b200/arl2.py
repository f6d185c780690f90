"""ctypes binding of ``libarl2.so`` (the C ABI in ``include/arl2.h``), same names.

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.
PyTorch appears here as the owner of device memory and streams -- tensors are passed as
``data_ptr()`` and the current CUDA stream as a ``void*``.  There is no fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libarl2.so")

ARL2_BF16, ARL2_FP32 = 0, 1
ARL2_FLAG_FORCE_SIMT = 1
ARL2_FLAG_TOKEN_GATES = 2
ARL2_FLAG_GATE_SCALAR = 4
ARL2_FLAG_GATE_ELEMENTWISE = 8
ARL2_FLAG_DELTA_DECAYED_PREDICTION = 32


def ARL2_FLAG_DEBUG_WAIT_LIMIT(polls: int) -> int:
    return (polls + 1) << 16

EXPORTS = (
    "arl2_workspace_bytes", "arl2_create", "arl2_set_params", "arl2_denoise_step", "arl2_commit",
    "arl2_reset", "arl2_get_state", "arl2_set_state", "arl2_sync_status", "arl2_launch_count",
    "arl2_set_profile_events", "arl2_commit_static_scratch", "arl2_commit_delta", "arl2_commit_tokens", "arl2_teacher_step", "arl2_commit_decay_tokens",
    "arl2_step_kernel_name", "arl2_destroy", "arl2_last_error", "arl2_version", "arl2_debug_set_wait_limit", "arl2_clean_pass", "arl2_denoise_step_token_level",
    "arl2_projection_workspace_bytes", "arl2_set_projections", "arl2_project_in", "arl2_project_out",
)


class Arl2Error(RuntimeError):
    pass


class arl2_config(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("L", ctypes.c_int32), ("D", ctypes.c_int32),
        ("io_dtype", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("l2_eps", ctypes.c_float),
        ("commit_rule", ctypes.c_int32), ("flags", ctypes.c_uint32),
    ]


_lib = None


def load(build_if_missing: bool = False) -> ctypes.CDLL:
    """Load the library (once).  Raises Arl2Error when it is absent: there is no CPU path."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        from . import build as _build

        _build.build_library()
    if not os.path.exists(LIB_PATH):
        raise Arl2Error(
            f"{LIB_PATH} is missing: build it with `python -m paper_2605_16579_b200.build` "
            "(nvcc, sm_100a).  The layer has no CPU or PyTorch fallback."
        )
    lib = ctypes.CDLL(LIB_PATH)
    vp, cp = ctypes.c_void_p, ctypes.POINTER(arl2_config)
    lib.arl2_workspace_bytes.restype = ctypes.c_size_t
    lib.arl2_workspace_bytes.argtypes = [cp]
    lib.arl2_create.restype = ctypes.c_int
    lib.arl2_create.argtypes = [cp, vp, vp, ctypes.c_size_t, vp, ctypes.POINTER(vp)]
    lib.arl2_set_params.restype = ctypes.c_int
    lib.arl2_set_params.argtypes = [vp] * 7
    lib.arl2_denoise_step.restype = ctypes.c_int
    lib.arl2_denoise_step.argtypes = [vp] * 7
    lib.arl2_commit.restype = ctypes.c_int
    lib.arl2_commit.argtypes = [vp] * 5
    lib.arl2_clean_pass.restype = ctypes.c_int
    lib.arl2_clean_pass.argtypes = [vp] * 8
    lib.arl2_denoise_step_token_level.restype = ctypes.c_int
    lib.arl2_denoise_step_token_level.argtypes = [vp] * 8
    lib.arl2_projection_workspace_bytes.restype = ctypes.c_size_t
    lib.arl2_projection_workspace_bytes.argtypes = [cp]
    lib.arl2_set_projections.restype = ctypes.c_int
    lib.arl2_set_projections.argtypes = [vp] * 7 + [ctypes.c_size_t, vp]
    lib.arl2_project_in.restype = ctypes.c_int
    lib.arl2_project_in.argtypes = [vp] * 7
    lib.arl2_project_out.restype = ctypes.c_int
    lib.arl2_project_out.argtypes = [vp] * 4
    lib.arl2_teacher_step.restype = ctypes.c_int
    lib.arl2_teacher_step.argtypes = [vp, vp, vp, vp, ctypes.c_int32, vp, vp]
    lib.arl2_commit_delta.restype = ctypes.c_int
    lib.arl2_commit_delta.argtypes = [vp] * 6
    lib.arl2_commit_decay_tokens.restype = ctypes.c_int
    lib.arl2_commit_decay_tokens.argtypes = [vp] * 5
    lib.arl2_commit_tokens.restype = ctypes.c_int
    lib.arl2_commit_tokens.argtypes = [vp] * 6
    lib.arl2_reset.restype = ctypes.c_int
    lib.arl2_reset.argtypes = [vp, ctypes.c_int32, vp]
    lib.arl2_get_state.restype = ctypes.c_int
    lib.arl2_get_state.argtypes = [vp, vp, vp]
    lib.arl2_set_state.restype = ctypes.c_int
    lib.arl2_set_state.argtypes = [vp, vp, vp]
    lib.arl2_sync_status.restype = ctypes.c_int
    lib.arl2_sync_status.argtypes = [vp, vp]
    lib.arl2_debug_set_wait_limit.restype = ctypes.c_int
    lib.arl2_debug_set_wait_limit.argtypes = [vp, ctypes.c_int32]
    lib.arl2_set_profile_events.restype = ctypes.c_int
    lib.arl2_set_profile_events.argtypes = [vp, vp, vp]
    lib.arl2_commit_static_scratch.restype = ctypes.c_int
    lib.arl2_commit_static_scratch.argtypes = [cp] + [vp] * 9
    lib.arl2_launch_count.restype = ctypes.c_uint64
    lib.arl2_launch_count.argtypes = [vp]
    lib.arl2_step_kernel_name.restype = ctypes.c_char_p
    lib.arl2_step_kernel_name.argtypes = [vp]
    lib.arl2_destroy.restype = None
    lib.arl2_destroy.argtypes = [vp]
    lib.arl2_last_error.restype = ctypes.c_char_p
    lib.arl2_version.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _check(status: int, what: str):
    if status != 0:
        msg = load().arl2_last_error().decode()
        raise Arl2Error(f"{what} failed with status {status}: {msg}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(B, H, L, D, dtype, softmax_scale=0.0, l2_eps=0.0, commit_rule=0, flags=0):
    io = {"bf16": ARL2_BF16, "fp32": ARL2_FP32, torch.bfloat16: ARL2_BF16,
          torch.float32: ARL2_FP32}[dtype]
    return arl2_config(ctypes.sizeof(arl2_config), B, H, L, D, io, softmax_scale, l2_eps,
                       commit_rule, flags)


def arl2_workspace_bytes(cfg: arl2_config) -> int:
    n = load().arl2_workspace_bytes(ctypes.byref(cfg))
    if n == 0:
        raise Arl2Error("arl2_workspace_bytes: " + load().arl2_last_error().decode())
    return n


class Layer:
    """One context: owns (through torch) the state and workspace buffers it hands to the library.

    Methods mirror the C entry points one to one; tensors must be contiguous CUDA tensors of
    the configured dtype.
    """

    def __init__(self, B, H, L, D, dtype="bf16", device="cuda:0", softmax_scale=0.0, l2_eps=0.0,
                 flags=0, state=None, workspace=None):
        """``state`` ([B, H, D, D] fp32) and ``workspace`` (uint8, >= arl2_workspace_bytes, 256-byte
        aligned) may be handed in by a caller that manages its own device memory; by default torch
        allocates them here."""
        lib = load()
        self.cfg = make_config(B, H, L, D, dtype, softmax_scale, l2_eps, 0, flags)
        self.B, self.H, self.L, self.D = B, H, L, D
        self.flags = flags
        self.device = torch.device(device)
        self.dtype = torch.bfloat16 if self.cfg.io_dtype == ARL2_BF16 else torch.float32
        self.workspace_bytes = arl2_workspace_bytes(self.cfg)
        with torch.cuda.device(self.device):
            if state is None:
                state = torch.empty(B, H, D, D, dtype=torch.float32, device=self.device)
            if workspace is None:
                workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
            self._want(state, (B, H, D, D), torch.float32, "state")
            if not (workspace.is_cuda and workspace.dtype == torch.uint8 and workspace.is_contiguous()
                    and workspace.numel() >= self.workspace_bytes):
                raise Arl2Error(f"workspace: expected >= {self.workspace_bytes} contiguous CUDA bytes")
            self.state, self.workspace = state, workspace
            ctx = ctypes.c_void_p()
            _check(lib.arl2_create(ctypes.byref(self.cfg), _ptr(self.state), _ptr(self.workspace),
                                   self.workspace.numel(), _stream(), ctypes.byref(ctx)),
                   "arl2_create")
        self._ctx = ctx
        self._params = None  # keeps the parameter tensors alive
        self.reset()

    # -- the C entry points ------------------------------------------------------------
    def set_params(self, wq=None, wk=None, wv=None, rope_cos=None, rope_sin=None):
        for w in (wq, wk, wv):
            if w is not None:
                self._want(w, (self.H, self.D, self.D), self.dtype, "feature map")
        for t in (rope_cos, rope_sin):
            if t is not None:
                self._want(t, (self.L, self.D // 2), torch.float32, "rope table")
        self._params = (wq, wk, wv, rope_cos, rope_sin)
        with torch.cuda.device(self.device):
            _check(load().arl2_set_params(self._ctx, _ptr(wq), _ptr(wk), _ptr(wv), _ptr(rope_cos),
                                          _ptr(rope_sin), _stream()), "arl2_set_params")

    def denoise_step(self, q, k, v, gate_logits, out=None):
        shape = (self.B, self.L, self.H, self.D)
        for t in (q, k, v):
            self._want(t, shape, self.dtype, "q/k/v")
        gshape = ((self.B, self.L) if self.flags & ARL2_FLAG_GATE_SCALAR else
                  (self.B, self.L, self.H, self.D) if self.flags & ARL2_FLAG_GATE_ELEMENTWISE else
                  (self.B, self.L, self.H))
        self._want(gate_logits, gshape, torch.float32, "gate_logits")
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=self.device)
        else:
            self._want(out, shape, self.dtype, "out")
        with torch.cuda.device(self.device):
            _check(load().arl2_denoise_step(self._ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(gate_logits),
                                            _ptr(out), _stream()), "arl2_denoise_step")
        return out

    def clean_pass(self, q, k_clean, v_clean, gate_logits, decay_logits, out=None):
        """The clean pass in one call: the output against the pre-update state, then the commit."""
        shape = (self.B, self.L, self.H, self.D)
        for t in (q, k_clean, v_clean):
            self._want(t, shape, self.dtype, "q/k_clean/v_clean")
        gshape = ((self.B, self.L) if self.flags & ARL2_FLAG_GATE_SCALAR else
                  (self.B, self.L, self.H, self.D) if self.flags & ARL2_FLAG_GATE_ELEMENTWISE else
                  (self.B, self.L, self.H))
        self._want(gate_logits, gshape, torch.float32, "gate_logits")
        self._want(decay_logits, (self.B, self.H), torch.float32, "decay_logits")
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=self.device)
        else:
            self._want(out, shape, self.dtype, "out")
        with torch.cuda.device(self.device):
            _check(load().arl2_clean_pass(self._ctx, _ptr(q), _ptr(k_clean), _ptr(v_clean), _ptr(gate_logits),
                                          _ptr(decay_logits), _ptr(out), _stream()), "arl2_clean_pass")
        return out

    def denoise_step_token_level(self, q, k, v, gate_logits, alpha_logits=None, out=None):
        """Comparison mode: token i reads the state advanced by the block's tokens before it."""
        shape = (self.B, self.L, self.H, self.D)
        for t in (q, k, v):
            self._want(t, shape, self.dtype, "q/k/v")
        self._want(gate_logits, (self.B, self.L, self.H), torch.float32, "gate_logits")
        if alpha_logits is not None:
            self._want(alpha_logits, (self.B, self.L, self.H), torch.float32, "alpha_logits")
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=self.device)
        else:
            self._want(out, shape, self.dtype, "out")
        with torch.cuda.device(self.device):
            _check(load().arl2_denoise_step_token_level(self._ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(gate_logits),
                                                        _ptr(alpha_logits), _ptr(out), _stream()),
                   "arl2_denoise_step_token_level")
        return out

    def set_projections(self, w_q, w_k, w_v, w_g, w_o):
        """W_q, W_k, W_v, W_o [d, d] and W_g [d, H], bf16, (in, out): the module around the core."""
        d = self.H * self.D
        for w in (w_q, w_k, w_v, w_o):
            self._want(w, (d, d), torch.bfloat16, "projection weight")
        self._want(w_g, (d, self.H), torch.bfloat16, "gate weight")
        n = load().arl2_projection_workspace_bytes(ctypes.byref(self.cfg))
        with torch.cuda.device(self.device):
            self._pack = torch.empty(n, dtype=torch.uint8, device=self.device)
            self._proj = (w_q, w_k, w_v, w_g, w_o)
            _check(load().arl2_set_projections(self._ctx, _ptr(w_q), _ptr(w_k), _ptr(w_v), _ptr(w_g), _ptr(w_o),
                                               _ptr(self._pack), n, _stream()), "arl2_set_projections")

    def project_in(self, x, q=None, k=None, v=None, gate_logits=None):
        """x [B, L, d] bf16 -> q, k, v [B, L, H, D] bf16 and gate logits [B, L, H] fp32."""
        d = self.H * self.D
        self._want(x, (self.B, self.L, d), torch.bfloat16, "x")
        shape = (self.B, self.L, self.H, self.D)
        q, k, v = (torch.empty(shape, dtype=torch.bfloat16, device=self.device) if t is None else t for t in (q, k, v))
        if gate_logits is None:
            gate_logits = torch.empty(self.B, self.L, self.H, dtype=torch.float32, device=self.device)
        for t in (q, k, v):
            self._want(t, shape, torch.bfloat16, "q/k/v")
        self._want(gate_logits, (self.B, self.L, self.H), torch.float32, "gate_logits")
        with torch.cuda.device(self.device):
            _check(load().arl2_project_in(self._ctx, _ptr(x), _ptr(q), _ptr(k), _ptr(v), _ptr(gate_logits), _stream()),
                   "arl2_project_in")
        return q, k, v, gate_logits

    def project_out(self, o, y=None):
        """o [B, L, H, D] bf16 -> y [B, L, d] bf16 = o W_o."""
        d = self.H * self.D
        self._want(o, (self.B, self.L, self.H, self.D), torch.bfloat16, "o")
        if y is None:
            y = torch.empty(self.B, self.L, d, dtype=torch.bfloat16, device=self.device)
        self._want(y, (self.B, self.L, d), torch.bfloat16, "y")
        with torch.cuda.device(self.device):
            _check(load().arl2_project_out(self._ctx, _ptr(o), _ptr(y), _stream()), "arl2_project_out")
        return y

    def teacher_step(self, q, k_cache, v_cache, out=None):
        """Eq. 1: softmax attention of q [B, L, H, D] over a cache [B, Lk, H, D] (no rotation, no state)."""
        shape = (self.B, self.L, self.H, self.D)
        self._want(q, shape, self.dtype, "q")
        lk = int(k_cache.shape[1])
        self._want(k_cache, (self.B, lk, self.H, self.D), self.dtype, "k_cache")
        self._want(v_cache, (self.B, lk, self.H, self.D), self.dtype, "v_cache")
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=self.device)
        else:
            self._want(out, shape, self.dtype, "out")
        with torch.cuda.device(self.device):
            _check(load().arl2_teacher_step(self._ctx, _ptr(q), _ptr(k_cache), _ptr(v_cache), lk,
                                            _ptr(out), _stream()), "arl2_teacher_step")
        return out

    def commit(self, k_clean, v_clean, decay_logits):
        shape = (self.B, self.L, self.H, self.D)
        self._want(k_clean, shape, self.dtype, "k_clean")
        self._want(v_clean, shape, self.dtype, "v_clean")
        self._want(decay_logits, (self.B, self.H), torch.float32, "decay_logits")
        with torch.cuda.device(self.device):
            _check(load().arl2_commit(self._ctx, _ptr(k_clean), _ptr(v_clean), _ptr(decay_logits),
                                      _stream()), "arl2_commit")

    def commit_delta(self, k_clean, v_clean, decay_logits, beta_logits=None):
        """Eq. 4 as printed, at block level: S <- sigmoid(a) S + K'^T diag(beta) (V' - K' S_old)."""
        shape = (self.B, self.L, self.H, self.D)
        self._want(k_clean, shape, self.dtype, "k_clean")
        self._want(v_clean, shape, self.dtype, "v_clean")
        self._want(decay_logits, (self.B, self.H), torch.float32, "decay_logits")
        if beta_logits is not None:
            self._want(beta_logits, (self.B, self.L, self.H), torch.float32, "beta_logits")
        with torch.cuda.device(self.device):
            _check(load().arl2_commit_delta(self._ctx, _ptr(k_clean), _ptr(v_clean), _ptr(decay_logits),
                                            _ptr(beta_logits), _stream()), "arl2_commit_delta")

    def commit_decay_tokens(self, k_clean, v_clean, alpha_logits):
        """Gated-linear commit with one forget gate per token: S <- alpha_l S + K'_l^T V'_l in order."""
        shape = (self.B, self.L, self.H, self.D)
        self._want(k_clean, shape, self.dtype, "k_clean")
        self._want(v_clean, shape, self.dtype, "v_clean")
        self._want(alpha_logits, (self.B, self.L, self.H), torch.float32, "alpha_logits")
        with torch.cuda.device(self.device):
            _check(load().arl2_commit_decay_tokens(self._ctx, _ptr(k_clean), _ptr(v_clean),
                                                   _ptr(alpha_logits), _stream()), "arl2_commit_decay_tokens")

    def commit_tokens(self, k_clean, v_clean, alpha_logits=None, beta_logits=None):
        """Eq. 4 token by token with per-token gates [B, L, H] (None = gate 1); the layer must have
        been created with flags=ARL2_FLAG_TOKEN_GATES."""
        shape = (self.B, self.L, self.H, self.D)
        self._want(k_clean, shape, self.dtype, "k_clean")
        self._want(v_clean, shape, self.dtype, "v_clean")
        for name, g in (("alpha_logits", alpha_logits), ("beta_logits", beta_logits)):
            if g is not None:
                self._want(g, (self.B, self.L, self.H), torch.float32, name)
        with torch.cuda.device(self.device):
            _check(load().arl2_commit_tokens(self._ctx, _ptr(k_clean), _ptr(v_clean), _ptr(alpha_logits),
                                             _ptr(beta_logits), _stream()), "arl2_commit_tokens")

    def reset(self, stream_index: int = -1):
        with torch.cuda.device(self.device):
            _check(load().arl2_reset(self._ctx, stream_index, _stream()), "arl2_reset")

    def get_state(self) -> torch.Tensor:
        """Copy of S as a CPU fp32 tensor [B, H, D, D] (synchronises the stream)."""
        dst = torch.empty(self.B, self.H, self.D, self.D, dtype=torch.float32)
        with torch.cuda.device(self.device):
            _check(load().arl2_get_state(self._ctx, _ptr(dst), _stream()), "arl2_get_state")
            torch.cuda.current_stream().synchronize()
        return dst

    def set_state(self, src: torch.Tensor):
        src = src.to(torch.float32).contiguous()
        assert tuple(src.shape) == (self.B, self.H, self.D, self.D)
        with torch.cuda.device(self.device):
            _check(load().arl2_set_state(self._ctx, _ptr(src), _stream()), "arl2_set_state")
            torch.cuda.current_stream().synchronize()

    def sync_status(self):
        with torch.cuda.device(self.device):
            _check(load().arl2_sync_status(self._ctx, _stream()), "arl2_sync_status")

    def debug_set_wait_limit(self, polls: int):
        """Test hook: bounded waits in the tensor-core kernels give up after ``polls`` polls (< 0: default)."""
        _check(load().arl2_debug_set_wait_limit(self._ctx, polls), "arl2_debug_set_wait_limit")

    def set_profile_events(self, before: "torch.cuda.Event", after: "torch.cuda.Event"):
        """The next denoise_step records these events around its dominant kernel."""
        for ev in (before, after):
            if not ev.cuda_event:   # torch creates the CUDA event lazily, at its first record
                ev.record()
        _check(load().arl2_set_profile_events(self._ctx, ctypes.c_void_p(before.cuda_event),
                                              ctypes.c_void_p(after.cuda_event)),
               "arl2_set_profile_events")

    @property
    def launch_count(self) -> int:
        return int(load().arl2_launch_count(self._ctx))

    @property
    def step_kernel(self) -> str:
        return load().arl2_step_kernel_name(self._ctx).decode()

    def close(self):
        if self._ctx is not None:
            load().arl2_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers -----------------------------------------------------------------------
    def _want(self, t, shape, dtype, what):
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()
                and tuple(t.shape) == tuple(shape) and t.dtype == dtype):
            raise Arl2Error(f"{what}: expected a contiguous CUDA tensor {tuple(shape)} {dtype}, got "
                            f"{tuple(t.shape)} {t.dtype} on {t.device}")


STATIC_SCRATCH_BYTES = 8 << 20


def commit_static_scratch(cfg: arl2_config, state, k_clean, v_clean, decay_logits, wk=None, wv=None,
                          rope_cos=None, rope_sin=None):
    """arl2_commit_static_scratch: the commit for callers that may not allocate device memory.

    Updates ``state`` ([B, H, D, D] fp32, CUDA) in place; no context, no workspace.  The partial
    sums of the reduction live in an array built into the library (8 MiB per GPU), so shapes
    with B*H*ceil(L/512)*D*D*4 bytes above that are refused, and calls that overlap on the GPU
    must be ordered by the caller.
    """
    with torch.cuda.device(state.device):
        _check(load().arl2_commit_static_scratch(ctypes.byref(cfg), _ptr(state), _ptr(k_clean),
                                                 _ptr(v_clean), _ptr(decay_logits), _ptr(wk), _ptr(wv),
                                                 _ptr(rope_cos), _ptr(rope_sin), _stream()),
               "arl2_commit_static_scratch")
