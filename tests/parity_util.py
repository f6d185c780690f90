"""Shared machinery of the GPU parity tests: runs the same seeded schedule through the CUDA
library (via its C ABI binding) and through the CPU float64 oracle and compares them.

Error measure (stated tolerance: 2e-2 for bf16 I/O, 1e-4 in fp32 mode): for each output
tensor and each (stream, head), max|gpu - ref| / max|ref| -- a per-head normalised maximum,
because an element-wise relative error is unbounded next to zeros of the reference.  Once the
state is non-zero the readout dominates the output's magnitude (sigmoid(g) Q'S is two orders of
magnitude above the softmax average of V on the seeded workloads), so the schedules also run
passes with the combine gate closed (logits of -40): those compare the intra-block softmax
branch alone, against its own normalisation.

Stand-ins for a memory checker: every output buffer handed to the library is filled with NaN
before the call (a row the kernel does not write stays NaN and fails the comparison), and the
output, state and workspace buffers sit between canary pads that are checked after every call.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2605_16579_b200 import workload

TOL = {"bf16": 2e-2, "fp32": 1e-4}
PAD = 1024          # canary bytes on each side of a guarded buffer
CANARY = 0xA5


def head_errors(got: np.ndarray, ref: np.ndarray, head_axis_first: bool = False):
    """Normalised max error per (b, h).  got/ref: [B, L, H, D] (outputs) or [B, H, D, D]."""
    got = np.asarray(got, dtype=np.float64)
    if head_axis_first:  # state [B, H, D, D]
        num = np.abs(got - ref).max(axis=(-1, -2))
        den = np.abs(ref).max(axis=(-1, -2))
    else:                # [B, L, H, D]
        num = np.abs(got - ref).max(axis=(1, 3))
        den = np.abs(ref).max(axis=(1, 3))
    return num / np.maximum(den, 1e-30)


def rows_error(got_rows: np.ndarray, ref_rows: np.ndarray, rows) -> float:
    """Sampled rows [n, D] of several (b, h): normalise by the max |ref| of each head's sample."""
    rows = np.asarray(rows)
    worst = 0.0
    for b, h in sorted({(int(r[0]), int(r[1])) for r in rows}):
        sel = (rows[:, 0] == b) & (rows[:, 1] == h)
        den = max(np.abs(ref_rows[sel]).max(), 1e-30)
        worst = max(worst, np.abs(got_rows[sel] - ref_rows[sel]).max() / den)
    return worst


class Guarded:
    """A device tensor between two canary pads (one flat byte buffer)."""

    def __init__(self, shape, dtype, device):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.n = n
        self.raw = torch.full((n + 2 * PAD,), CANARY, dtype=torch.uint8, device=device)
        self.t = self.raw[PAD:PAD + n].view(dtype).view(*shape)

    def intact(self) -> bool:
        return bool((self.raw[:PAD] == CANARY).all() and (self.raw[PAD + self.n:] == CANARY).all())


def unit_view(t: torch.Tensor, units):
    """[B, L, H, ...] -> [1, L, U, ...]: the listed (stream, head) units as the heads of one stream.
    Streams share L and the rotation tables, and heads never mix, so the oracle may be handed the
    units it has to follow as a narrower problem (sliced before the values are widened to float64)."""
    return torch.stack([t[b, :, h] for b, h in units], dim=1).unsqueeze(0)


class Pair:
    """The CUDA layer and the oracle side by side on one configuration.

    ``units``: the (stream, head) pairs the oracle follows (None = all of them).  The reference state
    of every other unit is NaN from the start and is never read: nothing is ever copied from the
    GPU into the reference.
    """

    def __init__(self, oracle, cfg, device="cuda:0", rope=True, maps=True, flags=0, eps=0.0,
                 scale=0.0, units=None):
        from paper_2605_16579_b200 import arl2

        self.oracle, self.cfg, self.dev = oracle, cfg, device
        self.g_state = Guarded((cfg.B, cfg.H, cfg.D, cfg.D), torch.float32, device)
        probe = arl2.make_config(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, scale, eps, 0, flags)
        self.g_ws = Guarded((arl2.arl2_workspace_bytes(probe),), torch.uint8, device)
        self.layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=device,
                                softmax_scale=scale, l2_eps=eps, flags=flags,
                                state=self.g_state.t, workspace=self.g_ws.t)
        self.g_out = Guarded((cfg.B, cfg.L, cfg.H, cfg.D), cfg.torch_dtype, device)
        self.eps = eps if eps > 0 else 1e-6
        self.scale = scale if scale > 0 else None
        self.wq = self.wk = self.wv = self.cos = self.sin = None
        if maps:
            self.wq, self.wk, self.wv = workload.feature_weights(cfg)
        if rope:
            self.cos, self.sin = workload.rope_tables(cfg.L, cfg.D)
        dv = lambda t: None if t is None else t.to(device)  # noqa: E731
        self.layer.set_params(dv(self.wq), dv(self.wk), dv(self.wv), dv(self.cos), dv(self.sin))
        self.tol = TOL[cfg.dtype]
        self.S_ref = np.zeros((cfg.B, cfg.H, cfg.D, cfg.D))
        self.tracked = np.ones((cfg.B, cfg.H), dtype=bool)
        if units is not None:
            self.restrict(units)

    # -- which units the oracle follows ------------------------------------------------
    def restrict(self, units):
        """From now on the oracle follows only ``units`` (a subset of what it follows so far)."""
        mask = np.zeros_like(self.tracked)
        for b, h in units:
            assert self.tracked[b, h], f"unit {(b, h)} is no longer followed by the oracle"
            mask[b, h] = True
        self.tracked = mask
        self.S_ref[~mask] = np.nan

    @property
    def units(self):
        return [(int(b), int(h)) for b, h in zip(*np.nonzero(self.tracked))]

    def _all(self):
        return bool(self.tracked.all())

    def check_guards(self):
        assert self.g_out.intact(), "the output buffer's canaries were overwritten"
        assert self.g_state.intact(), "the state buffer's canaries were overwritten"
        assert self.g_ws.intact(), "the workspace's canaries were overwritten"

    # -- denoise passes ------------------------------------------------------------------
    def step_gpu(self, q, k, v, g):
        d = self.dev
        self.g_out.t.fill_(float("nan"))
        out = self.layer.denoise_step(q.to(d), k.to(d), v.to(d), g.to(d), out=self.g_out.t)
        got = out.float().cpu().numpy()
        self.check_guards()
        return got

    def step_full(self, q, k, v, g):
        """Full comparison of one step; returns the worst per-head error."""
        assert self._all()
        got = self.step_gpu(q, k, v, g)
        ref = self.oracle.step(q, k, v, g, self.S_ref, self.wq, self.cos, self.sin,
                               scale=self.scale, eps=self.eps)
        assert np.isfinite(got).all()
        return float(head_errors(got, ref).max())

    def step_sampled(self, q, k, v, g, rows):
        """Sampled rows (b, h, i) of followed units; the whole output must still be finite."""
        got = self.step_gpu(q, k, v, g)
        assert np.isfinite(got).all()
        rows = np.asarray(rows)
        units = sorted({(int(r[0]), int(r[1])) for r in rows})
        assert all(self.tracked[b, h] for b, h in units)
        index = {u: n for n, u in enumerate(units)}
        urows = np.array([(0, index[(int(b), int(h))], int(i)) for b, h, i in rows])
        S_u = np.stack([self.S_ref[b, h] for b, h in units])[None]
        ref_rows = self.oracle.step_rows(unit_view(q, units), unit_view(k, units), unit_view(v, units),
                                         unit_view(g, units), S_u, urows, self._wu(self.wq, units),
                                         self.cos, self.sin, scale=self.scale, eps=self.eps)
        got_rows = got[rows[:, 0], rows[:, 2], rows[:, 1]]
        return rows_error(got_rows, ref_rows, rows)

    # -- commits -------------------------------------------------------------------------
    def _after_commit(self, oracle_call, heads):
        """Reads the GPU state, advances the reference over the followed units and compares them.
        oracle_call(view, S, units) -> new S, with view(t) narrowing [B, L, H, ...] inputs."""
        if heads is not None and set(map(tuple, heads)) != set(self.units):
            self.restrict([tuple(u) for u in heads])
        got = self.layer.get_state().numpy().astype(np.float64)
        self.check_guards()
        assert np.isfinite(got).all()
        if self._all():
            self.S_ref = oracle_call(lambda t: t, self.S_ref, None)
        else:
            units = self.units
            S_u = np.stack([self.S_ref[b, h] for b, h in units])[None]
            S_u = oracle_call(lambda t: None if t is None else unit_view(t, units), S_u, units)
            for n, (b, h) in enumerate(units):
                self.S_ref[b, h] = S_u[0, n]
        err = head_errors(got, self.S_ref, head_axis_first=True)
        return float(err[self.tracked].max())

    def _bh(self, a, units):
        """[B, H] per-unit values -> [1, U]."""
        return a if units is None else torch.stack([a[b, h] for b, h in units]).unsqueeze(0)

    def commit(self, kc, vc, a, heads=None):
        """Gated-linear commit on both sides; worst per-head error of S over the followed units."""
        d = self.dev
        self.layer.commit(kc.to(d), vc.to(d), a.to(d))
        return self._after_commit(
            lambda vw, S, u: self.oracle.commit(vw(kc), vw(vc), self._bh(a, u), S, self._wu(self.wk, u),
                                                self._wu(self.wv, u), self.cos, self.sin, eps=self.eps),
            heads)

    def commit_delta(self, kc, vc, a, beta, heads=None):
        """Delta-rule commit (Eq. 4 at block level) on both sides; worst per-head error of S."""
        d = self.dev
        self.layer.commit_delta(kc.to(d), vc.to(d), a.to(d), None if beta is None else beta.to(d))
        return self._after_commit(
            lambda vw, S, u: self.oracle.commit(vw(kc), vw(vc), self._bh(a, u), S, self._wu(self.wk, u),
                                                self._wu(self.wv, u), self.cos, self.sin, eps=self.eps,
                                                rule=1, beta_logit=vw(beta)),
            heads)

    def commit_decay_tokens(self, kc, vc, alpha, heads=None):
        """Gated-linear commit with per-token forget gates on both sides; worst per-head error of S."""
        d = self.dev
        self.layer.commit_decay_tokens(kc.to(d), vc.to(d), alpha.to(d))
        return self._after_commit(
            lambda vw, S, u: self.oracle.commit_decay_tokens(vw(kc), vw(vc), S, vw(alpha), self._wu(self.wk, u),
                                                             self._wu(self.wv, u), self.cos, self.sin,
                                                             eps=self.eps),
            heads)

    def commit_tokens(self, kc, vc, alpha, beta, heads=None, decayed_prediction=False):
        """Token-sequential commit with per-token gates on both sides; worst per-head error of S."""
        d = self.dev
        dv = lambda t: None if t is None else t.to(d)  # noqa: E731
        self.layer.commit_tokens(kc.to(d), vc.to(d), dv(alpha), dv(beta))
        return self._after_commit(
            lambda vw, S, u: self.oracle.commit_tokens(vw(kc), vw(vc), S, vw(alpha), vw(beta),
                                                       self._wu(self.wk, u), self._wu(self.wv, u), self.cos,
                                                       self.sin, eps=self.eps, decayed_prediction=decayed_prediction),
            heads)

    def clean_pass(self, q, kc, vc, g, a, rows=None):
        """The fused clean pass on both sides.  Returns (output error, state error): every element when
        the oracle follows all units (rows = None), else the sampled rows (b, h, i) and the followed units."""
        d = self.dev
        self.g_out.t.fill_(float("nan"))
        out = self.layer.clean_pass(q.to(d), kc.to(d), vc.to(d), g.to(d), a.to(d), out=self.g_out.t)
        got = out.float().cpu().numpy()
        self.check_guards()
        assert np.isfinite(got).all()
        if rows is None:
            assert self._all()
            ref = self.oracle.step(q, kc, vc, g, self.S_ref, self.wq, self.cos, self.sin,
                                   scale=self.scale, eps=self.eps)
            e_out = float(head_errors(got, ref).max())
        else:
            rows = np.asarray(rows)
            units = sorted({(int(r[0]), int(r[1])) for r in rows})
            assert all(self.tracked[b, h] for b, h in units)
            index = {u: n for n, u in enumerate(units)}
            urows = np.array([(0, index[(int(b), int(h))], int(i)) for b, h, i in rows])
            S_u = np.stack([self.S_ref[b, h] for b, h in units])[None]
            ref_rows = self.oracle.step_rows(unit_view(q, units), unit_view(kc, units), unit_view(vc, units),
                                             unit_view(g, units), S_u, urows, self._wu(self.wq, units),
                                             self.cos, self.sin, scale=self.scale, eps=self.eps)
            e_out = rows_error(got[rows[:, 0], rows[:, 2], rows[:, 1]], ref_rows, rows)
        e_state = self._after_commit(
            lambda vw, S, u: self.oracle.commit(vw(kc), vw(vc), self._bh(a, u), S, self._wu(self.wk, u),
                                                self._wu(self.wv, u), self.cos, self.sin, eps=self.eps),
            None)
        return e_out, e_state

    def _wu(self, w, units):
        return w if (w is None or units is None) else w[[h for _, h in units]]

    def reset(self, stream=-1):
        self.layer.reset(stream)
        self.S_ref = self.oracle.reset(self.S_ref, stream)
        self.S_ref[~self.tracked] = np.nan
        self.check_guards()
