"""Shared machinery of the GPU parity tests: runs the same seeded schedule through the CUDA
library (via its C ABI binding) and through the CPU float64 oracle and compares them.

Error measure (stated tolerance: 2e-2 for bf16 I/O, 1e-4 in fp32 mode): for each output
tensor and each (stream, head), max|gpu - ref| / max|ref| -- an element-wise relative
error is unbounded next to zeros of the reference.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2605_16579_b200 import workload

TOL = {"bf16": 2e-2, "fp32": 1e-4}


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


class Pair:
    """The CUDA layer and the oracle side by side on one configuration."""

    def __init__(self, oracle, cfg, device="cuda:0", rope=True, maps=True, flags=0, eps=0.0,
                 scale=0.0):
        from paper_2605_16579_b200 import arl2

        self.oracle, self.cfg, self.dev = oracle, cfg, device
        self.layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=device,
                                softmax_scale=scale, l2_eps=eps, flags=flags)
        self.eps = eps if eps > 0 else 1e-6
        self.scale = scale if scale > 0 else None
        self.wq = self.wk = self.wv = self.cos = self.sin = None
        if maps:
            self.wq, self.wk, self.wv = workload.feature_weights(cfg)
        if rope:
            self.cos, self.sin = workload.rope_tables(cfg.L, cfg.D)
        dv = lambda t: None if t is None else t.to(device)  # noqa: E731
        self.layer.set_params(dv(self.wq), dv(self.wk), dv(self.wv), dv(self.cos), dv(self.sin))
        self.S_ref = np.zeros((cfg.B, cfg.H, cfg.D, cfg.D))
        self.tol = TOL[cfg.dtype]

    def step_gpu(self, q, k, v, g):
        d = self.dev
        return self.layer.denoise_step(q.to(d), k.to(d), v.to(d), g.to(d)).float().cpu().numpy()

    def step_full(self, q, k, v, g):
        """Full comparison of one step; returns the worst per-head error."""
        got = self.step_gpu(q, k, v, g)
        ref = self.oracle.step(q, k, v, g, self.S_ref, self.wq, self.cos, self.sin,
                               scale=self.scale, eps=self.eps)
        assert np.isfinite(got).all()
        return float(head_errors(got, ref).max())

    def step_sampled(self, q, k, v, g, rows):
        got = self.step_gpu(q, k, v, g)
        assert np.isfinite(got).all()
        rows = np.asarray(rows)
        got_rows = got[rows[:, 0], rows[:, 2], rows[:, 1]]
        ref_rows = self.oracle.step_rows(q, k, v, g, self.S_ref, rows, self.wq, self.cos, self.sin,
                                         scale=self.scale, eps=self.eps)
        return rows_error(got_rows, ref_rows, rows)

    def commit(self, kc, vc, a, heads=None):
        """Commit on both sides; returns the worst per-head error of S (over `heads` if given)."""
        d = self.dev
        self.layer.commit(kc.to(d), vc.to(d), a.to(d))
        got = self.layer.get_state().numpy().astype(np.float64)
        self.S_ref = self.oracle.commit(kc, vc, a, self.S_ref, self.wk, self.wv, self.cos, self.sin,
                                        eps=self.eps, heads=heads)
        assert np.isfinite(got).all()
        err = head_errors(got, self.S_ref, head_axis_first=True)
        if heads is not None:
            # heads the oracle skipped follow the GPU from here on (they are not compared)
            mask = np.zeros(err.shape, dtype=bool)
            for b, h in heads:
                mask[b, h] = True
            self.S_ref[~mask] = got[~mask]
            err = err[mask]
        return float(err.max())

    def commit_delta(self, kc, vc, a, beta, heads=None):
        """Delta-rule commit (Eq. 4 at block level) on both sides; worst per-head error of S."""
        d = self.dev
        self.layer.commit_delta(kc.to(d), vc.to(d), a.to(d), None if beta is None else beta.to(d))
        got = self.layer.get_state().numpy().astype(np.float64)
        self.S_ref = self.oracle.commit(kc, vc, a, self.S_ref, self.wk, self.wv, self.cos, self.sin,
                                        eps=self.eps, rule=1, beta_logit=beta, heads=heads)
        assert np.isfinite(got).all()
        err = head_errors(got, self.S_ref, head_axis_first=True)
        if heads is not None:
            mask = np.zeros(err.shape, dtype=bool)
            for b, h in heads:
                mask[b, h] = True
            self.S_ref[~mask] = got[~mask]
            err = err[mask]
        return float(err.max())

    def commit_decay_tokens(self, kc, vc, alpha, heads=None):
        """Gated-linear commit with per-token forget gates on both sides; worst per-head error of S."""
        d = self.dev
        self.layer.commit_decay_tokens(kc.to(d), vc.to(d), alpha.to(d))
        got = self.layer.get_state().numpy().astype(np.float64)
        self.S_ref = self.oracle.commit_decay_tokens(kc, vc, self.S_ref, alpha, self.wk, self.wv,
                                                     self.cos, self.sin, eps=self.eps, heads=heads)
        assert np.isfinite(got).all()
        err = head_errors(got, self.S_ref, head_axis_first=True)
        if heads is not None:
            mask = np.zeros(err.shape, dtype=bool)
            for b, h in heads:
                mask[b, h] = True
            self.S_ref[~mask] = got[~mask]
            err = err[mask]
        return float(err.max())

    def commit_tokens(self, kc, vc, alpha, beta, heads=None):
        """Token-sequential commit with per-token gates on both sides; worst per-head error of S."""
        d = self.dev
        dv = lambda t: None if t is None else t.to(d)  # noqa: E731
        self.layer.commit_tokens(kc.to(d), vc.to(d), dv(alpha), dv(beta))
        got = self.layer.get_state().numpy().astype(np.float64)
        self.S_ref = self.oracle.commit_tokens(kc, vc, self.S_ref, alpha, beta, self.wk, self.wv,
                                               self.cos, self.sin, eps=self.eps, heads=heads)
        assert np.isfinite(got).all()
        err = head_errors(got, self.S_ref, head_axis_first=True)
        if heads is not None:
            mask = np.zeros(err.shape, dtype=bool)
            for b, h in heads:
                mask[b, h] = True
            self.S_ref[~mask] = got[~mask]
            err = err[mask]
        return float(err.max())

    def reset(self, stream=-1):
        self.layer.reset(stream)
        self.S_ref = self.oracle.reset(self.S_ref, stream)
