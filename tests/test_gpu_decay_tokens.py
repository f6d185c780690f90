"""Gated-linear commit with one forget gate per token against the oracle's token-by-token loop."""
import numpy as np
import pytest

from paper_2605_16579_b200 import workload
from parity_util import Pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,D,B,H,L", [
    ("fp32", 64, 1, 2, 1),
    ("fp32", 64, 2, 3, 300),
    ("fp32", 128, 1, 2, 700),      # two commit chunks, more tokens than scan threads
    ("bf16", 64, 1, 2, 333),
    ("bf16", 128, 2, 3, 700),      # tensor-core kernels
    ("bf16", 128, 1, 2, 1100),
])
def test_decay_tokens_matches_oracle(oracle, dtype, D, B, H, L):
    cfg = workload.custom(B=B, H=H, D=D, L=L, dtype=dtype, cfg_id=61)
    pair = Pair(oracle, cfg)
    for blk in range(3):
        kc, vc, a = workload.commit_inputs(cfg, blk)
        alpha, _ = workload.token_gate_logits(cfg, blk)
        err = pair.commit_decay_tokens(kc, vc, alpha)
        assert err <= pair.tol, f"block {blk}: error {err:.3e} > {pair.tol}"
    # strong forgetting, then a plain commit and a denoise pass on the same context
    kc, vc, a = workload.commit_inputs(cfg, 3)
    alpha, _ = workload.token_gate_logits(cfg, 3, alpha_mean=1.0)
    assert pair.commit_decay_tokens(kc, vc, alpha) <= pair.tol
    assert pair.commit(kc, vc, a) <= pair.tol
    q, k, v, g = workload.step_inputs(cfg, 0, 0)
    assert pair.step_full(q, k, v, g) <= pair.tol


def test_decay_tokens_full_size_sampled_heads(oracle):
    cfg = workload.CONFIGS["long"]
    pair = Pair(oracle, cfg)
    heads = [(0, 0), (0, cfg.H - 1)]
    for blk in range(2):
        kc, vc, _ = workload.commit_inputs(cfg, blk)
        alpha, _ = workload.token_gate_logits(cfg, blk)
        err = pair.commit_decay_tokens(kc, vc, alpha, heads=heads)
        assert err <= pair.tol, f"block {blk}: error {err:.3e}"
