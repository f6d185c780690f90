"""Delta-rule state commit (Eq. 4 as printed, applied once per block) against the oracle's rule 1."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import workload
from parity_util import Pair

pytestmark = pytest.mark.gpu


def _blocks(pair, cfg, schedule):
    """schedule: list of 'd' (delta commit), 'g' (gated-linear commit), 's' (denoise step)."""
    worst = 0.0
    for blk, what in enumerate(schedule):
        if what == "s":
            q, k, v, g = workload.step_inputs(cfg, blk, 0)
            err = pair.step_full(q, k, v, g)
        else:
            kc, vc, a = workload.commit_inputs(cfg, blk)
            if what == "d":
                err = pair.commit_delta(kc, vc, a, workload.beta_logits(cfg, blk))
            else:
                err = pair.commit(kc, vc, a)
        assert err <= pair.tol, f"block {blk} ({what}): error {err:.3e} > {pair.tol}"
        worst = max(worst, err)
    return worst


@pytest.mark.parametrize("dtype,D,B,H,L", [
    ("fp32", 64, 1, 2, 256),
    ("fp32", 128, 2, 2, 700),      # two chunks, ragged tail
    ("fp32", 64, 2, 3, 1100),      # three chunks
    ("bf16", 64, 1, 2, 333),       # plain-FMA kernels with bf16 I/O
    ("bf16", 128, 1, 2, 128),      # tensor-core path, exactly one tile
    ("bf16", 128, 2, 3, 700),      # two chunks, ragged tail, several streams
    ("bf16", 128, 1, 2, 1100),     # three chunks
])
def test_delta_commit_matches_oracle(oracle, dtype, D, B, H, L):
    cfg = workload.custom(B=B, H=H, D=D, L=L, dtype=dtype, cfg_id=31)
    pair = Pair(oracle, cfg)
    # the first delta commit sees S_old = 0 (pure outer-product sum); the later ones a full state
    _blocks(pair, cfg, ["d", "d", "s", "g", "d", "s"])


def test_delta_commit_without_beta_is_beta_one(oracle):
    cfg = workload.custom(B=1, H=2, D=128, L=200, dtype="bf16", cfg_id=32)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    assert pair.commit(kc, vc, a) <= pair.tol
    kc, vc, a = workload.commit_inputs(cfg, 1)
    assert pair.commit_delta(kc, vc, a, None) <= pair.tol


def test_delta_commit_on_zero_state_equals_gated_linear_with_beta_weights(oracle):
    """With S_old = 0 the prediction vanishes: the result is sum_l beta_l K'_l^T V'_l."""
    cfg = workload.custom(B=1, H=2, D=128, L=300, dtype="bf16", cfg_id=33)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    big = torch.full((cfg.B, cfg.L, cfg.H), 30.0)   # sigmoid = 1 to fp32 precision
    assert pair.commit_delta(kc, vc, a, big) <= pair.tol
    s_delta = pair.layer.get_state().numpy()
    pair.reset()
    assert pair.commit(kc, vc, a) <= pair.tol
    s_lin = pair.layer.get_state().numpy()
    np.testing.assert_array_equal(s_delta, s_lin)   # same kernels' arithmetic, bit for bit


def test_delta_commit_is_reproducible(oracle):
    cfg = workload.custom(B=2, H=2, D=128, L=700, dtype="bf16", cfg_id=34)
    outs = []
    for _ in range(2):
        pair = Pair(oracle, cfg)
        for blk in range(2):
            kc, vc, a = workload.commit_inputs(cfg, blk)
            pair.commit_delta(kc, vc, a, workload.beta_logits(cfg, blk))
        outs.append(pair.layer.get_state().numpy())
    np.testing.assert_array_equal(outs[0], outs[1])


def test_delta_commit_full_size_sampled_heads(oracle):
    """The bench's largest configuration; S compared in full for a few (stream, head) units."""
    cfg = workload.CONFIGS["long"]
    pair = Pair(oracle, cfg)
    heads = [(0, 0), (0, 17), (0, cfg.H - 1)]
    for blk in range(3):
        kc, vc, a = workload.commit_inputs(cfg, blk)
        err = pair.commit_delta(kc, vc, a, workload.beta_logits(cfg, blk), heads=heads)
        assert err <= pair.tol, f"block {blk}: error {err:.3e}"
