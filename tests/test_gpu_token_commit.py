"""Eq. 4 applied token by token with per-token gates (chunkwise kernels) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import Pair

pytestmark = pytest.mark.gpu
FLAG = arl2.ARL2_FLAG_TOKEN_GATES


@pytest.mark.parametrize("dtype,D,B,H,L", [
    ("fp32", 64, 1, 2, 64),        # exactly one chunk
    ("fp32", 64, 2, 3, 200),       # ragged last chunk
    ("fp32", 128, 1, 2, 333),
    ("bf16", 64, 1, 2, 130),
    ("bf16", 128, 2, 3, 700),      # tensor-core context: the bf16 copy of S is refreshed
    ("bf16", 128, 1, 2, 1),        # a single token
])
def test_token_commit_matches_oracle(oracle, dtype, D, B, H, L):
    cfg = workload.custom(B=B, H=H, D=D, L=L, dtype=dtype, cfg_id=41)
    pair = Pair(oracle, cfg, flags=FLAG)
    for blk in range(3):
        kc, vc, _ = workload.commit_inputs(cfg, blk)
        alpha, beta = workload.token_gate_logits(cfg, blk)
        err = pair.commit_tokens(kc, vc, alpha, beta)
        assert err <= pair.tol, f"block {blk}: error {err:.3e} > {pair.tol}"
        # the denoise pass reads the state this commit wrote (and its operand copy)
        q, k, v, g = workload.step_inputs(cfg, blk, 0)
        err = pair.step_full(q, k, v, g)
        assert err <= pair.tol, f"block {blk}: step error {err:.3e} > {pair.tol}"


def test_token_commit_strong_forgetting_and_missing_gates(oracle):
    cfg = workload.custom(B=1, H=2, D=64, L=150, dtype="fp32", cfg_id=42)
    pair = Pair(oracle, cfg, flags=FLAG)
    kc, vc, _ = workload.commit_inputs(cfg, 0)
    alpha, beta = workload.token_gate_logits(cfg, 0, alpha_mean=1.0, beta_mean=2.0)
    assert pair.commit_tokens(kc, vc, alpha, beta) <= pair.tol
    kc, vc, _ = workload.commit_inputs(cfg, 1)
    assert pair.commit_tokens(kc, vc, None, beta) <= pair.tol      # alpha = 1
    assert pair.commit_tokens(kc, vc, alpha, None) <= pair.tol     # beta = 1
    assert pair.commit_tokens(kc, vc, None, None) <= pair.tol


def test_token_commit_mixes_with_the_other_commits(oracle):
    cfg = workload.custom(B=1, H=2, D=128, L=300, dtype="bf16", cfg_id=43)
    pair = Pair(oracle, cfg, flags=FLAG)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    assert pair.commit(kc, vc, a) <= pair.tol
    alpha, beta = workload.token_gate_logits(cfg, 1)
    kc, vc, a = workload.commit_inputs(cfg, 1)
    assert pair.commit_tokens(kc, vc, alpha, beta) <= pair.tol
    kc, vc, a = workload.commit_inputs(cfg, 2)
    assert pair.commit_delta(kc, vc, a, workload.beta_logits(cfg, 2)) <= pair.tol


def test_token_commit_is_reproducible_and_needs_the_flag(oracle):
    cfg = workload.custom(B=2, H=2, D=128, L=260, dtype="bf16", cfg_id=44)
    outs = []
    for _ in range(2):
        pair = Pair(oracle, cfg, flags=FLAG)
        kc, vc, _ = workload.commit_inputs(cfg, 0)
        alpha, beta = workload.token_gate_logits(cfg, 0)
        pair.commit_tokens(kc, vc, alpha, beta)
        pair.commit_tokens(kc, vc, alpha, beta)
        outs.append(pair.layer.get_state().numpy())
    np.testing.assert_array_equal(outs[0], outs[1])
    plain = Pair(oracle, cfg)
    d = plain.dev
    with pytest.raises(arl2.Arl2Error, match="TOKEN_GATES"):
        plain.layer.commit_tokens(kc.to(d), vc.to(d), alpha.to(d), beta.to(d))


def test_token_commit_full_size_sampled_heads(oracle):
    cfg = workload.CONFIGS["long"]
    pair = Pair(oracle, cfg, flags=FLAG)
    heads = [(0, 0), (0, cfg.H - 1)]
    for blk in range(2):
        kc, vc, _ = workload.commit_inputs(cfg, blk)
        alpha, beta = workload.token_gate_logits(cfg, blk)
        err = pair.commit_tokens(kc, vc, alpha, beta, heads=heads)
        assert err <= pair.tol, f"block {blk}: error {err:.3e}"


@pytest.mark.parametrize("dtype,D,B,H,L", [("fp32", 64, 1, 2, 200), ("bf16", 128, 2, 3, 333), ("bf16", 128, 1, 2, 1100)])
def test_token_commit_with_the_prediction_against_the_decayed_state(oracle, dtype, D, B, H, L):
    """The other reading of Eq. 4 (each token predicts against alpha_j S_{j-1}), chosen by a context flag."""
    from paper_2605_16579_b200 import arl2

    cfg = workload.custom(B=B, H=H, D=D, L=L, dtype=dtype, cfg_id=46)
    pair = Pair(oracle, cfg, flags=FLAG | arl2.ARL2_FLAG_DELTA_DECAYED_PREDICTION)
    plain = Pair(oracle, cfg, flags=FLAG)
    for blk in range(3):
        kc, vc, _ = workload.commit_inputs(cfg, blk)
        alpha, beta = workload.token_gate_logits(cfg, blk, alpha_mean=3.0)
        err = pair.commit_tokens(kc, vc, alpha, beta, decayed_prediction=True)
        assert err <= pair.tol, f"block {blk}: error {err:.3e} > {pair.tol}"
        assert plain.commit_tokens(kc, vc, alpha, beta) <= plain.tol
    # the two readings do differ on these inputs
    a, b = pair.layer.get_state().numpy(), plain.layer.get_state().numpy()
    assert np.abs(a - b).max() > 1e-3 * np.abs(b).max()
