"""Token-level state access (the comparison mode of the paper's state-access ablation, Sec. 4.3): each
token reads the state advanced by the block's tokens before it.  The CUDA path (attention kernel with
the gate closed, then a chunkwise causal readout on tensor cores) against the oracle's token loop."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import Pair, head_errors, rows_error, unit_view

pytestmark = pytest.mark.gpu


def run(pair, q, k, v, g, alpha):
    d = pair.dev
    pair.g_out.t.fill_(float("nan"))
    out = pair.layer.denoise_step_token_level(q.to(d), k.to(d), v.to(d), g.to(d),
                                              None if alpha is None else alpha.to(d), out=pair.g_out.t)
    got = out.float().cpu().numpy()
    pair.check_guards()
    assert np.isfinite(got).all()
    return got


@pytest.mark.parametrize("B,H,L", [(1, 1, 1), (1, 2, 100), (2, 2, 128), (1, 2, 129), (2, 3, 333), (1, 2, 700)])
@pytest.mark.parametrize("gates", ["near one", "none", "forgetting"])
def test_token_level_matches_oracle(oracle, B, H, L, gates):
    cfg = workload.custom(B=B, H=H, D=128, L=L, dtype="bf16", cfg_id=61)
    pair = Pair(oracle, cfg)
    for blk in range(2):
        q, k, v, g = workload.step_inputs(cfg, blk, 0)
        alpha = None
        if gates != "none":
            alpha = workload.token_gate_logits(cfg, blk, alpha_mean=7.0 if gates == "near one" else 1.5)[0]
        got = run(pair, q, k, v, g, alpha)
        ref = oracle.step_token_level(q, k, v, g, pair.S_ref, alpha, pair.wq, pair.wk, pair.wv, pair.cos, pair.sin)
        err = float(head_errors(got, ref).max())
        assert err <= pair.tol, f"block {blk}: {err:.3e} > {pair.tol}"
        # the state is only read
        before = pair.layer.get_state().numpy().tobytes()
        run(pair, q, k, v, g, alpha)
        assert pair.layer.get_state().numpy().tobytes() == before
        kc, vc, a = workload.commit_inputs(cfg, blk)
        assert pair.commit(kc, vc, a) <= pair.tol
    pair.layer.sync_status()


def test_first_token_and_closed_gate_equal_the_frame_level_layer(oracle):
    cfg = workload.custom(B=1, H=2, D=128, L=260, dtype="bf16", cfg_id=62)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    pair.commit(kc, vc, a)
    q, k, v, g = workload.step_inputs(cfg, 1, 0)
    tok = run(pair, q, k, v, g, None)
    frame = pair.step_gpu(q, k, v, g)
    # token 0 reads S itself: same arithmetic up to the rounding of a second pass over the output
    e0 = np.abs(tok[:, 0] - frame[:, 0]).max() / np.abs(frame[:, 0]).max()
    assert e0 <= 1e-2, e0
    assert np.abs(tok[:, 5:] - frame[:, 5:]).max() > 1e-2 * np.abs(frame).max()
    closed = torch.full_like(g, -40.0)
    np.testing.assert_array_equal(run(pair, q, k, v, closed, None), pair.step_gpu(q, k, v, closed))


def test_token_level_full_size_sampled(oracle):
    """The bench's largest configuration on sampled rows of three heads (the oracle walks all tokens of
    those heads, which is what a token's state depends on)."""
    cfg = workload.CONFIGS["long"]
    units = workload.sample_units(cfg, heads_per_stream=3)
    pair = Pair(oracle, cfg, units=units)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    pair.commit(kc, vc, a)
    q, k, v, g = workload.step_inputs(cfg, 1, 0)
    alpha = workload.token_gate_logits(cfg, 1)[0]
    got = run(pair, q, k, v, g, alpha)
    S_u = np.stack([pair.S_ref[b, h] for b, h in units])[None]
    ref = oracle.step_token_level(unit_view(q, units), unit_view(k, units), unit_view(v, units), unit_view(g, units),
                                  S_u, unit_view(alpha, units), pair._wu(pair.wq, units), pair._wu(pair.wk, units),
                                  pair._wu(pair.wv, units), pair.cos, pair.sin)
    for n, (b, h) in enumerate(units):
        err = np.abs(got[b, :, h] - ref[0, :, n]).max() / np.abs(ref[0, :, n]).max()
        assert err <= pair.tol, f"unit {(b, h)}: {err:.3e}"
    pair.layer.sync_status()


def test_token_level_needs_the_tensor_core_context(oracle):
    cfg = workload.custom(B=1, H=2, D=64, L=64, dtype="fp32", cfg_id=63)
    pair = Pair(oracle, cfg)
    q, k, v, g = (t.to(pair.dev) for t in workload.step_inputs(cfg, 0, 0))
    with pytest.raises(arl2.Arl2Error, match="status -2"):
        pair.layer.denoise_step_token_level(q, k, v, g)
