"""Scalar and elementwise combine gates (the granularities of the paper's gate ablation) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import TOL, head_errors

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(oracle, cfg, gate_mode, flags):
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=DEV, flags=flags)
    wq, wk, wv = workload.feature_weights(cfg)
    cos, sin = workload.rope_tables(cfg.L, cfg.D)
    layer.set_params(wq.to(DEV), wk.to(DEV), wv.to(DEV), cos.to(DEV), sin.to(DEV))
    S = np.zeros((cfg.B, cfg.H, cfg.D, cfg.D))
    worst = 0.0
    for blk in range(2):
        q, k, v, g = workload.step_inputs(cfg, blk, 0)
        gen = torch.Generator(device="cpu")
        gen.manual_seed(9000 + blk)
        shape = {1: (cfg.B, cfg.L), 2: (cfg.B, cfg.L, cfg.H, cfg.D)}[gate_mode]
        gate = torch.randn(shape, generator=gen, dtype=torch.float32)      # gates well away from 1/2
        got = layer.denoise_step(q.to(DEV), k.to(DEV), v.to(DEV), gate.to(DEV)).float().cpu().numpy()
        ref = oracle.step_gate_mode(q, k, v, gate, S, gate_mode, wq, cos, sin)
        assert np.isfinite(got).all()
        worst = max(worst, float(head_errors(got, ref).max()))
        kc, vc, a = workload.commit_inputs(cfg, blk)
        layer.commit(kc.to(DEV), vc.to(DEV), a.to(DEV))
        S = oracle.commit(kc, vc, a, S, wk, wv, cos, sin)
    layer.sync_status()
    return worst


@pytest.mark.parametrize("dtype,D,B,H,L", [
    ("fp32", 64, 1, 2, 200),
    ("bf16", 128, 2, 3, 333),      # tensor-core kernels, ragged tiles packed across units
    ("bf16", 128, 1, 2, 640),
    ("bf16", 64, 1, 2, 130),       # plain-FMA kernels with bf16 I/O
])
@pytest.mark.parametrize("gate_mode", [1, 2])
def test_gate_granularities_match_oracle(oracle, gate_mode, dtype, D, B, H, L):
    cfg = workload.custom(B=B, H=H, D=D, L=L, dtype=dtype, cfg_id=81)
    flags = arl2.ARL2_FLAG_GATE_SCALAR if gate_mode == 1 else arl2.ARL2_FLAG_GATE_ELEMENTWISE
    err = _run(oracle, cfg, gate_mode, flags)
    assert err <= TOL[dtype], f"error {err:.3e}"


def test_both_gate_flags_are_rejected():
    with pytest.raises(arl2.Arl2Error, match="exclude"):
        arl2.Layer(1, 2, 64, 64, "fp32", device=DEV,
                   flags=arl2.ARL2_FLAG_GATE_SCALAR | arl2.ARL2_FLAG_GATE_ELEMENTWISE)
