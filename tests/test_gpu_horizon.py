"""Flat cost against the horizon: memory, workspace and state size do not depend on the block index,
and a stream can be reset in the middle of a run without touching the others (Algorithm 1)."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import Pair

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_memory_and_state_are_flat_over_many_blocks():
    cfg = workload.custom(B=2, H=4, D=128, L=700, dtype="bf16", cfg_id=71)
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=DEV)
    wq, wk, wv = (w.to(DEV) for w in workload.feature_weights(cfg))
    cos, sin = (t.to(DEV) for t in workload.rope_tables(cfg.L, cfg.D))
    layer.set_params(wq, wk, wv, cos, sin)
    layer.reset()
    q, k, v, g = (t.to(DEV) for t in workload.step_inputs(cfg, 0, 0))
    kc, vc, a = (t.to(DEV) for t in workload.commit_inputs(cfg, 0))
    out = torch.empty_like(q)
    mem, norms = [], []
    for blk in range(60):
        for _ in range(2):
            layer.denoise_step(q, k, v, g, out=out)
        layer.commit(kc, vc, a)
        torch.cuda.synchronize()
        mem.append(torch.cuda.memory_allocated(DEV))
        if blk % 10 == 9:
            norms.append(float(np.linalg.norm(layer.get_state().numpy())))
    layer.sync_status()
    assert len(set(mem)) == 1, "device memory changed with the block index"
    assert torch.isfinite(out.float()).all()
    # decay logits ~ N(3, .): alpha < 1, the state converges instead of growing with the horizon
    assert norms[-1] < 1.05 * norms[-2]
    assert layer.launch_count > 0


def test_one_stream_reset_mid_run(oracle):
    """Several independent streams; one of them starts a new video at block 2 (S <- 0 for it alone)."""
    cfg = workload.custom(B=3, H=2, D=128, L=300, dtype="bf16", cfg_id=72)
    pair = Pair(oracle, cfg)
    for blk in range(4):
        if blk == 2:
            pair.reset(stream=1)
            got = pair.layer.get_state().numpy()
            assert not got[1].any() and got[0].any() and got[2].any()
        q, k, v, g = workload.step_inputs(cfg, blk, 0)
        assert pair.step_full(q, k, v, g) <= pair.tol
        kc, vc, a = workload.commit_inputs(cfg, blk)
        assert pair.commit(kc, vc, a) <= pair.tol
