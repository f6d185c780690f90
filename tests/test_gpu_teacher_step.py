"""Eq. 1 over a key/value cache (the teacher's layer, for the horizon comparison) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import TOL, head_errors

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(cfg, lk, seed):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    q = torch.randn(cfg.B, cfg.L, cfg.H, cfg.D, generator=gen).to(torch.bfloat16)
    k = torch.randn(cfg.B, lk, cfg.H, cfg.D, generator=gen).to(torch.bfloat16)
    v = torch.randn(cfg.B, lk, cfg.H, cfg.D, generator=gen).to(torch.bfloat16)
    return q, k, v


@pytest.mark.parametrize("B,H,L,Lk", [
    (1, 2, 128, 128),      # cache = the block itself
    (1, 2, 256, 700),      # longer cache, ragged last key tile
    (2, 3, 333, 1000),     # ragged query tiles packed across (stream, head) units
    (1, 3, 100, 50),       # cache shorter than the block
    (1, 1, 300, 2500),
])
def test_teacher_step_matches_oracle(oracle, B, H, L, Lk):
    cfg = workload.custom(B=B, H=H, D=128, L=L, dtype="bf16", cfg_id=51)
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=DEV)
    wq, wk, wv = (w.to(DEV) for w in workload.feature_weights(cfg))
    cos, sin = (t.to(DEV) for t in workload.rope_tables(cfg.L, cfg.D))
    layer.set_params(wq, wk, wv, cos, sin)      # must play no part
    kc, vc, a = (t.to(DEV) for t in workload.commit_inputs(cfg, 0))
    layer.reset()
    layer.commit(kc, vc, a)                      # a non-zero state, which must play no part either
    q, k, v = _inputs(cfg, Lk, 1234 + Lk)
    got = layer.teacher_step(q.to(DEV), k.to(DEV), v.to(DEV)).float().cpu().numpy()
    layer.sync_status()
    ref = oracle.attend_cache(q, k, v)
    assert np.isfinite(got).all()
    err = float(head_errors(got, ref).max())
    assert err <= TOL["bf16"], f"error {err:.3e}"
    # the layer itself still works afterwards (the two entry points share the scheduler counters)
    qq, kk, vv, g = workload.step_inputs(cfg, 0, 0)
    out = layer.denoise_step(qq.to(DEV), kk.to(DEV), vv.to(DEV), g.to(DEV))
    assert torch.isfinite(out.float()).all()


def test_teacher_step_full_size_sampled_rows(oracle):
    """The base geometry over a cache of two blocks: 222 work items on 148 SMs, the last 74 cut into
    two ranges of 37 key tiles each.  Query rows are independent, so the oracle takes sampled rows
    (tile edges, the ragged tail tile in full) as a shorter block over the whole cache."""
    cfg = workload.CONFIGS["chunked"]
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=DEV)
    lk = 2 * cfg.L
    q, k, v = _inputs(cfg, lk, 4321)
    out = torch.full((cfg.B, cfg.L, cfg.H, cfg.D), float("nan"), dtype=torch.bfloat16, device=DEV)
    layer.teacher_step(q.to(DEV), k.to(DEV), v.to(DEV), out=out)
    layer.sync_status()
    assert torch.isfinite(out.float()).all()
    gen = torch.Generator().manual_seed(99)
    rows = sorted(set([0, 127, 128, 255, 256, 4479, 4480, 4607] + list(range(4608, cfg.L))
                      + torch.randint(0, cfg.L, (40,), generator=gen).tolist()))
    ref = oracle.attend_cache(q[:, rows].contiguous(), k, v)
    got = out.index_select(1, torch.tensor(rows, device=DEV)).float().cpu().numpy()
    err = float(head_errors(got, ref).max())
    print(f"teacher step, chunked geometry, cache of 2 blocks: error {err:.2e} on {len(rows)} rows per head")
    assert err <= TOL["bf16"], f"error {err:.3e}"


def test_teacher_step_rejects_other_contexts(oracle):
    cfg = workload.custom(B=1, H=2, D=64, L=64, dtype="fp32", cfg_id=52)
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=DEV)
    q = torch.zeros(1, 64, 2, 64, device=DEV)
    with pytest.raises(arl2.Arl2Error, match="D = 128"):
        layer.teacher_step(q, q.clone(), q.clone())
