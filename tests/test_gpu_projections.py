"""The projections around the core (Sec. 3.1, Eq. 6-7) on the tcgen05 GEMM kernel against the oracle's
plain matrix products, and the whole module (project in -> layer -> project out) against the oracle's
composition."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import Pair, TOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def weights(d, H, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: (torch.randn(*s, generator=g) / np.sqrt(d)).to(torch.bfloat16)  # noqa: E731
    return mk(d, d), mk(d, d), mk(d, d), mk(d, H), mk(d, d)


def norm_err(got, ref):
    return float(np.abs(np.asarray(got, dtype=np.float64) - ref).max() / np.abs(ref).max())


@pytest.mark.parametrize("B,H,L", [(1, 1, 1), (1, 2, 100), (2, 3, 333), (1, 12, 700), (3, 5, 129)])
def test_projections_match_oracle(oracle, B, H, L):
    d = H * 128
    layer = arl2.Layer(B, H, L, 128, "bf16", device=DEV)
    w_q, w_k, w_v, w_g, w_o = weights(d, H, 7)
    layer.set_projections(*(w.to(DEV) for w in (w_q, w_k, w_v, w_g, w_o)))
    x = torch.randn(B, L, d, generator=torch.Generator().manual_seed(8)).to(torch.bfloat16)
    nan = float("nan")
    q, k, v = (torch.full((B, L, H, 128), nan, dtype=torch.bfloat16, device=DEV) for _ in range(3))
    g = torch.full((B, L, H), nan, device=DEV)
    layer.project_in(x.to(DEV), q, k, v, g)
    rq, rk, rv, rg = oracle.project_in(x, w_q, w_k, w_v, w_g, H)
    for name, got, ref in (("q", q, rq), ("k", k, rk), ("v", v, rv), ("g", g, rg)):
        got = got.float().cpu().numpy()
        assert np.isfinite(got).all(), name
        assert norm_err(got, ref) <= TOL["bf16"], (name, norm_err(got, ref))
    o = torch.randn(B, L, H, 128, generator=torch.Generator().manual_seed(9)).to(torch.bfloat16)
    y = torch.full((B, L, d), nan, dtype=torch.bfloat16, device=DEV)
    layer.project_out(o.to(DEV), y)
    y = y.float().cpu().numpy()
    assert np.isfinite(y).all()
    assert norm_err(y, oracle.project_out(o, w_o)) <= TOL["bf16"]
    layer.sync_status()


def test_whole_module_against_the_oracle_composition(oracle):
    """x -> (W_q, W_k, W_v, W_g) -> hybrid core -> W_o, Eq. 7: y' = (O_intra + G . O_inter) W_o."""
    cfg = workload.custom(B=2, H=3, D=128, L=333, dtype="bf16", cfg_id=91)
    pair = Pair(oracle, cfg)
    d = cfg.H * cfg.D
    w_q, w_k, w_v, w_g, w_o = weights(d, cfg.H, 17)
    pair.layer.set_projections(*(w.to(DEV) for w in (w_q, w_k, w_v, w_g, w_o)))
    kc, vc, a = workload.commit_inputs(cfg, 0)
    assert pair.commit(kc, vc, a) <= pair.tol          # a non-zero state
    x = (3.0 * torch.randn(cfg.B, cfg.L, d, generator=torch.Generator().manual_seed(18))).to(torch.bfloat16)
    q, k, v, g = pair.layer.project_in(x.to(DEV))
    o = pair.layer.denoise_step(q, k, v, g)
    y = pair.layer.project_out(o).float().cpu().numpy()
    # the oracle, given what the device passes from stage to stage rounded the same way (bf16 tensors
    # between the calls are part of the interface), and once more end to end in float64
    rq, rk, rv, rg = oracle.project_in(x, w_q, w_k, w_v, w_g, cfg.H)
    ro = oracle.step(rq, rk, rv, rg, pair.S_ref, pair.wq, pair.cos, pair.sin)
    ry = oracle.project_out(ro, w_o)
    assert norm_err(y, ry) <= pair.tol, norm_err(y, ry)
    pair.layer.sync_status()


def test_projection_argument_errors(oracle):
    layer = arl2.Layer(1, 2, 64, 128, "bf16", device=DEV)
    lib = arl2.load()
    x = torch.zeros(1, 64, 256, dtype=torch.bfloat16, device=DEV)
    assert lib.arl2_project_in(layer._ctx, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), None) == -1
    assert b"set_projections" in lib.arl2_last_error()
    assert lib.arl2_project_out(layer._ctx, x.data_ptr(), x.data_ptr(), None) == -1
    simt = arl2.Layer(1, 2, 64, 64, "fp32", device=DEV)
    assert lib.arl2_set_projections(simt._ctx, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                    x.data_ptr(), 1 << 20, None) == -2
