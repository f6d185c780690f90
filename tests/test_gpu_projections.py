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


@pytest.mark.parametrize("B,H", [(1, 12), (2, 20)])
def test_projections_full_size_sampled_rows(oracle, B, H):
    """The base model's geometry (4680 tokens, d = 1536) and a wider, two-stream one: 37 and 74 row
    tiles walk more than one band of the persistent tile order, the output projection takes the
    192-column tile.  A GEMM's rows are independent, so the oracle computes sampled rows (first and
    last rows of tiles, band boundaries, the ragged tail tile in full) as a shorter sequence."""
    L, d = 4680, H * 128
    layer = arl2.Layer(B, H, L, 128, "bf16", device=DEV)
    w_q, w_k, w_v, w_g, w_o = weights(d, H, 27)
    layer.set_projections(*(w.to(DEV) for w in (w_q, w_k, w_v, w_g, w_o)))
    gen = torch.Generator().manual_seed(28)
    x = torch.randn(B, L, d, generator=gen).to(torch.bfloat16)
    o = torch.randn(B, L, H, 128, generator=gen).to(torch.bfloat16)
    rows = sorted(set([0, 1, 127, 128, 255, 256, 4095, 4096, 4097, 4223, 4224]
                      + list(range(4608, 4680))
                      + torch.randint(0, L, (48,), generator=gen).tolist()))
    nan = float("nan")
    q, k, v = (torch.full((B, L, H, 128), nan, dtype=torch.bfloat16, device=DEV) for _ in range(3))
    g = torch.full((B, L, H), nan, device=DEV)
    y = torch.full((B, L, d), nan, dtype=torch.bfloat16, device=DEV)
    layer.project_in(x.to(DEV), q, k, v, g)
    layer.project_out(o.to(DEV), y)
    layer.sync_status()
    for t in (q, k, v, g, y):
        assert torch.isfinite(t.float()).all()          # every element was written
    rq, rk, rv, rg = oracle.project_in(x[:, rows].contiguous(), w_q, w_k, w_v, w_g, H)
    ry = oracle.project_out(o[:, rows].contiguous(), w_o)
    idx = torch.tensor(rows, device=DEV)
    worst = 0.0
    for name, got, ref in (("q", q, rq), ("k", k, rk), ("v", v, rv), ("g", g, rg), ("y", y, ry)):
        e = norm_err(got.index_select(1, idx).float().cpu().numpy(), ref)
        worst = max(worst, e)
        assert e <= TOL["bf16"], (name, e)
    print(f"projections B={B} H={H} L={L}: worst normalised error {worst:.2e} on {len(rows)} rows per stream")


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
