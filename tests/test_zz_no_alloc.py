"""arl2_commit_static_scratch: the commit for callers that cannot allocate device memory
(plugins whose host owns the memory pool, code running while a stream is being captured by
someone else).  It keeps the partial sums of the reduction in an array built into the library,
so it needs neither a context nor a workspace.  Checked here on two commits in a row against
the ordinary entry point (arl2_commit on a context) and, directly, against the CPU oracle,
within the tolerance of the other GPU tests.  Collected last on purpose: a failure here cannot
hide the results of the other tests."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import workload
from parity_util import TOL, head_errors

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,D,L", [("fp32", 64, 1100), ("bf16", 128, 700)])
def test_static_scratch_commit_matches_context_commit_and_oracle(oracle, dtype, D, L):
    from paper_2605_16579_b200 import arl2

    dev = "cuda:0"
    cfg = workload.custom(B=2, H=3, D=D, L=L, dtype=dtype, cfg_id=41)
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, dtype, device=dev)
    host_w = workload.feature_weights(cfg)
    host_t = workload.rope_tables(L, D)
    wq, wk, wv = (w.to(dev) for w in host_w)
    cos, sin = (t.to(dev) for t in host_t)
    layer.set_params(wq, wk, wv, cos, sin)
    state = torch.zeros(cfg.B, cfg.H, D, D, dtype=torch.float32, device=dev)
    S_ref = np.zeros((cfg.B, cfg.H, D, D))
    before = torch.cuda.memory_allocated(dev)
    for blk in range(2):   # two calls in a row: the second starts from the first one's state
        hk, hv, ha = workload.commit_inputs(cfg, blk)
        kc, vc, a = hk.to(dev), hv.to(dev), ha.to(dev)
        layer.commit(kc, vc, a)
        arl2.commit_static_scratch(layer.cfg, state, kc, vc, a, wk, wv, cos, sin)
        torch.cuda.synchronize()
        ctx_state = layer.get_state().numpy().astype(np.float64)
        got = state.cpu().numpy()
        assert np.isfinite(got).all()
        err = head_errors(got, ctx_state, head_axis_first=True).max()
        assert err <= TOL[dtype], f"commit {blk} against arl2_commit: {err:.3e} > {TOL[dtype]}"
        S_ref = oracle.commit(hk, hv, ha, S_ref, host_w[1], host_w[2], host_t[0], host_t[1])
        err = head_errors(got, S_ref, head_axis_first=True).max()
        assert err <= TOL[dtype], f"commit {blk} against the oracle: {err:.3e} > {TOL[dtype]}"
        del kc, vc, a
    assert torch.cuda.memory_allocated(dev) == before   # nothing was allocated through torch either
    layer.sync_status()


def test_static_scratch_rejects_oversized_shapes_and_misaligned_pointers():
    from paper_2605_16579_b200 import arl2

    lib = arl2.load()
    dev = "cuda:0"
    # B*H*ceil(L/512)*D*D*4 = 8*12*10*128*128*4 bytes = 63 MB > 8 MiB
    big = arl2.make_config(8, 12, 4680, 128, "bf16")
    dummy = torch.zeros(16, device=dev)
    rc = lib.arl2_commit_static_scratch(ctypes.byref(big), dummy.data_ptr(), dummy.data_ptr(),
                                        dummy.data_ptr(), dummy.data_ptr(), None, None, None, None, None)
    assert rc == -5
    msg = lib.arl2_last_error().decode()
    assert "scratch" in msg and str(arl2.STATIC_SCRATCH_BYTES) in msg
    assert lib.arl2_commit_static_scratch(None, None, None, None, None, None, None, None, None, None) == -1
    # a slice that starts 4 bytes into a buffer is refused on the host, before any launch: the
    # state keeps its contents and the CUDA context stays healthy
    cfg = workload.custom(B=1, H=2, D=64, L=64, dtype="fp32", cfg_id=42)
    c = arl2.make_config(cfg.B, cfg.H, cfg.L, cfg.D, "fp32")
    kc, vc, a = (t.to(dev) for t in workload.commit_inputs(cfg, 0))
    state = torch.full((cfg.B * cfg.H * cfg.D * cfg.D + 4,), 3.0, device=dev)
    cos, sin = (t.to(dev) for t in workload.rope_tables(cfg.L, cfg.D))
    for args in ((state.data_ptr() + 4, kc.data_ptr(), vc.data_ptr(), a.data_ptr(), None, None, None, None),
                 (state.data_ptr(), kc.data_ptr() + 4, vc.data_ptr(), a.data_ptr(), None, None, None, None),
                 (state.data_ptr(), kc.data_ptr(), vc.data_ptr() + 8, a.data_ptr(), None, None, None, None),
                 (state.data_ptr(), kc.data_ptr(), vc.data_ptr(), a.data_ptr(), None, None,
                  cos.data_ptr() + 4, sin.data_ptr())):
        assert lib.arl2_commit_static_scratch(ctypes.byref(c), *args, None) == -1
        assert "aligned" in lib.arl2_last_error().decode()
    torch.cuda.synchronize()
    assert bool((state == 3.0).all())
