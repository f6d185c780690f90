"""The bounded-wait path, exercised without faulting or hanging anything: a test hook shortens the
poll limit of every wait inside the tensor-core kernels to zero, so the first wait of an otherwise
normal launch expires.  The kernel must record the time-out and return through its common exit
(copies in flight awaited, tensor memory freed); the host must report it once, clear it, and the
same context must then work as before."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import arl2, workload
from parity_util import Pair

pytestmark = pytest.mark.gpu


def expect_timeout(layer):
    with pytest.raises(arl2.Arl2Error) as err:
        layer.sync_status()
    text = str(err.value)
    assert "status -4" in text and "site" in text, text
    layer.sync_status()          # the status word was cleared by the report


def test_expired_wait_is_reported_and_the_context_recovers(oracle):
    cfg = workload.custom(B=2, H=3, D=128, L=300, dtype="bf16", cfg_id=81)
    pair = Pair(oracle, cfg)
    assert pair.layer.step_kernel == "tcgen05"
    kc, vc, a = workload.commit_inputs(cfg, 0)
    assert pair.commit(kc, vc, a) <= pair.tol
    q, k, v, g = workload.step_inputs(cfg, 0, 0)
    assert pair.step_full(q, k, v, g) <= pair.tol
    saved = pair.layer.get_state()

    # ---- a denoise pass whose first wait expires
    pair.layer.debug_set_wait_limit(0)
    pair.step_gpu(q, k, v, g)                     # returns; the output is undefined
    expect_timeout(pair.layer)
    assert torch.equal(pair.layer.get_state(), saved)
    # ---- a commit whose first wait expires: the reduction sees the error and leaves S alone
    d = pair.dev
    pair.layer.commit(kc.to(d), vc.to(d), a.to(d))
    expect_timeout(pair.layer)
    assert torch.equal(pair.layer.get_state(), saved)
    pair.check_guards()

    # ---- back to the normal bound: the same context matches the oracle again, twice
    pair.layer.debug_set_wait_limit(-1)
    for blk in (1, 2):
        q, k, v, g = workload.step_inputs(cfg, blk, 0)
        assert pair.step_full(q, k, v, g) <= pair.tol
        kc, vc, a = workload.commit_inputs(cfg, blk)
        assert pair.commit(kc, vc, a) <= pair.tol
    pair.layer.sync_status()


def test_wait_limit_flag_at_creation(oracle):
    cfg = workload.custom(B=1, H=2, D=128, L=200, dtype="bf16", cfg_id=82)
    pair = Pair(oracle, cfg, flags=arl2.ARL2_FLAG_DEBUG_WAIT_LIMIT(0))
    q, k, v, g = workload.step_inputs(cfg, 0, 0)
    pair.step_gpu(q, k, v, g)
    expect_timeout(pair.layer)
    pair.layer.debug_set_wait_limit(-1)
    assert pair.step_full(q, k, v, g) <= pair.tol


def test_two_contexts_from_two_threads(oracle):
    """Distinct contexts are independent: two host threads create their own context and run the same
    seeded pass concurrently (the per-device set-up of the kernels is done once, under a lock)."""
    import threading

    cfg = workload.custom(B=1, H=2, D=128, L=260, dtype="bf16", cfg_id=83)
    q, k, v, g = workload.step_inputs(cfg, 0, 0)
    results, errors = [None, None], []

    def worker(i):
        try:
            dev = "cuda:0"
            s = torch.cuda.Stream(device=dev)
            with torch.cuda.stream(s):
                layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=dev)
                layer.set_params(*(w.to(dev) for w in workload.feature_weights(cfg)),
                                 *(t.to(dev) for t in workload.rope_tables(cfg.L, cfg.D)))
                for _ in range(3):
                    out = layer.denoise_step(q.to(dev), k.to(dev), v.to(dev), g.to(dev))
                layer.sync_status()
                results[i] = out.float().cpu()
        except Exception as e:  # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert torch.equal(results[0], results[1])
    ref = oracle.step(q, k, v, g, np.zeros((cfg.B, cfg.H, cfg.D, cfg.D)), *workload.feature_weights(cfg)[:1],
                      *workload.rope_tables(cfg.L, cfg.D))
    err = np.abs(results[0].numpy() - ref).max() / np.abs(ref).max()
    assert err <= 2e-2
