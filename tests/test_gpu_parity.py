"""GPU parity: the CUDA library (through its C ABI) against the CPU float64 oracle on the
same seeded inputs.  Small and ragged shapes are compared element by element; the full-size
configurations on seeded samples of rows (always including the ragged tail tile) and on the
full state of sampled heads after every commit."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import workload
from parity_util import Pair, head_errors

pytestmark = pytest.mark.gpu


def run_schedule(pair, blocks, steps, full=True, heads_per_stream=2, rows_per_head=64):
    cfg = pair.cfg
    worst_o, worst_s = 0.0, 0.0
    for blk in range(blocks):
        for st in range(steps):
            q, k, v, g = workload.step_inputs(cfg, blk, st)
            if full:
                e = pair.step_full(q, k, v, g)
            else:
                rows = workload.sample_rows(cfg, blk, st, heads_per_stream, rows_per_head)
                e = pair.step_sampled(q, k, v, g, rows)
            worst_o = max(worst_o, e)
            assert e <= pair.tol, f"block {blk} step {st}: output error {e:.3e} > {pair.tol}"
        kc, vc, a = workload.commit_inputs(cfg, blk)
        heads = None
        if not full:
            heads = sorted({(b, h) for b, h, _ in workload.sample_rows(cfg, blk, 0, heads_per_stream, 1)})
        e = pair.commit(kc, vc, a, heads)
        worst_s = max(worst_s, e)
        assert e <= pair.tol, f"block {blk}: state error {e:.3e} > {pair.tol}"
    pair.layer.sync_status()
    return worst_o, worst_s


def test_tiny_full_schedule_fp32(oracle):
    """Configuration 1 in full: 4 blocks x 2 steps + commit, fp32 mode, every element."""
    cfg = workload.CONFIGS["tiny"]
    pair = Pair(oracle, cfg)
    o, s = run_schedule(pair, cfg.blocks, cfg.steps, full=True)
    print(f"tiny: worst output error {o:.2e}, worst state error {s:.2e}")


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("D,L", [(64, 1), (64, 24), (128, 127), (128, 129), (64, 200), (128, 333), (64, 1100)])
def test_ragged_shapes(oracle, dtype, D, L):
    """Edge sizes: a single token, tails shorter and longer than a tile, several tiles."""
    cfg = workload.custom(B=2, H=3, D=D, L=L, dtype=dtype, cfg_id=11)
    pair = Pair(oracle, cfg)
    run_schedule(pair, 2, 2, full=True)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_no_maps_no_rope(oracle, dtype):
    """NULL feature maps (identity) and NULL tables (no rotation)."""
    cfg = workload.custom(B=1, H=2, D=64, L=150, dtype=dtype, cfg_id=12)
    for rope, maps in ((False, False), (True, False), (False, True)):
        pair = Pair(oracle, cfg, rope=rope, maps=maps)
        run_schedule(pair, 2, 1, full=True)


def test_custom_scale_and_eps(oracle):
    cfg = workload.custom(B=1, H=2, D=64, L=100, dtype="fp32", cfg_id=13)
    pair = Pair(oracle, cfg, eps=1e-3, scale=0.05)
    run_schedule(pair, 2, 2, full=True)


def test_small_config_bf16(oracle):
    """Configuration 2 (one 30x52 frame, H=12, D=128): two blocks in full, then sampled."""
    cfg = workload.CONFIGS["small"]
    pair = Pair(oracle, cfg)
    o, s = run_schedule(pair, 2, 2, full=True)
    print(f"small: worst output error {o:.2e}, worst state error {s:.2e}")


def test_step_never_writes_state(oracle):
    """Clean-pass-only update: S is bitwise unchanged by any number of denoise calls."""
    cfg = workload.custom(B=2, H=2, D=128, L=300, dtype="bf16", cfg_id=14)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    pair.commit(kc, vc, a)
    before = pair.layer.get_state().numpy().tobytes()
    ws_state = pair.layer.state.clone()
    for n in range(7):
        q, k, v, g = workload.step_inputs(cfg, 1, n)
        pair.step_gpu(q, k, v, g)
    assert pair.layer.get_state().numpy().tobytes() == before
    assert torch.equal(ws_state, pair.layer.state)


def test_first_block_is_pure_attention(oracle):
    """S = 0 (Algorithm 1, first line): the output does not depend on the gate."""
    cfg = workload.custom(B=1, H=2, D=64, L=130, dtype="fp32", cfg_id=15)
    pair = Pair(oracle, cfg)
    q, k, v, g = workload.step_inputs(cfg, 0, 0)
    a = pair.step_gpu(q, k, v, g)
    b = pair.step_gpu(q, k, v, g + 5.0)
    assert np.array_equal(a, b)


def test_commit_is_bitwise_reproducible(oracle):
    cfg = workload.custom(B=1, H=2, D=128, L=1100, dtype="bf16", cfg_id=16)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    states = []
    for _ in range(2):
        pair = Pair(oracle, cfg)
        for _ in range(2):
            pair.layer.commit(kc.cuda(), vc.cuda(), a.cuda())
        states.append(pair.layer.get_state().numpy().tobytes())
    assert states[0] == states[1]


def test_reset_one_stream_and_state_roundtrip(oracle):
    cfg = workload.custom(B=3, H=2, D=64, L=90, dtype="fp32", cfg_id=17)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    pair.commit(kc, vc, a)
    pair.reset(1)
    got = pair.layer.get_state().numpy()
    assert (got[1] == 0).all() and (got[0] != 0).any() and (got[2] != 0).any()
    kc, vc, a = workload.commit_inputs(cfg, 1)
    assert pair.commit(kc, vc, a) <= pair.tol
    # checkpoint / resume
    saved = pair.layer.get_state()
    pair.layer.reset()
    assert (pair.layer.get_state().numpy() == 0).all()
    pair.layer.set_state(saved)
    assert torch.equal(pair.layer.get_state(), saved)
    q, k, v, g = workload.step_inputs(cfg, 2, 0)
    assert pair.step_full(q, k, v, g) <= pair.tol


def test_token_order_equivariance_on_gpu(oracle):
    """Frame-level access (Eq. 8): permuting the block's tokens permutes the outputs."""
    cfg = workload.custom(B=1, H=2, D=64, L=160, dtype="fp32", cfg_id=18)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    pair.commit(kc, vc, a)
    q, k, v, g = workload.step_inputs(cfg, 1, 0)
    base = pair.step_gpu(q, k, v, g)
    perm = torch.randperm(cfg.L, generator=torch.Generator().manual_seed(5))
    pair.layer.set_params(pair.wq.cuda(), pair.wk.cuda(), pair.wv.cuda(),
                          pair.cos[perm].contiguous().cuda(), pair.sin[perm].contiguous().cuda())
    got = pair.step_gpu(q[:, perm].contiguous(), k[:, perm].contiguous(),
                        v[:, perm].contiguous(), g[:, perm].contiguous())
    err = head_errors(got, base[:, perm.numpy()].astype(np.float64)).max()
    assert err <= 1e-5


def test_argument_errors_leave_state_untouched(oracle):
    from paper_2605_16579_b200 import arl2

    cfg = workload.custom(B=1, H=2, D=64, L=64, dtype="fp32", cfg_id=19)
    pair = Pair(oracle, cfg)
    kc, vc, a = workload.commit_inputs(cfg, 0)
    pair.commit(kc, vc, a)
    before = pair.layer.get_state().numpy().tobytes()
    lib = arl2.load()
    assert lib.arl2_commit(pair.layer._ctx, None, None, None, None) == -1
    assert lib.arl2_denoise_step(pair.layer._ctx, None, None, None, None, None, None) == -1
    assert lib.arl2_reset(pair.layer._ctx, 7, None) == -1
    with pytest.raises(arl2.Arl2Error):
        pair.layer.commit(kc.cuda()[:, :32].contiguous(), vc.cuda(), a.cuda())
    assert pair.layer.get_state().numpy().tobytes() == before
    # too small a workspace is refused
    c = arl2.make_config(1, 2, 64, 64, "fp32")
    import ctypes
    buf = torch.empty(1024, dtype=torch.uint8, device="cuda")
    st = torch.empty(1, 2, 64, 64, device="cuda")
    ctx = ctypes.c_void_p()
    assert lib.arl2_create(ctypes.byref(c), st.data_ptr(), buf.data_ptr(), 1024, None,
                           ctypes.byref(ctx)) == -5


@pytest.mark.parametrize("name", ["chunked", "batched", "long"])
def test_full_size_configs_sampled(oracle, name):
    """Configurations 3-5 at full size, in the launch configuration the bench times: sampled
    rows of sampled heads per step (every row of the ragged tail tile included) and the whole
    state of those heads after every commit."""
    cfg = workload.CONFIGS[name]
    pair = Pair(oracle, cfg)
    o, s = run_schedule(pair, 2, 2, full=False, heads_per_stream=2, rows_per_head=32)
    if name == "batched":  # per-stream reset in the middle of a run
        pair.reset(3)
        o2, s2 = run_schedule(pair, 1, 1, full=False, heads_per_stream=2, rows_per_head=16)
        o, s = max(o, o2), max(s, s2)
    print(f"{name}: worst sampled output error {o:.2e}, worst state error {s:.2e}")


@pytest.mark.parametrize("B,H,L", [(1, 1, 100), (1, 3, 333), (3, 1, 200), (1, 5, 640)])
def test_odd_unit_counts_bf16(oracle, B, H, L):
    """The tensor-core step kernel packs the ragged last tiles of two (stream, head) units into
    one work item: odd numbers of units leave one of them alone, and L a multiple of the tile
    leaves none."""
    cfg = workload.custom(B=B, H=H, D=128, L=L, dtype="bf16", cfg_id=23)
    pair = Pair(oracle, cfg)
    run_schedule(pair, 2, 2, full=True)
