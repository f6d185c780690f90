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


CLOSED = -40.0   # combine-gate logit of a pass that compares the softmax branch alone


def run_schedule(pair, blocks, steps, closed_gate_blocks=()):
    """Every element of every pass and the whole state after every commit.  In the blocks listed in
    closed_gate_blocks one more pass runs with the gate closed (the softmax branch on its own)."""
    cfg = pair.cfg
    worst_o, worst_s, worst_c = 0.0, 0.0, 0.0
    for blk in range(blocks):
        for st in range(steps):
            q, k, v, g = workload.step_inputs(cfg, blk, st)
            e = pair.step_full(q, k, v, g)
            worst_o = max(worst_o, e)
            assert e <= pair.tol, f"block {blk} step {st}: output error {e:.3e} > {pair.tol}"
            if blk in closed_gate_blocks and st == steps - 1:
                e = pair.step_full(q, k, v, torch.full_like(g, CLOSED))
                worst_c = max(worst_c, e)
                assert e <= pair.tol, f"block {blk}: closed-gate output error {e:.3e} > {pair.tol}"
        kc, vc, a = workload.commit_inputs(cfg, blk)
        e = pair.commit(kc, vc, a)
        worst_s = max(worst_s, e)
        assert e <= pair.tol, f"block {blk}: state error {e:.3e} > {pair.tol}"
    pair.layer.sync_status()
    return worst_o, worst_s, worst_c


def run_horizon(pair, check_blocks, rows_per_head=32, reset_at=None):
    """A configuration's whole schedule at full size.  The oracle follows the pair's units from the
    first block to the last: their state is compared after EVERY commit; in check_blocks every pass
    runs on fresh seeded inputs and is compared on sampled rows of those units (the ragged tail tile
    in full), plus one pass with the gate closed; in the other blocks the passes run on a ring of
    resident inputs (they cannot change the state, which a bitwise check confirms).
    reset_at = (block, stream): that stream starts a new video there."""
    cfg, d = pair.cfg, pair.dev
    units = pair.units
    ring = [tuple(t.to(d) for t in workload.step_inputs(cfg, 0, s)) for s in range(2)]
    out = torch.empty(cfg.B, cfg.L, cfg.H, cfg.D, dtype=cfg.torch_dtype, device=d)
    worst_o, worst_s, worst_c = 0.0, 0.0, 0.0
    for blk in range(cfg.blocks):
        if reset_at is not None and blk == reset_at[0]:
            pair.reset(reset_at[1])
        if blk in check_blocks:
            for st in range(cfg.steps):
                q, k, v, g = workload.step_inputs(cfg, blk, st)
                rows = workload.sample_rows(cfg, blk, st, rows_per_head=rows_per_head, units=units)
                e = pair.step_sampled(q, k, v, g, rows)
                worst_o = max(worst_o, e)
                assert e <= pair.tol, f"block {blk} step {st}: output error {e:.3e} > {pair.tol}"
            e = pair.step_sampled(q, k, v, torch.full_like(g, CLOSED), rows)
            worst_c = max(worst_c, e)
            assert e <= pair.tol, f"block {blk}: closed-gate output error {e:.3e} > {pair.tol}"
        else:
            before = pair.layer.state.clone() if blk % 16 == 5 else None
            for st in range(cfg.steps):
                pair.layer.denoise_step(*ring[st % 2], out=out)
            if before is not None:
                assert torch.equal(before, pair.layer.state), "a denoise pass changed the state"
        kc, vc, a = workload.commit_inputs(cfg, blk)
        e = pair.commit(kc, vc, a)
        worst_s = max(worst_s, e)
        assert e <= pair.tol, f"block {blk}: state error {e:.3e} > {pair.tol}"
    pair.layer.sync_status()
    return worst_o, worst_s, worst_c


def test_tiny_full_schedule_fp32(oracle):
    """Configuration 1 in full: 4 blocks x 2 steps + commit, fp32 mode, every element."""
    cfg = workload.CONFIGS["tiny"]
    pair = Pair(oracle, cfg)
    o, s, c = run_schedule(pair, cfg.blocks, cfg.steps, closed_gate_blocks=(2,))
    print(f"tiny: worst output error {o:.2e}, closed gate {c:.2e}, worst state error {s:.2e}")


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("D,L", [(64, 1), (64, 24), (128, 127), (128, 129), (64, 200), (128, 333), (64, 1100)])
def test_ragged_shapes(oracle, dtype, D, L):
    """Edge sizes: a single token, tails shorter and longer than a tile, several tiles."""
    cfg = workload.custom(B=2, H=3, D=D, L=L, dtype=dtype, cfg_id=11)
    pair = Pair(oracle, cfg)
    run_schedule(pair, 2, 2, closed_gate_blocks=(1,))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_no_maps_no_rope(oracle, dtype):
    """NULL feature maps (identity) and NULL tables (no rotation)."""
    cfg = workload.custom(B=1, H=2, D=64, L=150, dtype=dtype, cfg_id=12)
    for rope, maps in ((False, False), (True, False), (False, True)):
        pair = Pair(oracle, cfg, rope=rope, maps=maps)
        run_schedule(pair, 2, 1)


def test_custom_scale_and_eps(oracle):
    cfg = workload.custom(B=1, H=2, D=64, L=100, dtype="fp32", cfg_id=13)
    pair = Pair(oracle, cfg, eps=1e-3, scale=0.05)
    run_schedule(pair, 2, 2, closed_gate_blocks=(1,))


def test_small_config_bf16(oracle):
    """Configuration 2 (one 30x52 frame, H=12, D=128) in full: 8 blocks x 4 steps + commit, every
    element of every pass and of the state after every commit."""
    cfg = workload.CONFIGS["small"]
    pair = Pair(oracle, cfg)
    o, s, c = run_schedule(pair, cfg.blocks, cfg.steps, closed_gate_blocks=(1, cfg.blocks - 1))
    print(f"small: worst output error {o:.2e}, closed gate {c:.2e}, worst state error {s:.2e}")


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
def test_full_size_configs_whole_horizon(oracle, name):
    """Configurations 3-5 at full size, in the launch configuration the bench times, over their whole
    schedules (16 / 32 / 120 blocks x 4 steps + commit).  The oracle follows three (stream, head)
    units per stream (head 0, the last head, one drawn from the middle of the grid): their state is
    compared after every commit, their outputs on sampled rows (every row of the ragged tail tile
    included) in the first, second, a middle and the last block.  On `batched`, stream 3 starts a new
    video at block 16."""
    cfg = workload.CONFIGS[name]
    units = workload.sample_units(cfg, heads_per_stream=3)
    assert any(0 < h < cfg.H - 1 for _, h in units)
    pair = Pair(oracle, cfg, units=units)
    check = (0, 1, cfg.blocks // 2, cfg.blocks - 1)
    o, s, c = run_horizon(pair, check, rows_per_head=24 if name == "batched" else 32,
                          reset_at=(16, 3) if name == "batched" else None)
    print(f"{name}: {cfg.blocks} blocks, {len(units)} units followed; worst sampled output error {o:.2e}, "
          f"closed gate {c:.2e}, worst state error {s:.2e}")


@pytest.mark.parametrize("B,H,L", [(1, 1, 100), (1, 3, 333), (3, 1, 200), (1, 5, 640)])
def test_odd_unit_counts_bf16(oracle, B, H, L):
    """The tensor-core step kernel packs the ragged last tiles of two (stream, head) units into
    one work item: odd numbers of units leave one of them alone, and L a multiple of the tile
    leaves none."""
    cfg = workload.custom(B=B, H=H, D=128, L=L, dtype="bf16", cfg_id=23)
    pair = Pair(oracle, cfg)
    run_schedule(pair, 2, 2, closed_gate_blocks=(1,))


@pytest.mark.parametrize("B,H,L", [(1, 3, 1100), (1, 2, 1700), (2, 2, 2100), (1, 1, 2048)])
def test_key_range_split_bf16(oracle, B, H, L):
    """With fewer work items in its last wave than half the SMs, the tensor-core step kernel cuts
    those items into 2 to 4 ranges of key tiles and merges the parts' rows: every element against
    the oracle (pair items and ragged items, 9 to 17 key tiles), and the same call twice must give
    the same bits (the merge runs in part order whoever finishes last)."""
    cfg = workload.custom(B=B, H=H, D=128, L=L, dtype="bf16", cfg_id=29)
    pair = Pair(oracle, cfg)
    run_schedule(pair, 2, 2, closed_gate_blocks=(1,))
    d = pair.dev
    q, k, v, g = (t.to(d) for t in workload.step_inputs(cfg, 1, 0))
    outs = []
    for _ in range(3):
        out = torch.full((cfg.B, cfg.L, cfg.H, cfg.D), float("nan"), dtype=cfg.torch_dtype, device=d)
        pair.layer.denoise_step(q, k, v, g, out=out)
        outs.append(out)
    pair.layer.sync_status()
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
    assert torch.equal(outs[0].view(torch.int16), outs[2].view(torch.int16))
