"""The fused clean pass (Algorithm 1, clean-pass branch): one call returns the layer's output against
the pre-update state and commits the block, with K_c read and rotated once.  Checked against the
oracle (output and state) and, bit for bit, against the two separate calls on a twin context."""
import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import workload
from parity_util import Pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,D,B,H,L", [
    ("fp32", 64, 1, 2, 200),       # plain-FMA kernels
    ("bf16", 64, 2, 2, 333),       # plain-FMA kernels, bf16 I/O
    ("bf16", 128, 1, 1, 1),        # a single token
    ("bf16", 128, 1, 2, 128),      # exactly one tile
    ("bf16", 128, 2, 3, 333),      # ragged tail, several streams
    ("bf16", 128, 1, 3, 1100),     # runs of tiles that cross heads
    ("bf16", 128, 3, 5, 700),      # odd number of units
])
def test_clean_pass_matches_oracle(oracle, dtype, D, B, H, L):
    cfg = workload.custom(B=B, H=H, D=D, L=L, dtype=dtype, cfg_id=51)
    pair = Pair(oracle, cfg)
    for blk in range(3):
        q, k, v, g = workload.step_inputs(cfg, blk, 0)
        assert pair.step_full(q, k, v, g) <= pair.tol                  # a denoise pass ...
        kc, vc, a = workload.commit_inputs(cfg, blk)
        e_out, e_state = pair.clean_pass(q, kc, vc, g, a)              # ... then the clean pass
        assert e_out <= pair.tol, f"block {blk}: output error {e_out:.3e} > {pair.tol}"
        assert e_state <= pair.tol, f"block {blk}: state error {e_state:.3e} > {pair.tol}"
    pair.layer.sync_status()


@pytest.mark.parametrize("rope,maps", [(True, True), (False, True), (True, False), (False, False)])
def test_clean_pass_equals_the_two_calls_bitwise(oracle, rope, maps):
    cfg = workload.custom(B=2, H=3, D=128, L=700, dtype="bf16", cfg_id=52)
    fused, split = Pair(oracle, cfg, rope=rope, maps=maps), Pair(oracle, cfg, rope=rope, maps=maps)
    d = fused.dev
    for blk in range(3):
        q, _, _, g = (t.to(d) for t in workload.step_inputs(cfg, blk, 0))
        kc, vc, a = (t.to(d) for t in workload.commit_inputs(cfg, blk))
        o1 = fused.layer.clean_pass(q, kc, vc, g, a)
        o2 = split.layer.denoise_step(q, kc, vc, g)
        split.layer.commit(kc, vc, a)
        assert torch.equal(o1, o2), f"block {blk}: outputs differ"
        assert torch.equal(fused.layer.get_state(), split.layer.get_state()), f"block {blk}: states differ"
    fused.layer.sync_status()


def test_clean_pass_full_size_sampled(oracle):
    """The bench's largest configuration: sampled rows of three heads, their state after each pass."""
    cfg = workload.CONFIGS["long"]
    units = workload.sample_units(cfg, heads_per_stream=3)
    pair = Pair(oracle, cfg, units=units)
    for blk in range(3):
        q, _, _, g = workload.step_inputs(cfg, blk, 0)
        kc, vc, a = workload.commit_inputs(cfg, blk)
        rows = workload.sample_rows(cfg, blk, 0, rows_per_head=24, units=units)
        e_out, e_state = pair.clean_pass(q, kc, vc, g, a, rows=rows)
        assert e_out <= pair.tol and e_state <= pair.tol, (blk, e_out, e_state)
    pair.layer.sync_status()


def test_clean_pass_argument_errors(oracle):
    from paper_2605_16579_b200 import arl2

    cfg = workload.custom(B=1, H=2, D=128, L=130, dtype="bf16", cfg_id=53)
    pair = Pair(oracle, cfg)
    lib = arl2.load()
    before = pair.layer.get_state().numpy().tobytes()
    assert lib.arl2_clean_pass(None, None, None, None, None, None, None, None) == -1
    assert lib.arl2_clean_pass(pair.layer._ctx, None, None, None, None, None, None, None) == -1
    q = torch.zeros(1, 130, 2, 128, dtype=torch.bfloat16, device=pair.dev)
    g = torch.zeros(1, 130, 2, device=pair.dev)
    a = torch.zeros(1, 2, device=pair.dev)
    # out aliasing an input
    assert lib.arl2_clean_pass(pair.layer._ctx, q.data_ptr(), q.data_ptr(), q.data_ptr(), g.data_ptr(),
                               a.data_ptr(), q.data_ptr(), None) == -1
    assert pair.layer.get_state().numpy().tobytes() == before
