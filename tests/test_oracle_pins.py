"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each pin is chosen so that a plausible
mistake in the oracle (a dropped term, a wrong sign or index, a transposed operand)
fails at least one of them: brute force with independent code on tiny inputs, closed
forms, invariants, and special cases that reduce to a library routine.
"""
import cmath
import math

import numpy as np
import pytest
import torch

from paper_2605_16579_b200 import workload

RNG = np.random.default_rng(20260516)


def rnd(*shape, scale=1.0):
    return RNG.standard_normal(shape) * scale


def rope_np(x, cos, sin):
    """Adjacent pairs rotated as a complex product, via torch's complex view (library)."""
    t = torch.from_numpy(np.ascontiguousarray(x)).double()
    B, L, H, D = t.shape
    z = torch.view_as_complex(t.reshape(B, L, H, D // 2, 2).contiguous())
    rot = torch.complex(torch.from_numpy(cos).double(), torch.from_numpy(sin).double())
    z = z * rot.view(1, L, 1, D // 2)
    return torch.view_as_real(z).reshape(B, L, H, D).numpy()


def tables(L, D):
    """Exact float64 cos/sin of 1-D positions (so that cos^2 + sin^2 = 1 to rounding)."""
    ang = np.arange(L)[:, None] * (10000.0 ** (-2.0 * np.arange(D // 2) / D))[None, :]
    return np.cos(ang), np.sin(ang)


# ----------------------------------------------------------------------------------------
# A1: intra-block softmax (Eq. 2)
# ----------------------------------------------------------------------------------------

def brute_force_layer(q, k, v, g, S, wq, cos, sin, scale, eps):
    """Pure-Python restatement with independent structure: complex numbers for the
    rotation, naive exp(s)/sum exp(s) without max subtraction, list arithmetic."""
    B, L, H, D = q.shape
    out = np.zeros_like(q)

    def rot(vec, pos):
        res = []
        for m in range(D // 2):
            z = complex(vec[2 * m], vec[2 * m + 1]) * complex(cos[pos][m], sin[pos][m])
            res += [z.real, z.imag]
        return res

    for b in range(B):
        for h in range(H):
            kr = [rot(list(k[b, j, h]), j) for j in range(L)]
            for i in range(L):
                qr = rot(list(q[b, i, h]), i)
                e = [math.exp(scale * sum(x * y for x, y in zip(qr, kr[j]))) for j in range(L)]
                z = sum(e)
                o = [sum(e[j] / z * v[b, j, h, d] for j in range(L)) for d in range(D)]
                u = [sum(q[b, i, h, a] * wq[h, a, c] for a in range(D)) for c in range(D)]
                u = rot(u, i)
                n = math.sqrt(sum(x * x for x in u) + eps)
                u = [x / n for x in u]
                gate = 1.0 / (1.0 + math.exp(-g[b, i, h]))
                for c in range(D):
                    o[c] += gate * sum(u[a] * S[b, h, a, c] for a in range(D))
                out[b, i, h] = o
    return out


@pytest.mark.parametrize("L,D", [(1, 2), (5, 4), (8, 4)])
def test_step_brute_force_tiny(oracle, L, D):
    B, H = 2, 2
    q, k, v = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D)
    g, S, wq = rnd(B, L, H), rnd(B, H, D, D), rnd(H, D, D)
    ang = rnd(L, D // 2)
    cos, sin = np.cos(ang), np.sin(ang)
    ref = brute_force_layer(q, k, v, g, S, wq, cos, sin, 0.37, 1e-6)
    got = oracle.step(q, k, v, g, S, wq, cos, sin, scale=0.37, eps=1e-6)
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-12)


def test_softmax_matches_library_attention(oracle):
    """S = 0, no rotation: the layer is textbook attention (first block, Algorithm 1)."""
    B, L, H, D = 2, 37, 3, 16
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    S = np.zeros((B, H, D, D))
    got = oracle.step(q, k, v, g, S, rnd(H, D, D))
    tq, tk, tv = (torch.from_numpy(x).permute(0, 2, 1, 3) for x in (q, k, v))
    ref = torch.softmax(tq @ tk.transpose(-1, -2) / math.sqrt(D), dim=-1) @ tv
    np.testing.assert_allclose(got, ref.permute(0, 2, 1, 3).numpy(), rtol=1e-11, atol=1e-13)


def test_softmax_with_rope_matches_library(oracle):
    B, L, H, D = 1, 29, 2, 8
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    cos, sin = tables(L, D)
    got = oracle.step(q, k, v, g, np.zeros((B, H, D, D)), None, cos, sin)
    tq, tk = (torch.from_numpy(rope_np(x, cos, sin)).permute(0, 2, 1, 3) for x in (q, k))
    tv = torch.from_numpy(v).permute(0, 2, 1, 3)
    ref = torch.softmax(tq @ tk.transpose(-1, -2) / math.sqrt(D), dim=-1) @ tv
    np.testing.assert_allclose(got, ref.permute(0, 2, 1, 3).numpy(), rtol=1e-11, atol=1e-13)


def test_zero_query_gives_column_mean(oracle):
    B, L, H, D = 1, 23, 2, 8
    k, v = rnd(B, L, H, D), rnd(B, L, H, D)
    cos, sin = tables(L, D)
    got = oracle.step(np.zeros((B, L, H, D)), k, v, rnd(B, L, H), np.zeros((B, H, D, D)),
                      None, cos, sin, eps=1e-6)
    ref = np.broadcast_to(v.mean(axis=1, keepdims=True), v.shape)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_key_shift_invariance(oracle):
    B, L, H, D = 1, 19, 2, 8
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    S = np.zeros((B, H, D, D))
    c = rnd(1, 1, H, D)
    a = oracle.step(q, k, v, g, S)
    b = oracle.step(q, k + c, v, g, S)
    np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)


def test_large_scores_do_not_overflow(oracle):
    """Max subtraction: scores of +-800 would overflow a naive exp."""
    B, L, H, D = 1, 6, 1, 4
    q = rnd(B, L, H, D) * 40
    k = rnd(B, L, H, D) * 40
    v = rnd(B, L, H, D)
    out = oracle.step(q, k, v, rnd(B, L, H), np.zeros((B, H, D, D)), scale=1.0)
    assert np.isfinite(out).all()
    assert (out.min(axis=1) >= v.min(axis=1) - 1e-12).all()
    assert (out.max(axis=1) <= v.max(axis=1) + 1e-12).all()


# ----------------------------------------------------------------------------------------
# A2: feature maps (Eq. 3)
# ----------------------------------------------------------------------------------------

def test_feature_map_against_library_ops(oracle):
    B, L, H, D = 2, 11, 3, 8
    x, W = rnd(B, L, H, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    got = oracle.feature(x, W, cos, sin, 1e-6, 0)
    u = torch.einsum("blhi,hio->blho", torch.from_numpy(x), torch.from_numpy(W)).numpy()
    u = rope_np(u, cos, sin)
    ref = u / np.sqrt((u * u).sum(-1, keepdims=True) + 1e-6)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)
    got_v = oracle.feature(x, W, cos, sin, 1e-6, 1)
    ref_v = torch.einsum("blhi,hio->blho", torch.from_numpy(x), torch.from_numpy(W)).numpy()
    np.testing.assert_allclose(got_v, ref_v, rtol=1e-12, atol=1e-14)


def test_feature_unit_norm_and_commutation(oracle):
    B, L, H, D = 1, 13, 2, 16
    x, W = rnd(B, L, H, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    y = oracle.feature(x, W, cos, sin, 0.0, 0)
    np.testing.assert_allclose((y * y).sum(-1), 1.0, rtol=1e-12)
    # rotation preserves the norm, so normalising before or after it is the same
    y_nr = oracle.feature(x, W, None, None, 0.0, 0)
    np.testing.assert_allclose(rope_np(y_nr, cos, sin), y, rtol=1e-12, atol=1e-14)
    # identity map, no rotation: Q' = Q / |Q|
    y_id = oracle.feature(x, None, None, None, 0.0, 0)
    np.testing.assert_allclose(y_id, x / np.linalg.norm(x, axis=-1, keepdims=True), rtol=1e-12)
    # identity tables (angle 0) are a no-op
    y_0 = oracle.feature(x, W, np.ones((L, D // 2)), np.zeros((L, D // 2)), 0.0, 0)
    np.testing.assert_allclose(y_0, y_nr, rtol=1e-13)


def test_rope_quarter_turn(oracle):
    """A rotation by 90 degrees sends (x0, x1) to (-x1, x0): fixes the sign convention."""
    B, L, H, D = 1, 2, 1, 4
    x = rnd(B, L, H, D)
    y = oracle.feature(x, None, np.zeros((L, 2)), np.ones((L, 2)), 0.0, 0)
    n = np.linalg.norm(x, axis=-1, keepdims=True)
    ref = np.stack([-x[..., 1], x[..., 0], -x[..., 3], x[..., 2]], axis=-1) / n
    np.testing.assert_allclose(y, ref, rtol=1e-13)


# ----------------------------------------------------------------------------------------
# A3 / A4: frame-level readout and the gated combination (Eq. 5-8)
# ----------------------------------------------------------------------------------------

def test_zero_values_isolate_inter_branch(oracle):
    B, L, H, D = 2, 9, 2, 8
    q, k, g, S, wq = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H), rnd(B, H, D, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    got = oracle.step(q, k, np.zeros((B, L, H, D)), g, S, wq, cos, sin)
    qf = oracle.feature(q, wq, cos, sin, 1e-6, 0)
    ref = torch.einsum("blhd,bhde->blhe", torch.from_numpy(qf), torch.from_numpy(S)).numpy()
    ref = ref / (1.0 + np.exp(-g))[..., None]
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-13)
    # positive rescaling of Q leaves Q' (eps = 0) and hence the readout unchanged
    a = oracle.step(q, k, np.zeros((B, L, H, D)), g, S, wq, cos, sin, eps=0.0)
    b = oracle.step(3.7 * q, k, np.zeros((B, L, H, D)), g, S, wq, cos, sin, eps=0.0)
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-13)


def test_closed_gate_and_linearity_in_state(oracle):
    B, L, H, D = 1, 10, 2, 8
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    S1, S2, wq = rnd(B, H, D, D), rnd(B, H, D, D), rnd(H, D, D)
    zero = np.zeros_like(S1)
    intra = oracle.step(q, k, v, g, zero, wq)
    shut = oracle.step(q, k, v, np.full_like(g, -800.0), S1, wq)
    np.testing.assert_allclose(shut, intra, rtol=1e-13, atol=1e-15)
    o1 = oracle.step(q, k, v, g, S1, wq) - intra
    o2 = oracle.step(q, k, v, g, S2, wq) - intra
    o12 = oracle.step(q, k, v, g, 2.0 * S1 - 0.5 * S2, wq) - intra
    np.testing.assert_allclose(o12, 2.0 * o1 - 0.5 * o2, rtol=1e-9, atol=1e-12)


def test_token_order_equivariance(oracle):
    """All tokens read the same pre-update state (Eq. 8): permuting the block's tokens
    permutes the outputs and leaves the committed state unchanged."""
    B, L, H, D = 2, 21, 2, 8
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    S, a = rnd(B, H, D, D), rnd(B, H)
    wq, wk, wv = rnd(H, D, D), rnd(H, D, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    perm = RNG.permutation(L)
    o = oracle.step(q, k, v, g, S, wq, cos, sin)
    op = oracle.step(q[:, perm], k[:, perm], v[:, perm], g[:, perm], S, wq, cos[perm], sin[perm])
    np.testing.assert_allclose(op, o[:, perm], rtol=1e-10, atol=1e-12)
    s = oracle.commit(k, v, a, S, wk, wv, cos, sin)
    sp = oracle.commit(k[:, perm], v[:, perm], a, S, wk, wv, cos[perm], sin[perm])
    np.testing.assert_allclose(sp, s, rtol=1e-12, atol=1e-12)


def test_step_never_writes_state(oracle):
    B, L, H, D = 1, 12, 2, 8
    S = rnd(B, H, D, D)
    keep = S.copy()
    for n in range(7):
        oracle.step(rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H), S,
                    rnd(H, D, D))
        assert S.tobytes() == keep.tobytes()


# ----------------------------------------------------------------------------------------
# A6 / A7: commit and reset
# ----------------------------------------------------------------------------------------

def test_commit_against_library_ops(oracle):
    B, L, H, D = 2, 17, 3, 8
    kc, vc, a, S = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, H), rnd(B, H, D, D)
    wk, wv = rnd(H, D, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    got = oracle.commit(kc, vc, a, S, wk, wv, cos, sin)
    kf = torch.from_numpy(oracle.feature(kc, wk, cos, sin, 1e-6, 0))
    vf = torch.from_numpy(oracle.feature(vc, wv, cos, sin, 1e-6, 1))
    alpha = 1.0 / (1.0 + np.exp(-a))
    ref = alpha[..., None, None] * S + torch.einsum("blhd,blhe->bhde", kf, vf).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-13)
    # subset of heads: the others stay as they were
    part = oracle.commit(kc, vc, a, S, wk, wv, cos, sin, heads=[(1, 2), (0, 0)])
    np.testing.assert_allclose(part[1, 2], ref[1, 2], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(part[0, 0], ref[0, 0], rtol=1e-11, atol=1e-13)
    assert part[0, 1].tobytes() == S[0, 1].tobytes()


def test_commit_closed_form_over_blocks(oracle):
    """S_T = (prod alpha) S_0 + sum_t (prod_{s>t} alpha_s) K'_t^T V'_t."""
    B, L, H, D, T = 1, 9, 2, 8, 6
    wk, wv = rnd(H, D, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    S0 = rnd(B, H, D, D)
    ks, vs, as_ = [rnd(B, L, H, D) for _ in range(T)], [rnd(B, L, H, D) for _ in range(T)], \
        [rnd(B, H) + 2.0 for _ in range(T)]
    S = S0
    for t in range(T):
        S = oracle.commit(ks[t], vs[t], as_[t], S, wk, wv, cos, sin)
    alphas = [1.0 / (1.0 + np.exp(-x)) for x in as_]
    ref = np.prod(alphas, axis=0)[..., None, None] * S0
    for t in range(T):
        kf = torch.from_numpy(oracle.feature(ks[t], wk, cos, sin, 1e-6, 0))
        vf = torch.from_numpy(oracle.feature(vs[t], wv, cos, sin, 1e-6, 1))
        w = np.ones((B, H))
        for s in range(t + 1, T):
            w = w * alphas[s]
        ref = ref + w[..., None, None] * torch.einsum("blhd,blhe->bhde", kf, vf).numpy()
    np.testing.assert_allclose(S, ref, rtol=1e-11, atol=1e-12)


def orthonormal_keys(B, L, H, D):
    k = np.empty((B, L, H, D))
    for b in range(B):
        for h in range(H):
            qmat, _ = np.linalg.qr(rnd(D, D))
            k[b, :, h, :] = qmat[:, :L].T
    return k


@pytest.mark.parametrize("rule", [0, 1, 2])
def test_associative_memory(oracle, rule):
    """alpha = 1, orthonormal keys, empty state: reading with key j returns value j."""
    B, L, H, D = 1, 6, 2, 8
    k, v = orthonormal_keys(B, L, H, D), rnd(B, L, H, D)
    a = np.full((B, H), 800.0)                  # sigmoid -> exactly 1
    beta = np.full((B, L, H), 800.0)
    S = oracle.commit(k, v, a, np.zeros((B, H, D, D)), eps=0.0, rule=rule, beta_logit=beta)
    out = oracle.step(k, k, np.zeros_like(v), np.full((B, L, H), 800.0), S, eps=0.0)
    np.testing.assert_allclose(out, v, rtol=1e-10, atol=1e-12)


def test_delta_rules_overwrite_and_coincide(oracle):
    """Eq. 4 with orthonormal keys and alpha = beta = 1 replaces what the state held for
    those keys (K' S_new = V'), and the frame-level and token-sequential forms agree."""
    B, L, H, D = 1, 5, 2, 8
    k, v = orthonormal_keys(B, L, H, D), rnd(B, L, H, D)
    S0 = rnd(B, H, D, D)
    one, beta = np.full((B, H), 800.0), np.full((B, L, H), 800.0)
    s1 = oracle.commit(k, v, one, S0, eps=0.0, rule=1, beta_logit=beta)
    s2 = oracle.commit(k, v, one, S0, eps=0.0, rule=2, beta_logit=beta)
    np.testing.assert_allclose(s1, s2, rtol=1e-10, atol=1e-12)
    read = torch.einsum("blhd,bhde->blhe", torch.from_numpy(k), torch.from_numpy(s1)).numpy()
    np.testing.assert_allclose(read, v, rtol=1e-10, atol=1e-12)
    # with an empty state and beta = 1 the correction term vanishes at frame level
    a = rnd(B, H)
    kk, vv = rnd(B, L, H, D), rnd(B, L, H, D)
    r0 = oracle.commit(kk, vv, a, np.zeros_like(S0), rule=0)
    r1 = oracle.commit(kk, vv, a, np.zeros_like(S0), rule=1, beta_logit=beta)
    np.testing.assert_allclose(r0, r1, rtol=1e-12, atol=1e-14)
    # frame-level Eq. 4 against library ops, general keys, decay and learning rates
    a, bl = rnd(B, H), rnd(B, L, H)
    got = oracle.commit(kk, vv, a, S0, rule=1, beta_logit=bl)
    kf = torch.from_numpy(oracle.feature(kk, None, None, None, 1e-6, 0))
    tv, tS = torch.from_numpy(vv), torch.from_numpy(S0)
    resid = tv - torch.einsum("blhd,bhde->blhe", kf, tS)
    resid = resid * torch.from_numpy(1.0 / (1.0 + np.exp(-bl)))[..., None]
    ref = torch.from_numpy(1.0 / (1.0 + np.exp(-a)))[..., None, None] * tS \
        + torch.einsum("blhd,blhe->bhde", kf, resid)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-11, atol=1e-13)


def sig(x):
    return 1.0 / (1.0 + np.exp(-x))


def test_token_sequential_rule_decays_before_the_tokens(oracle):
    """Rule 2 (decay once, then Eq. 4 token by token) with orthonormal keys and GENERAL alpha and
    beta: the tokens do not interact, so S_new = alpha S_0 + sum_j beta_j K'_j^T (V'_j - alpha K'_j S_0),
    i.e. K'_j S_new = alpha (1 - beta_j) K'_j S_0 + beta_j V'_j and directions no key spans are only
    decayed.  A decay applied after the tokens, to the correction only, or not at all fails this."""
    B, L, H, D = 2, 5, 2, 8
    k, v = orthonormal_keys(B, L, H, D), rnd(B, L, H, D)
    S0 = rnd(B, H, D, D)
    a, bl = rnd(B, H), rnd(B, L, H)
    got = oracle.commit(k, v, a, S0, eps=0.0, rule=2, beta_logit=bl)
    alpha, beta = sig(a), sig(bl)
    tk, tv, tS = torch.from_numpy(k), torch.from_numpy(v), torch.from_numpy(S0)
    aS = torch.from_numpy(alpha)[..., None, None] * tS
    resid = (tv - torch.einsum("blhd,bhde->blhe", tk, aS)) * torch.from_numpy(beta)[..., None]
    ref = aS + torch.einsum("blhd,blhe->bhde", tk, resid)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-11, atol=1e-13)
    read = torch.einsum("blhd,bhde->blhe", tk, torch.from_numpy(got)).numpy()
    old = torch.einsum("blhd,bhde->blhe", tk, tS).numpy()
    np.testing.assert_allclose(read, alpha[:, None, :, None] * (1 - beta[..., None]) * old + beta[..., None] * v,
                               rtol=1e-10, atol=1e-12)
    assert not np.allclose(got, oracle.commit(k, v, np.full((B, H), 800.0), S0, eps=0.0, rule=2, beta_logit=bl))


def test_gate_granularities(oracle):
    """Scalar and elementwise combine gates: with the same logit repeated they are the headwise
    layer; an elementwise gate closed on some channels leaves exactly the intra branch there and
    the fully open layer elsewhere."""
    B, L, H, D = 2, 6, 3, 8
    q, k, v, S = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, H, D, D)
    cos, sin = tables(L, D)
    g_tok = rnd(B, L)
    head = oracle.step(q, k, v, np.repeat(g_tok[..., None], H, axis=2), S, None, cos, sin)
    np.testing.assert_allclose(oracle.step_gate_mode(q, k, v, g_tok, S, 1, None, cos, sin), head, rtol=1e-13)
    g_head = rnd(B, L, H)
    ref = oracle.step(q, k, v, g_head, S, None, cos, sin)
    elem = oracle.step_gate_mode(q, k, v, np.repeat(g_head[..., None], D, axis=3), S, 2, None, cos, sin)
    np.testing.assert_allclose(elem, ref, rtol=1e-13)
    np.testing.assert_allclose(oracle.step_gate_mode(q, k, v, g_head, S, 0, None, cos, sin), ref, rtol=0)
    closed = oracle.step(q, k, v, np.full((B, L, H), -800.0), S, None, cos, sin)
    opened = oracle.step(q, k, v, np.full((B, L, H), 800.0), S, None, cos, sin)
    mask = np.random.default_rng(5).random((B, L, H, D)) < 0.5
    mixed = oracle.step_gate_mode(q, k, v, np.where(mask, 800.0, -800.0), S, 2, None, cos, sin)
    np.testing.assert_allclose(mixed, np.where(mask, opened, closed), rtol=1e-13, atol=1e-15)


def test_cache_attention_against_library_and_the_layer(oracle):
    """Eq. 1 over a longer cache: the library's attention routine; with a cache of exactly the
    block and a closed gate it is the layer's intra branch without rotation; a cache of one token
    returns that token's value; explicit softmax weights with a custom scale."""
    B, L, Lk, H, D = 2, 5, 13, 2, 8
    q, k, v = rnd(B, L, H, D), rnd(B, Lk, H, D), rnd(B, Lk, H, D)
    got = oracle.attend_cache(q, k, v)
    tq, tk, tv = (torch.from_numpy(t).permute(0, 2, 1, 3) for t in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-12)
    same = oracle.step(q, k[:, :L], v[:, :L], np.full((B, L, H), -800.0), rnd(B, H, D, D))
    np.testing.assert_allclose(oracle.attend_cache(q, k[:, :L], v[:, :L]), same, rtol=1e-12, atol=1e-14)
    one = oracle.attend_cache(q, k[:, :1], v[:, :1])
    np.testing.assert_allclose(one, np.broadcast_to(v[:, :1], one.shape), rtol=1e-12)
    # explicit weights (einsum + exp) with an extra zero key and a custom scale
    far = np.concatenate([k, np.zeros_like(k[:, :1])], axis=1)
    v2 = np.concatenate([v, 1e3 * np.ones_like(v[:, :1])], axis=1)
    big = oracle.attend_cache(q, far, v2, scale=1.0)
    sc = np.einsum("blhd,bjhd->bhlj", q, far)
    w = np.exp(sc - sc.max(-1, keepdims=True))
    w /= w.sum(-1, keepdims=True)
    np.testing.assert_allclose(big, np.einsum("bhlj,bjhe->blhe", w, v2), rtol=1e-10, atol=1e-10)


@pytest.mark.parametrize("decayed", [False, True])
def test_token_gates_matrix_product_form(oracle, decayed):
    """Per-token Eq. 4 rewritten as S_j = (alpha_j I - beta_j k_j^T k_j) S_{j-1} + beta_j k_j^T v_j
    and evaluated with explicit D x D transition matrices (library matmul), with feature maps,
    rotation and normalisation taken from the library-pinned feature routine.  The other reading
    (prediction against the decayed state) has the transition alpha_j (I - beta_j k_j^T k_j)."""
    B, L, H, D = 2, 9, 2, 8
    k, v, S0 = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, H, D, D)
    al, bl = rnd(B, L, H) + 1.0, rnd(B, L, H)
    wk, wv = np.eye(D) + 0.1 * rnd(H, D, D), np.eye(D) + 0.1 * rnd(H, D, D)
    cos, sin = tables(L, D)
    got = oracle.commit_tokens(k, v, S0, al, bl, wk, wv, cos, sin, eps=1e-6, decayed_prediction=decayed)
    kf = oracle.feature(k, wk, cos, sin, 1e-6, 0)
    vf = oracle.feature(v, wv, None, None, 1e-6, 1)
    ref = S0.copy()
    for b in range(B):
        for h in range(H):
            S = torch.from_numpy(S0[b, h])
            for j in range(L):
                kk = torch.from_numpy(kf[b, j, h])[None, :]          # 1 x D
                vv = torch.from_numpy(vf[b, j, h])[None, :]
                eye = torch.eye(D, dtype=torch.float64)
                if decayed:
                    M = sig(al[b, j, h]) * (eye - sig(bl[b, j, h]) * (kk.T @ kk))
                else:
                    M = sig(al[b, j, h]) * eye - sig(bl[b, j, h]) * (kk.T @ kk)
                S = M @ S + sig(bl[b, j, h]) * (kk.T @ vv)
            ref[b, h] = S.numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-13)


def test_token_gates_orthonormal_keys_closed_form(oracle):
    """With orthonormal keys token j only rewrites row-space direction k_j: along it the state
    holds (prod_{m<j} alpha_m) k_j S_0 before token j, becomes (alpha_j - beta_j) of that plus
    beta_j v_j, and decays with the later alphas; the orthogonal complement only decays."""
    B, L, H, D = 1, 5, 2, 8
    k, v, S0 = orthonormal_keys(B, L, H, D), rnd(B, L, H, D), rnd(B, H, D, D)
    al, bl = rnd(B, L, H) + 1.0, rnd(B, L, H)
    got = oracle.commit_tokens(k, v, S0, al, bl, eps=0.0)
    a, bt = sig(al), sig(bl)
    for h in range(H):
        total = np.prod(a[0, :, h])
        proj = np.zeros((D, D))
        for j in range(L):
            kj = k[0, j, h]
            before = np.prod(a[0, :j, h]) * (kj @ S0[0, h])
            after_j = (a[0, j, h] - bt[0, j, h]) * before + bt[0, j, h] * v[0, j, h]
            read = np.prod(a[0, j + 1:, h]) * after_j
            np.testing.assert_allclose(kj @ got[0, h], read, rtol=1e-10, atol=1e-12)
            proj += np.outer(kj, kj)
        rest = (np.eye(D) - proj) @ got[0, h]
        np.testing.assert_allclose(rest, total * (np.eye(D) - proj) @ S0[0, h], rtol=1e-10, atol=1e-12)


def test_token_gates_special_cases(oracle):
    B, L, H, D = 1, 7, 2, 8
    k, v, S0 = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, H, D, D)
    al, bl = rnd(B, L, H) + 1.0, rnd(B, L, H)
    # no learning: only the decays act
    got = oracle.commit_tokens(k, v, S0, al, np.full((B, L, H), -800.0))
    np.testing.assert_allclose(got, np.prod(sig(al), axis=1)[..., None, None] * S0, rtol=1e-12)
    # alpha = 1 everywhere: the token-sequential rule with one block-level decay of 1 (rule 2)
    got = oracle.commit_tokens(k, v, S0, None, bl)
    ref = oracle.commit(k, v, np.full((B, H), 800.0), S0, rule=2, beta_logit=bl)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)
    # one token: Eq. 4 once, against library ops
    k1, v1 = k[:, :1], v[:, :1]
    got = oracle.commit_tokens(k1, v1, S0, al[:, :1], bl[:, :1])
    kf = oracle.feature(k1, None, None, None, 1e-6, 0)
    for h in range(H):
        kk, vv = kf[0, 0, h][None, :], v1[0, 0, h][None, :]
        ref = sig(al[0, 0, h]) * S0[0, h] + sig(bl[0, 0, h]) * kk.T @ (vv - kk @ S0[0, h])
        np.testing.assert_allclose(got[0, h], ref, rtol=1e-12, atol=1e-14)
    # heads subset leaves the others untouched
    got = oracle.commit_tokens(k, v, S0, al, bl, heads=[(0, 1)])
    np.testing.assert_array_equal(got[0, 0], S0[0, 0])
    assert not np.allclose(got[0, 1], S0[0, 1])


def test_per_token_decay_closed_form(oracle):
    """S <- alpha_j S + k_j^T v_j in order equals (prod alpha) S_0 + sum_j (prod_{i>j} alpha_i) k_j^T v_j
    (library cumulative products and einsum); with every gate open it is the block-level commit."""
    B, L, H, D = 2, 11, 2, 8
    k, v, S0 = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, H, D, D)
    al = rnd(B, L, H) + 1.0
    wk, wv = np.eye(D) + 0.1 * rnd(H, D, D), np.eye(D) + 0.1 * rnd(H, D, D)
    cos, sin = tables(L, D)
    got = oracle.commit_decay_tokens(k, v, S0, al, wk, wv, cos, sin)
    kf = torch.from_numpy(oracle.feature(k, wk, cos, sin, 1e-6, 0))
    vf = torch.from_numpy(oracle.feature(v, wv, None, None, 1e-6, 1))
    a = torch.from_numpy(sig(al))
    suffix = torch.flip(torch.cumprod(torch.flip(a, dims=[1]), dim=1), dims=[1])      # prod_{i>=j}
    w = suffix / a                                                                    # prod_{i>j}
    ref = suffix[:, 0][..., None, None] * torch.from_numpy(S0) \
        + torch.einsum("blhd,blhe->bhde", kf * w[..., None], vf)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-11, atol=1e-13)
    ones = oracle.commit_decay_tokens(k, v, S0, np.full((B, L, H), 800.0), wk, wv, cos, sin)
    block = oracle.commit(k, v, np.full((B, H), 800.0), S0, wk, wv, cos, sin)
    np.testing.assert_allclose(ones, block, rtol=1e-12, atol=1e-14)
    part = oracle.commit_decay_tokens(k, v, S0, al, heads=[(1, 0)])
    np.testing.assert_array_equal(part[0], S0[0])


def test_state_norm_stays_bounded(oracle):
    """Unit-norm keys and alpha <= alpha_max < 1: |S_T|_F <= max_t |K'^T V'|_F / (1 - alpha_max)."""
    B, L, H, D, T = 1, 12, 2, 8, 60
    S = np.zeros((B, H, D, D))
    amax = 1.0 / (1.0 + math.exp(-2.5))
    bound = 0.0
    norms = []
    for t in range(T):
        k, v = rnd(B, L, H, D), rnd(B, L, H, D)
        a = np.minimum(rnd(B, H) * 0.5 + 2.0, 2.5)
        delta = oracle.commit(k, v, np.full((B, H), -800.0), np.zeros_like(S))
        bound = max(bound, np.sqrt((delta ** 2).sum(axis=(-1, -2))).max())
        S = oracle.commit(k, v, a, S)
        norms.append(np.sqrt((S ** 2).sum(axis=(-1, -2))).max())
    assert max(norms) <= bound / (1.0 - amax)
    assert max(norms[T // 2:]) < 1.5 * max(norms[: T // 2])   # flat, not growing with T


def test_clean_pass_reads_the_state_before_it_commits(oracle):
    """The clean pass is the step on the pre-update state followed by the commit (Sec. 3.3, Eq. 8).
    Pinned through a case with a closed form: with V_c = 0 nothing is written (S_new = alpha S) and
    the output is sigmoid(g) Q' S_old, so alpha * out must equal what a step reads from S_new --
    an output that saw the new state would be off by the factor alpha."""
    B, L, H, D = 2, 7, 2, 8
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    a, S0 = rnd(B, H), rnd(B, H, D, D)
    wq, wk, wv = rnd(H, D, D), rnd(H, D, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    out, S1 = oracle.clean_pass(q, k, v, g, a, S0, wq, wk, wv, cos, sin)
    np.testing.assert_array_equal(out, oracle.step(q, k, v, g, S0, wq, cos, sin))
    np.testing.assert_array_equal(S1, oracle.commit(k, v, a, S0, wk, wv, cos, sin))
    assert not np.allclose(out, oracle.step(q, k, v, g, S1, wq, cos, sin))
    zero = np.zeros_like(v)
    out0, S1z = oracle.clean_pass(q, k, zero, g, a, S0, wq, wk, wv, cos, sin)
    alpha = sig(a)
    np.testing.assert_allclose(S1z, alpha[..., None, None] * S0, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(alpha[:, None, :, None] * out0, oracle.step(q, k, zero, g, S1z, wq, cos, sin),
                               rtol=1e-11, atol=1e-13)


def test_token_level_access_against_sequential_commits_and_library_ops(oracle):
    """Token-level state access (Sec. 4.3): token i reads the state advanced by the tokens before it.
    (a) brute force through functions pinned elsewhere: commit the tokens one at a time with the per-token
    gated-linear commit and read row i with the frame-level layer; (b) the causal linear-attention closed
    form with library ops: O_inter_i = (prod_{j<i} alpha_j) Q'_i S + sum_{j<i} (prod_{j<m<i} alpha_m) (Q'_i . K'_j) V'_j;
    (c) token 0 and one-token blocks coincide with the frame-level layer."""
    B, L, H, D = 2, 6, 2, 8
    q, k, v, g = rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H, D), rnd(B, L, H)
    al, S0 = rnd(B, L, H) + 1.0, rnd(B, H, D, D)
    wq, wk, wv = rnd(H, D, D), rnd(H, D, D), rnd(H, D, D)
    cos, sin = tables(L, D)
    got = oracle.step_token_level(q, k, v, g, S0, al, wq, wk, wv, cos, sin)
    # (a)
    ref = np.empty_like(got)
    S = S0.copy()
    for i in range(L):
        rows = np.array([(b, h, i) for b in range(B) for h in range(H)])
        ref[:, i] = oracle.step_rows(q, k, v, g, S, rows, wq, cos, sin).reshape(B, H, D)
        S = oracle.commit_decay_tokens(k[:, i:i + 1], v[:, i:i + 1], S, al[:, i:i + 1], wk, wv,
                                       cos[i:i + 1], sin[i:i + 1])
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-13)
    # (b): subtract the frame-level layer with the gate closed (the softmax branch alone)
    intra = oracle.step(q, k, v, np.full_like(g, -800.0), S0, wq, cos, sin)
    qf = torch.from_numpy(oracle.feature(q, wq, cos, sin, 1e-6, 0))
    kf = torch.from_numpy(oracle.feature(k, wk, cos, sin, 1e-6, 0))
    vf = torch.from_numpy(oracle.feature(v, wv, None, None, 1e-6, 1))
    alpha = torch.from_numpy(sig(al))
    incl = torch.cumprod(alpha, dim=1)                               # prod_{m<=i} alpha_m
    excl = incl / alpha                                              # prod_{m<i}
    decay = (excl[:, :, None, :] / incl[:, None, :, :])              # [b, i, j, h] = prod_{j<m<i} for j < i
    mask = torch.tril(torch.ones(L, L), diagonal=-1)[None, :, :, None]
    scores = torch.einsum("bihd,bjhd->bijh", qf, kf) * decay * mask
    inter = excl[..., None] * torch.einsum("bihd,bhde->bihe", qf, torch.from_numpy(S0)) \
        + torch.einsum("bijh,bjhe->bihe", scores, vf)
    ref_b = intra + sig(g)[..., None] * inter.numpy()
    np.testing.assert_allclose(got, ref_b, rtol=1e-10, atol=1e-12)
    # (c)
    frame = oracle.step(q, k, v, g, S0, wq, cos, sin)
    np.testing.assert_array_equal(got[:, 0], frame[:, 0])
    assert not np.allclose(got[:, 1:], frame[:, 1:])
    one = oracle.step_token_level(q[:, :1], k[:, :1], v[:, :1], g[:, :1], S0, al[:, :1], wq, wk, wv, cos[:1], sin[:1])
    np.testing.assert_array_equal(one, oracle.step(q[:, :1], k[:, :1], v[:, :1], g[:, :1], S0, wq, cos[:1], sin[:1]))
    # gates absent = all gates open; the caller's state is never written
    S_keep = S0.copy()
    np.testing.assert_allclose(oracle.step_token_level(q, k, v, g, S0, None, wq, wk, wv, cos, sin),
                               oracle.step_token_level(q, k, v, g, S0, np.full((B, L, H), 800.0), wq, wk, wv, cos, sin),
                               rtol=1e-13, atol=1e-15)
    np.testing.assert_array_equal(S0, S_keep)


def test_projections_against_library_matmul(oracle):
    """Sec. 3.1 and Eq. 6-7: the projections are plain matrix products in the [B, L, H, D] layout of the core."""
    B, L, H, D = 2, 5, 3, 4
    d = H * D
    x = rnd(B, L, d)
    w_q, w_k, w_v, w_o, w_g = rnd(d, d), rnd(d, d), rnd(d, d), rnd(d, d), rnd(d, H)
    q, k, v, g = oracle.project_in(x, w_q, w_k, w_v, w_g, H)
    np.testing.assert_allclose(q, (x @ w_q).reshape(B, L, H, D), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(k, (x @ w_k).reshape(B, L, H, D), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(v, (x @ w_v).reshape(B, L, H, D), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(g, x @ w_g, rtol=1e-12, atol=1e-13)
    # head h of a token is columns [h D, (h + 1) D) of the projected row
    np.testing.assert_allclose(q[1, 2, 1], x[1, 2] @ w_q[:, D:2 * D], rtol=1e-12, atol=1e-13)
    o = rnd(B, L, H, D)
    np.testing.assert_allclose(oracle.project_out(o, w_o), o.reshape(B, L, d) @ w_o, rtol=1e-12, atol=1e-13)
    # identity weights pass the tokens through; a weight with one non-zero entry moves one channel
    eye = np.eye(d)
    np.testing.assert_array_equal(oracle.project_out(o, eye), o.reshape(B, L, d))
    one = np.zeros((d, d)); one[3, 7] = 2.0
    y = oracle.project_out(o, one)
    np.testing.assert_allclose(y[..., 7], 2.0 * o.reshape(B, L, d)[..., 3]); assert not y[..., :7].any()


def test_reset(oracle):
    S = rnd(3, 2, 4, 4)
    r = oracle.reset(S, 1)
    assert (r[1] == 0).all() and r[0].tobytes() == S[0].tobytes() and r[2].tobytes() == S[2].tobytes()
    assert (oracle.reset(S) == 0).all()


def test_step_rows_matches_full_step(oracle):
    cfg = workload.custom(B=2, H=3, D=8, L=40)
    q, k, v, g = workload.step_inputs(cfg, 0, 0)
    S, wq = rnd(2, 3, 8, 8), rnd(3, 8, 8)
    cos, sin = tables(40, 8)
    full = oracle.step(q, k, v, g, S, wq, cos, sin)
    rows = [(0, 0, 0), (1, 2, 39), (0, 1, 17), (1, 0, 5)]
    got = oracle.step_rows(q, k, v, g, S, rows, wq, cos, sin)
    for r, (b, h, i) in enumerate(rows):
        assert got[r].tobytes() == full[b, i, h].tobytes()


def test_golden_fixture_regression(oracle):
    """The stored tiny case (written by tests/golden/make_golden.py from the oracle alone)."""
    import json
    import os

    with open(os.path.join(os.path.dirname(__file__), "golden", "tiny_layer.json")) as f:
        doc = json.load(f)
    A = lambda key: np.array(doc[key], dtype=np.float64)  # noqa: E731
    cos, sin = np.cos(A("angle")), np.sin(A("angle"))
    out = oracle.step(A("q"), A("k"), A("v"), A("g"), A("S0"), A("wq"), cos, sin, eps=doc["eps"])
    S1 = oracle.commit(A("kc"), A("vc"), A("a"), A("S0"), A("wk"), A("wv"), cos, sin,
                       eps=doc["eps"])
    np.testing.assert_allclose(out, A("out"), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(S1, A("S1"), rtol=1e-13, atol=1e-15)
    # and the same case through the independent pure-Python restatement
    ref = brute_force_layer(A("q"), A("k"), A("v"), A("g"), A("S0"), A("wq"), cos, sin,
                            1.0 / math.sqrt(doc["D"]), doc["eps"])
    np.testing.assert_allclose(A("out"), ref, rtol=1e-11, atol=1e-13)
