"""ctypes front end of the CPU float64 oracle (``arl2_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
bench's CPU-baseline leg.  Nothing on the product path imports this module, and
this module imports nothing from the CUDA package.

Every function takes numpy arrays or torch CPU tensors of any float dtype, widens
them to float64 (so the oracle sees exactly the bf16 / fp32 values the GPU saw) and
returns float64 numpy arrays.  Shapes follow the C file's header comment.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "arl2_oracle.c")
_BUILD = os.path.join(_HERE, "_build")
_SO = os.path.join(_BUILD, "libarl2_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp); returns the path of the library."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            os.makedirs(_BUILD, exist_ok=True)
            tmp = _SO + ".%d.tmp" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.arl2_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().arl2_oracle_threads())


def _f64(x):
    """Widen to a contiguous float64 numpy array (None stays None)."""
    if x is None:
        return None
    if hasattr(x, "detach"):  # torch tensor
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _ip(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def feature(x, W, rope_cos, rope_sin, eps: float, mode: int):
    """Eq. 3: mode 0 = L2Norm(RoPE(phi(x))), mode 1 = phi(x).  x is [B, L, H, D]."""
    x, W, rope_cos, rope_sin = _f64(x), _f64(W), _f64(rope_cos), _f64(rope_sin)
    B, L, H, D = x.shape
    y = np.empty_like(x)
    _load().arl2_oracle_feature(
        B, H, L, D, _p(x), _p(W), _p(rope_cos), _p(rope_sin), ctypes.c_double(eps), mode, _p(y)
    )
    return y


def step(q, k, v, g, S, wq=None, rope_cos=None, rope_sin=None, scale=None, eps=1e-6):
    """One denoise-step call of the layer: returns O [B, L, H, D]; S is only read."""
    q, k, v, g, S = _f64(q), _f64(k), _f64(v), _f64(g), _f64(S)
    wq, rope_cos, rope_sin = _f64(wq), _f64(rope_cos), _f64(rope_sin)
    B, L, H, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty_like(q)
    _load().arl2_oracle_step(
        B, H, L, D, _p(q), _p(k), _p(v), _p(g), _p(S), _p(wq), _p(rope_cos), _p(rope_sin),
        ctypes.c_double(scale), ctypes.c_double(eps), _p(out),
    )
    return out


def step_gate_mode(q, k, v, g, S, gate_mode, wq=None, rope_cos=None, rope_sin=None, scale=None, eps=1e-6):
    """The layer with the combine gate at another granularity: gate_mode 0 headwise g [B, L, H],
    1 scalar g [B, L], 2 elementwise g [B, L, H, D]."""
    q, k, v, g, S = _f64(q), _f64(k), _f64(v), _f64(g), _f64(S)
    wq, rope_cos, rope_sin = _f64(wq), _f64(rope_cos), _f64(rope_sin)
    B, L, H, D = q.shape
    assert g.shape == {0: (B, L, H), 1: (B, L), 2: (B, L, H, D)}[gate_mode]
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty_like(q)
    _load().arl2_oracle_step_gate_mode(
        B, H, L, D, gate_mode, _p(q), _p(k), _p(v), _p(g), _p(S), _p(wq), _p(rope_cos), _p(rope_sin),
        ctypes.c_double(scale), ctypes.c_double(eps), _p(out),
    )
    return out


def step_rows(q, k, v, g, S, rows, wq=None, rope_cos=None, rope_sin=None, scale=None,
              eps=1e-6):
    """Outputs of the sampled (b, h, i) triples in ``rows`` ([n, 3] ints): returns [n, D]."""
    q, k, v, g, S = _f64(q), _f64(k), _f64(v), _f64(g), _f64(S)
    wq, rope_cos, rope_sin = _f64(wq), _f64(rope_cos), _f64(rope_sin)
    B, L, H, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    rows = np.asarray(rows, dtype=np.int32).reshape(-1, 3)
    bs = np.ascontiguousarray(rows[:, 0])
    hs = np.ascontiguousarray(rows[:, 1])
    is_ = np.ascontiguousarray(rows[:, 2])
    assert (bs >= 0).all() and (bs < B).all() and (hs >= 0).all() and (hs < H).all()
    assert (is_ >= 0).all() and (is_ < L).all()
    out = np.empty((rows.shape[0], D), dtype=np.float64)
    _load().arl2_oracle_step_rows(
        B, H, L, D, _p(q), _p(k), _p(v), _p(g), _p(S), _p(wq), _p(rope_cos), _p(rope_sin),
        ctypes.c_double(scale), ctypes.c_double(eps), rows.shape[0], _ip(bs), _ip(hs), _ip(is_),
        _p(out),
    )
    return out


def step_token_level(q, k, v, g, S, alpha_logit=None, wq=None, wk=None, wv=None, rope_cos=None, rope_sin=None,
                     scale=None, eps=1e-6):
    """Token-level state access (comparison mode): token i reads S advanced by the block's tokens before it
    (gated-linear update with per-token forget gates alpha_logit [B, L, H], None = 1).  Returns O; S is only read."""
    q, k, v, g, S = _f64(q), _f64(k), _f64(v), _f64(g), _f64(S)
    wq, wk, wv, rope_cos, rope_sin = _f64(wq), _f64(wk), _f64(wv), _f64(rope_cos), _f64(rope_sin)
    alpha_logit = _f64(alpha_logit)
    B, L, H, D = q.shape
    assert S.shape == (B, H, D, D) and g.shape == (B, L, H)
    assert alpha_logit is None or alpha_logit.shape == (B, L, H)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty_like(q)
    _load().arl2_oracle_step_token_level(
        B, H, L, D, _p(q), _p(k), _p(v), _p(g), _p(alpha_logit), _p(S), _p(wq), _p(wk), _p(wv),
        _p(rope_cos), _p(rope_sin), ctypes.c_double(scale), ctypes.c_double(eps), _p(out),
    )
    return out


def attend_cache(q, k_cache, v_cache, scale=None):
    """Eq. 1: softmax attention of q [B, L, H, D] over a cache [B, Lk, H, D]; scale None = 1/sqrt(D)."""
    q, k_cache, v_cache = _f64(q), _f64(k_cache), _f64(v_cache)
    B, L, H, D = q.shape
    Lk = k_cache.shape[1]
    assert k_cache.shape == (B, Lk, H, D) and v_cache.shape == (B, Lk, H, D)
    out = np.empty((B, L, H, D), dtype=np.float64)
    sc = (1.0 / np.sqrt(D)) if scale is None else float(scale)
    _load().arl2_oracle_attend_cache(B, H, L, Lk, D, _p(q), _p(k_cache), _p(v_cache),
                                     ctypes.c_double(sc), _p(out))
    return out


def commit(kc, vc, a, S, wk=None, wv=None, rope_cos=None, rope_sin=None, eps=1e-6, rule=0,
           beta_logit=None, heads=None):
    """State commit, once per block.  Returns the new S (the argument is not modified).

    ``heads``: optional [n, 2] list of (b, h) pairs; other heads are left as they were.
    """
    kc, vc, a = _f64(kc), _f64(vc), _f64(a)
    wk, wv, rope_cos, rope_sin = _f64(wk), _f64(wv), _f64(rope_cos), _f64(rope_sin)
    beta_logit = _f64(beta_logit)
    S = _f64(S).copy()
    B, L, H, D = kc.shape
    assert S.shape == (B, H, D, D) and a.shape == (B, H)
    if heads is None:
        n, bs, hs = 0, None, None
    else:
        heads = np.asarray(heads, dtype=np.int32).reshape(-1, 2)
        n = heads.shape[0]
        bs = np.ascontiguousarray(heads[:, 0])
        hs = np.ascontiguousarray(heads[:, 1])
    _load().arl2_oracle_commit(
        B, H, L, D, _p(kc), _p(vc), _p(a), _p(beta_logit), _p(wk), _p(wv), _p(rope_cos),
        _p(rope_sin), ctypes.c_double(eps), rule, n, _p(bs), _p(hs), _p(S),
    )
    return S


def clean_pass(q, kc, vc, g, a, S, wq=None, wk=None, wv=None, rope_cos=None, rope_sin=None, scale=None,
               eps=1e-6):
    """The clean pass of a block: returns (out, S_new); out is read against the state passed in."""
    q, kc, vc, g, a = _f64(q), _f64(kc), _f64(vc), _f64(g), _f64(a)
    wq, wk, wv, rope_cos, rope_sin = _f64(wq), _f64(wk), _f64(wv), _f64(rope_cos), _f64(rope_sin)
    S = _f64(S).copy()
    B, L, H, D = q.shape
    assert S.shape == (B, H, D, D) and a.shape == (B, H) and g.shape == (B, L, H)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty_like(q)
    _load().arl2_oracle_clean_pass(
        B, H, L, D, _p(q), _p(kc), _p(vc), _p(g), _p(a), _p(wq), _p(wk), _p(wv), _p(rope_cos), _p(rope_sin),
        ctypes.c_double(scale), ctypes.c_double(eps), _p(S), _p(out),
    )
    return out, S


def commit_tokens(kc, vc, S, alpha_logit=None, beta_logit=None, wk=None, wv=None, rope_cos=None,
                  rope_sin=None, eps=1e-6, heads=None, decayed_prediction=False):
    """Eq. 4 token by token with per-token gates [B, L, H] (None = gate 1).  Returns the new S.
    decayed_prediction: each token predicts against alpha_j S instead of S (the other reading of Eq. 4)."""
    kc, vc = _f64(kc), _f64(vc)
    wk, wv, rope_cos, rope_sin = _f64(wk), _f64(wv), _f64(rope_cos), _f64(rope_sin)
    alpha_logit, beta_logit = _f64(alpha_logit), _f64(beta_logit)
    S = _f64(S).copy()
    B, L, H, D = kc.shape
    assert S.shape == (B, H, D, D)
    for g in (alpha_logit, beta_logit):
        assert g is None or g.shape == (B, L, H)
    if heads is None:
        n, bs, hs = 0, None, None
    else:
        heads = np.asarray(heads, dtype=np.int32).reshape(-1, 2)
        n = heads.shape[0]
        bs = np.ascontiguousarray(heads[:, 0])
        hs = np.ascontiguousarray(heads[:, 1])
    _load().arl2_oracle_commit_tokens(
        B, H, L, D, _p(kc), _p(vc), _p(alpha_logit), _p(beta_logit), _p(wk), _p(wv), _p(rope_cos),
        _p(rope_sin), ctypes.c_double(eps), n, _p(bs), _p(hs), int(bool(decayed_prediction)), _p(S),
    )
    return S


def commit_decay_tokens(kc, vc, S, alpha_logit, wk=None, wv=None, rope_cos=None, rope_sin=None,
                        eps=1e-6, heads=None):
    """Gated-linear update with per-token forget gates [B, L, H], token by token.  Returns the new S."""
    kc, vc, alpha_logit = _f64(kc), _f64(vc), _f64(alpha_logit)
    wk, wv, rope_cos, rope_sin = _f64(wk), _f64(wv), _f64(rope_cos), _f64(rope_sin)
    S = _f64(S).copy()
    B, L, H, D = kc.shape
    assert S.shape == (B, H, D, D) and alpha_logit.shape == (B, L, H)
    if heads is None:
        n, bs, hs = 0, None, None
    else:
        heads = np.asarray(heads, dtype=np.int32).reshape(-1, 2)
        n = heads.shape[0]
        bs = np.ascontiguousarray(heads[:, 0])
        hs = np.ascontiguousarray(heads[:, 1])
    _load().arl2_oracle_commit_decay_tokens(
        B, H, L, D, _p(kc), _p(vc), _p(alpha_logit), _p(wk), _p(wv), _p(rope_cos), _p(rope_sin),
        ctypes.c_double(eps), n, _p(bs), _p(hs), _p(S),
    )
    return S


def project_in(x, w_q, w_k, w_v, w_g, H):
    """Sec. 3.1 / Eq. 6: Q, K, V = x W_q, x W_k, x W_v as [B, L, H, D] and the gate logits x W_g [B, L, H]."""
    x, w_q, w_k, w_v, w_g = _f64(x), _f64(w_q), _f64(w_k), _f64(w_v), _f64(w_g)
    B, L, d = x.shape
    assert d % H == 0 and w_q.shape == (d, d) and w_k.shape == (d, d) and w_v.shape == (d, d) and w_g.shape == (d, H)
    q, k, v = (np.empty((B, L, d)) for _ in range(3))
    g = np.empty((B, L, H))
    _load().arl2_oracle_project_in(ctypes.c_long(B * L), d, H, _p(x), _p(w_q), _p(w_k), _p(w_v), _p(w_g),
                                   _p(q), _p(k), _p(v), _p(g))
    D = d // H
    return q.reshape(B, L, H, D), k.reshape(B, L, H, D), v.reshape(B, L, H, D), g


def project_out(o, w_o):
    """Eq. 7: y = O W_o with O [B, L, H, D] read as [B, L, d]."""
    o, w_o = _f64(o), _f64(w_o)
    B, L, H, D = o.shape
    d = H * D
    assert w_o.shape == (d, d)
    y = np.empty((B, L, d))
    _load().arl2_oracle_project_out(ctypes.c_long(B * L), d, _p(o), _p(w_o), _p(y))
    return y


def reset(S, stream: int = -1):
    """S <- 0 for one stream or all (stream < 0).  Returns a new array."""
    S = _f64(S).copy()
    B, H, D, _ = S.shape
    _load().arl2_oracle_reset(B, H, D, stream, _p(S))
    return S
