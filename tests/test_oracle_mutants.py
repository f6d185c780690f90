"""Planted mistakes: each one is put into a COPY of the oracle's C source (never into the CUDA
path), the copy is compiled, and the pins of test_oracle_pins.py are run against it.  Every
mistake must fail at least one pin -- that is what makes the pins worth trusting.  The stored
regression fixture is left out on purpose: a mutant has to be caught by a closed form, an
invariant, brute force or a library routine, not by numbers the oracle itself once wrote."""
import importlib.util
import inspect
import os

import pytest

import test_oracle_pins as pins

HERE = os.path.dirname(os.path.abspath(__file__))
ORACLE_DIR = os.path.join(os.path.dirname(HERE), "oracle")

# (name, text in arl2_oracle.c, what replaces its first occurrence)
MUTANTS = [
    ("rotation sign", "x[2 * m]     = x0 * c - x1 * s;", "x[2 * m]     = x0 * c + x1 * s;"),
    ("feature map transposed", "acc += x[i] * Wh[(size_t)i * D + o];", "acc += x[i] * Wh[(size_t)o * D + i];"),
    ("state transposed in the readout", "acc += qf[d] * Sh[(size_t)d * D + e];", "acc += qf[d] * Sh[(size_t)e * D + d];"),
    ("outer product transposed", "dS[(size_t)d * D + e] += kf[d] * vf[e];", "dS[(size_t)d * D + e] += kf[e] * vf[d];"),
    ("combine gate dropped", "o[e] += gate * acc;", "o[e] += acc;"),
    ("softmax scale dropped", "p[j] = s * scale;", "p[j] = s;"),
    ("query feature rotated at position 0", "rope(qf, D, rope_cos, rope_sin, i);", "rope(qf, D, rope_cos, rope_sin, 0);"),
    ("eps outside the root", "double r = 1.0 / sqrt(ss + eps);", "double r = 1.0 / (sqrt(ss) + eps);"),
    ("decay applied to the new term too", "Sh[t] = alpha * Sh[t] + dS[t];", "Sh[t] = alpha * (Sh[t] + dS[t]);"),
    ("value map replaced by the key map", "phi(vc + off, wv, h, D, vf);", "phi(vc + off, wk, h, D, vf);"),
    ("token-sequential rule without its decay", "Sh[t] *= alpha;", "Sh[t] *= 1.0;"),
    ("frame-level delta rule writes into the running state",
     "double *dst = (rule == 1) ? dS : Sh;", "double *dst = Sh;"),
    ("per-token rule predicts from the decayed state when asked for the printed form",
     "err[e] = vf[e] - (decayed ? alpha * acc : acc);", "err[e] = vf[e] - alpha * acc;"),
    ("per-token rule ignores the request for the decayed prediction",
     "err[e] = vf[e] - (decayed ? alpha * acc : acc);", "err[e] = vf[e] - acc;"),
    ("per-token rule forgets the learning rate",
     "alpha * Sh[(size_t)d * D + e] + beta * kf[d] * err[e];", "alpha * Sh[(size_t)d * D + e] + kf[d] * err[e];"),
    ("per-token decay applied to the new term", "alpha * Sh[(size_t)d * D + e] + kf[d] * vf[e];",
     "alpha * (Sh[(size_t)d * D + e] + kf[d] * vf[e]);"),
    ("cache attention without its scale", "w[j] = sc * scale;", "w[j] = sc;"),
    ("softmax normalised by the maximum term only", "double w = p[j] / den;", "double w = p[j];"),
    ("elementwise gate indexed per head", "gate_mode == 2 ? (((size_t)b * L + i) * H + h) * D + e",
     "gate_mode == 2 ? (((size_t)b * L + i) * H + h) * D"),
    ("clean pass reads the state it has just written",
     "    arl2_oracle_step(B, H, L, D, q, kc, vc, g, S, wq, rope_cos, rope_sin, scale, eps, out);\n"
     "    arl2_oracle_commit(B, H, L, D, kc, vc, a, NULL, wk, wv, rope_cos, rope_sin, eps, 0, 0, NULL, NULL, S);",
     "    arl2_oracle_commit(B, H, L, D, kc, vc, a, NULL, wk, wv, rope_cos, rope_sin, eps, 0, 0, NULL, NULL, S);\n"
     "    arl2_oracle_step(B, H, L, D, q, kc, vc, g, S, wq, rope_cos, rope_sin, scale, eps, out);"),
    ("token-level access reads the state after the token's own write",
     "            step_row(b, h, i, H, L, D, 0, q, k, v, g, Sloc, wq, rope_cos, rope_sin, scale, eps,\n"
     "                     out + off, scratch);\n            /* then the token's own write */",
     "            /* then the token's own write */"),
    ("token-level access decays the new term",
     "Sloc[(size_t)d * D + e] = alpha * Sloc[(size_t)d * D + e] + kf[d] * vf[e];",
     "Sloc[(size_t)d * D + e] = alpha * (Sloc[(size_t)d * D + e] + kf[d] * vf[e]);"),
    ("projection weight read transposed", "acc += x[(size_t)r * K + kk] * w[(size_t)kk * N + n];",
     "acc += x[(size_t)r * K + kk] * w[(size_t)n * K + kk];"),
    ("keys projected with the query weights", "matmul_rows(rows, d, d, x, w_k, k);", "matmul_rows(rows, d, d, x, w_q, k);"),
    ("gate logits projected from the wrong weights", "matmul_rows(rows, d, H, x, w_g, g);", "matmul_rows(rows, d, H, x, w_v, g);"),
    ("reset clears the wrong stream", "else memset(S + per * stream, 0, sizeof(double) * per);",
     "else memset(S, 0, sizeof(double) * per);"),
]


def pin_calls():
    """Every pin as (name, callable taking the oracle module), parametrised ones expanded."""
    out = []
    for name, fn in sorted(vars(pins).items()):
        if not name.startswith("test_") or not inspect.isfunction(fn):
            continue
        if name == "test_golden_fixture_regression":
            continue
        params = [p for p in inspect.signature(fn).parameters if p != "oracle"]
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not params:
            out.append((name, fn))
            continue
        assert len(marks) == 1, name
        names = [n.strip() for n in marks[0].args[0].split(",")]
        assert sorted(names) == sorted(params), name
        for vals in marks[0].args[1]:
            vals = vals if isinstance(vals, (tuple, list)) else (vals,)
            kw = dict(zip(names, vals))
            out.append((f"{name}{list(vals)}", lambda o, fn=fn, kw=kw: fn(o, **kw)))
    return out


def mutant_module(tmp_path, index, old, new):
    src = open(os.path.join(ORACLE_DIR, "arl2_oracle.c")).read()
    assert old in src, f"the oracle no longer contains `{old}`: update this mutant"
    c_path = tmp_path / "arl2_oracle.c"
    c_path.write_text(src.replace(old, new, 1))
    spec = importlib.util.spec_from_file_location(f"arl2_oracle_mutant_{index}",
                                                  os.path.join(ORACLE_DIR, "arl2_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod._SRC, mod._BUILD = str(c_path), str(tmp_path / "_build")
    mod._SO = os.path.join(mod._BUILD, "libarl2_oracle.so")
    mod.build(force=True)
    return mod


def test_the_unmutated_oracle_passes_every_pin(oracle):
    for name, call in pin_calls():
        call(oracle)


@pytest.mark.parametrize("index", range(len(MUTANTS)), ids=[m[0].replace(" ", "_") for m in MUTANTS])
def test_planted_mistake_fails_a_pin(tmp_path, index):
    name, old, new = MUTANTS[index]
    mod = mutant_module(tmp_path, index, old, new)
    caught = None
    for pin_name, call in pin_calls():
        try:
            call(mod)
        except AssertionError:
            caught = pin_name
            break
    assert caught is not None, f"planted mistake `{name}` passes every pin"
    print(f"{name}: caught by {caught}")
