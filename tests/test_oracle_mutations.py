"""The pins have teeth: a plausible mistake planted in a copy of the oracle's C source makes one of them fail.

Each case rewrites one line of oracle/firp_oracle.c into a temporary copy, builds it, runs the same comparison
against the independent fp64 library decoder that the pins use (every row of a random tree == a causal forward
over prefix + its root path; the pseudo chain == a forward with rows replaced at layer l) and requires the
error to leave the 1e-5 band on at least one shape, while the unaltered source stays inside it on all of them.
Nothing here touches a GPU, and the planted mistakes never leave the temporary directory.
"""
import ctypes
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si
from hf_reference import build_hf_llama, hf_logits, hf_logits_with_replaced_rows

SRC = os.path.join(os.path.dirname(oracle.__file__), "firp_oracle.c")

MUTATIONS = {
    "gains of the attention and MLP norms swapped": [
        ("rmsnorm(h, w->g_attn[j], c->eps, x, rows, d);", "rmsnorm(h, w->g_mlp[j], c->eps, x, rows, d);"),
        ("rmsnorm(h, w->g_mlp[j], c->eps, x, rows, d);\n    linear(w->wgate", "rmsnorm(h, w->g_attn[j], c->eps, x, rows, d);\n    linear(w->wgate")],
    "final norm takes a layer's gain": [("rmsnorm(h, w->g_final, c->eps, x, M, d);", "rmsnorm(h, w->g_attn[0], c->eps, x, M, d);")],
    "gain dropped from RMSNorm": [("* r * (double)bf16f(g[c]));", "* r);")],
    "query head mapped to kv head by remainder": [("const int kvh = hd / (H / Hkv);", "const int kvh = hd % Hkv;")],
    "rotary sign flipped": [("x[c] = (float)(a * cs - b * sn);", "x[c] = (float)(a * cs + b * sn);")],
    "Eq. 3 reads the map transposed": [
        ("for (int c = 0; c < n_in; ++c) wrow[c] = bf16f(W[(size_t)o * n_in + c]);",
         "for (int c = 0; c < n_in; ++c) wrow[c] = bf16f(n_in == n_out && M == 1 ? W[(size_t)c * n_in + o] : W[(size_t)o * n_in + c]);")],
    "scores not scaled by sqrt(dh)": [("p[u] = s / sqrt((double)dh);", "p[u] = s;")],
    "eps left out of the norm": [("double r = 1.0 / sqrt(ss / d + (double)eps);", "double r = 1.0 / sqrt(ss / d);")],
}

SHAPES = {
    "gains": (dict(), True),
    "gqa2": (dict(Hkv=2), False),
    "big_eps": (dict(eps=0.5), False),     # a shape on which the eps term is not negligible
}


@pytest.fixture(scope="module")
def cases():
    out = {}
    for name, (over, gains) in SHAPES.items():
        shape = si.scaled(si.CONFIGS["c1"], **over)
        weights = si.all_weights(shape, gains=gains)
        out[name] = (shape, weights, build_hf_llama(shape, weights))
    return out


def pin_error(shape, weights, hfm) -> float:
    """max |oracle - library decoder| over the rows of a tree step (tree rows and the pseudo chain)."""
    prompt = si.prompt(shape, length=9)
    k, l, T = 3, 1, 7
    o = oracle.Oracle(shape, weights, max_ctx=64, kv_bf16=False)
    o.forward(prompt, si.chain_template(prompt.size), 0, 0)
    o.commit(np.arange(prompt.size))
    parents = si.random_tree(5, T, 3, 1)
    tokens = si.random_tokens(shape, T, 3)
    out = o.forward(tokens, parents, k, l, anchor=0)
    err = 0.0
    for v in range(T):
        path, u = [], v
        while u >= 0:
            path.append(u)
            u = int(parents[u])
        ref = hf_logits(hfm, list(prompt) + [int(tokens[u]) for u in path[::-1]])[-1]
        err = max(err, float(np.abs(out["logits"][v] - ref).max()))
    Wf = si.bf16_bits_to_f32(weights["pred_w"]).astype(np.float64)
    ids = list(prompt) + [int(tokens[0])] + [0] * k
    ref = hf_logits_with_replaced_rows(hfm, ids, l, prompt.size + 1, list(Wf), list(np.zeros((k, shape.d))), prompt.size)
    return max(err, float(np.abs(out["logits"][T:] - ref[prompt.size + 1:]).max()))


def test_unaltered_oracle_is_inside_the_band(cases):
    for name, case in cases.items():
        assert pin_error(*case) < 1e-5, name


@pytest.mark.parametrize("what", sorted(MUTATIONS))
def test_planted_mistake_fails_a_pin(what, cases, tmp_path, monkeypatch):
    text = open(SRC).read()
    for old, new in MUTATIONS[what]:
        assert text.count(old) == 1, "the line to alter must exist exactly once: %r" % old
        text = text.replace(old, new)
    src = tmp_path / "altered.c"
    src.write_text(text)
    lib = oracle.bind(ctypes.CDLL(oracle.compile_source(str(src), str(tmp_path / "altered.so"))))
    monkeypatch.setattr(oracle, "_lib", lib)
    errs = {name: pin_error(*case) for name, case in cases.items()}
    assert max(errs.values()) > 1e-3, "no pin noticed: %s (%r)" % (what, errs)
