"""Pins for the CPU oracle: it is checked against things other than itself.

  P1  T=1, k=0 stepping == cache-free greedy decoding by an independent library decoder
  P2  every tree row's logits == a plain causal forward over prefix + root->row path
  P3  Eq. 3 closed forms (W = I, W = 0, permutation W, non-zero bias)
  P4  losslessness (Eq. 1): emitted tokens == the autoregressive greedy stream
  P5  tree rows do not depend on k or on the predictor maps
  P6  committed cache == keys/values of a from-scratch forward over the committed tokens
  P7  forced-accept mode accepts the full depth every step
  P8  the pseudo chain == a causal forward whose rows are replaced at layer l
  P9  predictor size k*d^2 equals the draft-module sizes printed in the paper's Table 1
  P10 one insertion layer per prediction step (Section 3.3): the chain == a causal forward whose row i is
      replaced at layer t_i; step i does not depend on the layers of later steps; W = I closed form
  P11 a chain of k pseudo rows under every tree node: every chain row == a causal forward over prefix + the
      node's root path with rows replaced at the insertion layer(s); the root's chain == the single chain;
      mask == brute-force closure; the free-running decode stays lossless
  P12 the "Masked" setting of Section 4.3: the chain == a forward over prefix + root + k rows replaced at the
      insertion layer whose mask hides the pseudo rows from one another; step 1 and the tree rows are unchanged
plus hand-worked cases for the mask, the acceptance walk, the tie rules and the next tree.
"""
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si
from hf_reference import (build_hf_llama, hf_greedy, hf_kv, hf_logits, hf_logits_with_replaced_rows)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def hf(c1, c1_weights):
    return build_hf_llama(c1, c1_weights)


def fresh(c1, weights, max_ctx=256, n_seq=1, kv_bf16=False):
    # the library decoder keeps fp64 keys/values, so the 1e-5 pins run with an fp32 cache;
    # the bf16 cache mode has its own pins below
    return oracle.Oracle(c1, weights, max_ctx=max_ctx, n_seq=n_seq, kv_bf16=kv_bf16)


def path_to(parents, v):
    p = []
    while v >= 0:
        p.append(v)
        v = int(parents[v])
    return p[::-1]


# ---------------------------------------------------------------- P1
def test_p1_t1_k0_is_autoregressive_greedy(c1, c1_weights, hf):
    prompt = si.prompt(c1)
    want = hf_greedy(hf, prompt, 12)
    o = fresh(c1, c1_weights)
    r = o.prefill(prompt, 0, 0, None)
    got, tok, ids = [r["root"]], r["root"], list(prompt)
    one = np.array([-1], np.int32)
    for _ in range(11):
        out = o.step([tok], one, 0, 0)
        ids.append(tok)
        ref = hf_logits(hf, ids)[-1]
        assert np.abs(out["logits"][0] - ref).max() < 1e-5
        assert out["n_accepted"] == 1 and out["path"].tolist() == [0]
        o.commit([0])
        tok = int(out["accepted"][0])
        got.append(tok)
    assert got == want


# ---------------------------------------------------------------- P2
@pytest.mark.parametrize("case", range(4))
def test_p2_tree_rows_equal_per_path_causal_forward(c1, c1_weights, hf, case):
    prompt = si.prompt(c1, length=20 + 3 * case)
    T = (8, 13, 16, 5)[case]
    parents = si.tree_template(8) if case == 0 else si.random_tree(7, T, 3, case)
    tokens = si.random_tokens(c1, T, case)
    o = fresh(c1, c1_weights)
    o.prefill(prompt, 0, 0, None)
    out = o.forward(tokens, parents, 3, 1)
    for v in range(T):
        ids = list(prompt) + [int(tokens[u]) for u in path_to(parents, v)]
        ref = hf_logits(hf, ids)[-1]
        assert np.abs(out["logits"][v] - ref).max() < 1e-5, v
        assert out["depth"][v] == len(path_to(parents, v)) - 1


def test_mask_is_ancestor_closure_bruteforce():
    for case in range(6):
        T, k = 5 + 4 * case, case % 4
        parents = si.random_tree(11, T, 6, case)
        anchor = case % T
        tp = oracle.tree_prep(parents, k, anchor)
        ext = list(parents) + [anchor if i == 0 else T + i - 1 for i in range(k)]
        for v in range(T + k):
            anc = set(path_to(ext, v))
            assert set(np.nonzero(tp["mask"][v])[0].tolist()) == anc
            assert tp["depth"][v] == len(anc) - 1
        # tree rows never see pseudo rows
        assert not tp["mask"][:T, T:].any()
        for v in range(1, T):
            sib = [u for u in range(1, T) if parents[u] == parents[v]]
            assert tp["rank"][v] == sib.index(v)


def test_mask_worked_example():
    # the 8-node 2-2-1 template: root->1->2->3, root->4->6, 1->5->7; pseudo chain off the root
    tp = oracle.tree_prep(si.tree_template(8), 3, 0)
    with open(os.path.join(GOLDEN, "mask_t8_k3.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    want = np.array([[int(c) for c in r] for r in rows], np.uint8)
    assert (tp["mask"] == want).all()
    assert tp["depth"].tolist() == [0, 1, 2, 3, 1, 2, 2, 3, 1, 2, 3]


def test_malformed_trees_rejected():
    for bad in ([0, 0], [-1, 1], [-1, 2, 0], [-1, -1]):
        with pytest.raises(ValueError):
            oracle.tree_prep(np.array(bad, np.int32), 0, 0)


# ---------------------------------------------------------------- P3
def with_maps(weights, pred_w_f32, pred_b_f32):
    import torch
    w = dict(weights)
    to_bits = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    w["pred_w"], w["pred_b"] = to_bits(pred_w_f32), to_bits(pred_b_f32)
    return w


def test_p3_eq3_closed_forms(c1, c1_weights):
    d, k = c1.d, 3
    prompt = si.prompt(c1)
    tokens, parents = si.random_tokens(c1, 8, 5), si.tree_template(8)
    perm = np.roll(np.arange(d), 5)
    Wp = np.zeros((d, d), np.float32); Wp[np.arange(d), perm] = 1.0          # h~[o] = h[perm[o]]
    W = np.stack([np.eye(d, dtype=np.float32), np.zeros((d, d), np.float32), 2.0 * Wp])
    b = np.zeros((k, d), np.float32); b[1] = np.linspace(-1, 1, d); b[2] = 0.5
    w = with_maps(c1_weights, W, b)
    b_rounded = si.bf16_bits_to_f32(w["pred_b"])
    for anchor in (0, 4):
        o = fresh(c1, w)
        o.prefill(prompt, 0, 0, None)
        out = o.forward(tokens, parents, k, 1, anchor=anchor, want_h_at_l=True)
        h = out["h_at_l"]
        assert np.array_equal(h[8], h[anchor])                                 # W = I, b = 0
        assert np.array_equal(h[9], b_rounded[1])                              # W = 0
        assert np.allclose(h[10], 2.0 * h[anchor][perm] + b_rounded[2], rtol=0, atol=1e-6)   # permutation
        assert out["depth"][8:].tolist() == [out["depth"][anchor] + i for i in (1, 2, 3)]


def test_p3_eq3_orientation_out_in(c1, c1_weights):
    # a single non-zero entry W[o=3][c=7] = 1.5 must move coordinate 7 into coordinate 3
    d = c1.d
    W = np.zeros((3, d, d), np.float32); W[0, 3, 7] = 1.5
    w = with_maps(c1_weights, W, np.zeros((3, d), np.float32))
    o = fresh(c1, w)
    o.prefill(si.prompt(c1), 0, 0, None)
    h = o.forward([5], [-1], 3, 1, want_h_at_l=True)["h_at_l"]
    want = np.zeros(d, np.float32); want[3] = np.float32(1.5) * h[0, 7]
    assert np.allclose(h[1], want, rtol=0, atol=1e-7) and h[0, 7] != 0


# ---------------------------------------------------------------- P8
@pytest.mark.parametrize("l", [0, 1])
def test_p8_pseudo_chain_is_causal_forward_with_replaced_rows(c1, c1_weights, hf, l):
    k = 3
    prompt = si.prompt(c1, length=17)
    Wf = si.bf16_bits_to_f32(c1_weights["pred_w"]).astype(np.float64)
    bf = np.zeros((k, c1.d))
    o = fresh(c1, c1_weights)
    # plain picture of Section 3.2: chain over the prompt, anchor = last prompt token
    chain = si.chain_template(prompt.size)
    out = o.forward(prompt, chain, k, l, anchor=prompt.size - 1)
    ids = list(prompt) + [0] * k            # filler ids: their rows are replaced at layer l
    ref = hf_logits_with_replaced_rows(hf, ids, l, prompt.size, list(Wf), list(bf), prompt.size - 1)
    assert np.abs(out["logits"][prompt.size:] - ref[prompt.size:]).max() < 1e-5
    assert np.abs(out["logits"][: prompt.size] - ref[: prompt.size]).max() < 1e-5
    # chain off the root of a tree step (anchor 0) on top of a committed prefix
    o.commit(np.arange(prompt.size))
    tokens, parents = si.random_tokens(c1, 8, 9), si.tree_template(8)
    out = o.forward(tokens, parents, k, l, anchor=0)
    ids = list(prompt) + [int(tokens[0])] + [0] * k
    ref = hf_logits_with_replaced_rows(hf, ids, l, prompt.size + 1, list(Wf), list(bf), prompt.size)
    assert np.abs(out["logits"][8:] - ref[prompt.size + 1:]).max() < 1e-5


# ---------------------------------------------------------------- P10
@pytest.fixture(scope="module")
def c1_deep():
    shape = si.scaled(si.CONFIGS["c1"], L=4, l=1)
    return shape, si.all_weights(shape)


@pytest.mark.parametrize("layers", [(0, 1, 3), (1, 1, 2), (2, 3, 3), (0, 0, 0)])
def test_p10_per_step_layers_chain_is_causal_forward_with_rows_replaced_at_their_layers(c1_deep, layers):
    shape, weights = c1_deep
    hf4 = build_hf_llama(shape, weights)
    k = 3
    prompt = si.prompt(shape, length=13)
    Wf = si.bf16_bits_to_f32(weights["pred_w"]).astype(np.float64)
    bf = np.zeros((k, shape.d))
    o = fresh(shape, weights)
    o.forward(prompt, si.chain_template(prompt.size), 0, 0)
    o.commit(np.arange(prompt.size))
    tokens, parents = si.random_tokens(shape, 8, 9), si.tree_template(8)
    out = o.forward(tokens, parents, k, list(layers), anchor=0)
    ids = list(prompt) + [int(tokens[0])] + [0] * k
    ref = hf_logits_with_replaced_rows(hf4, ids, layers, prompt.size + 1, list(Wf), list(bf), prompt.size)
    assert np.abs(out["logits"][8:] - ref[prompt.size + 1:]).max() < 1e-5
    # the tree rows are those of a plain tree step
    plain = o.forward(tokens, parents, 0, 0)["logits"]
    assert np.array_equal(out["logits"][:8], plain)
    # the same layer for every step is the single-layer call
    if len(set(layers)) == 1:
        assert np.array_equal(out["logits"], o.forward(tokens, parents, k, layers[0])["logits"])


def test_p10_a_step_ignores_the_layers_of_later_steps_and_identity_maps_copy_the_anchor(c1_deep):
    shape, weights = c1_deep
    d, k = shape.d, 3
    prompt = si.prompt(shape)
    tokens, parents = si.random_tokens(shape, 8, 4), si.tree_template(8)
    o = fresh(shape, weights)
    o.prefill(prompt, 0, 0, None)
    a = o.forward(tokens, parents, k, [1, 2, 3])["logits"]
    b = o.forward(tokens, parents, k, [1, 3, 3])["logits"]
    c = o.forward(tokens, parents, 1, 1)["logits"]
    assert np.array_equal(a[8], b[8]) and np.array_equal(a[8], c[8])          # step 1 sees no later step
    assert not np.array_equal(a[9], b[9])                                      # step 2 moved from layer 2 to 3
    with pytest.raises(ValueError):
        o.forward(tokens, parents, k, [2, 1, 3])                               # layers must not decrease
    with pytest.raises(ValueError):
        o.forward(tokens, parents, k, [1, 2, 4])                               # layer outside the decoder
    # W = I, b = 0: pseudo row i is the anchor's residual entering layer t_i
    wI = with_maps(weights, np.stack([np.eye(d, dtype=np.float32)] * k), np.zeros((k, d), np.float32))
    oI = fresh(shape, wI)
    oI.prefill(prompt, 0, 0, None)
    for anchor in (0, 3):
        h_ins = oI.forward(tokens, parents, k, [0, 2, 3], anchor=anchor, want_h_at_l=True)["h_ins"]
        for i, t in enumerate((0, 2, 3)):
            h_t = oI.forward(tokens, parents, 0, t, want_h_at_l=True)["h_at_l"]   # k = 0: plain residual at layer t
            assert np.array_equal(h_ins[i], h_t[anchor])


# ---------------------------------------------------------------- P11
def test_p11_chain_bookkeeping_is_the_closure_of_its_parents():
    parents = si.tree_template(8)
    T, k = 8, 3
    tp = oracle.tree_prep_chains(parents, k)
    M = T * (1 + k)
    base = oracle.tree_prep(parents)
    for v in range(T):
        for i in range(1, k + 1):
            r = oracle.chain_row(T, v, i)
            assert tp["depth"][r] == base["depth"][v] + i                      # position id pos[v] + i (Section 3.3)
            want = np.zeros(M, np.uint8)
            want[:T] = base["mask"][v]                                         # what v sees among the tree rows
            for j in range(1, i + 1):
                want[oracle.chain_row(T, v, j)] = 1                            # earlier rows of its own chain, itself
            assert np.array_equal(tp["mask"][r], want)
    assert np.array_equal(tp["mask"][:T, :T], base["mask"]) and not tp["mask"][:T, T:].any()   # tree rows see no chain


@pytest.mark.parametrize("layers", [1, (0, 1, 3), (2, 2, 3)])
def test_p11_every_chain_row_is_a_causal_forward_over_its_nodes_path(c1_deep, layers):
    shape, weights = c1_deep
    hf4 = build_hf_llama(shape, weights)
    k, T = 3, 8
    prompt = si.prompt(shape, length=11)
    Wf = si.bf16_bits_to_f32(weights["pred_w"]).astype(np.float64)
    bf = np.zeros((k, shape.d))
    o = fresh(shape, weights)
    o.forward(prompt, si.chain_template(prompt.size), 0, 0)
    o.commit(np.arange(prompt.size))
    tokens, parents = si.random_tokens(shape, T, 6), si.tree_template(T)
    out = o.forward_chains(tokens, parents, k, layers if np.isscalar(layers) else list(layers))
    for v in range(T):
        path = path_to(parents, v)
        ids = list(prompt) + [int(tokens[u]) for u in path] + [0] * k
        first = prompt.size + len(path)
        ref = hf_logits_with_replaced_rows(hf4, ids, layers, first, list(Wf), list(bf), first - 1)
        got = out["logits"][[oracle.chain_row(T, v, i) for i in (1, 2, 3)]]
        assert np.abs(got - ref[first:]).max() < 1e-5, "chain of node %d" % v
        assert np.abs(out["logits"][v] - ref[first - 1]).max() < 1e-5
    # the root's chain is the single chain of the plain step; tree rows do not depend on the chains
    one = o.forward(tokens, parents, k, layers if np.isscalar(layers) else list(layers), anchor=0)["logits"]
    assert np.array_equal(out["logits"][:T], one[:T])
    assert np.array_equal(out["logits"][[oracle.chain_row(T, 0, i) for i in (1, 2, 3)]], one[T:])
    assert np.array_equal(o.forward(tokens, parents, k, 1, anchor=5)["logits"][T:],
                          o.forward_chains(tokens, parents, k, 1)["logits"][[oracle.chain_row(T, 5, i) for i in (1, 2, 3)]])


def test_p11_decoding_with_chains_is_lossless_and_reads_the_end_nodes_chain(c1, c1_weights, hf):
    prompt = si.prompt(c1)
    want = hf_greedy(hf, prompt, 40)
    parents = si.tree_template(c1.T)
    o = fresh(c1, c1_weights)
    r = o.prefill(prompt, c1.k, c1.l, parents)
    tokens, emitted = r["next_tokens"].copy(), [r["root"]]
    for _ in range(10):
        out = o.step_chains(tokens, parents, c1.k, c1.l)
        end = out["end_node"]
        assert end == out["path"][-1]
        rows = [oracle.chain_row(c1.T, end, i) for i in (1, 2, 3)]
        for i, rr in enumerate(rows):                      # candidates of depth i+1 come from row i+1 of the end node's chain
            order = np.lexsort((np.arange(c1.V), -out["logits"][rr]))[:8]
            assert np.array_equal(out["topb_ids"][i], order)
        o.commit(out["path"])
        emitted += out["accepted"].tolist()
        tokens = out["next_tokens"].copy()
    assert emitted == want[: len(emitted)]                 # Eq. 1: the stream is the greedy stream


# ---------------------------------------------------------------- P12
def test_p12_masked_pseudo_rows_see_no_other_pseudo_row(c1, c1_weights, hf):
    k, l = 3, 1
    prompt = si.prompt(c1, length=15)
    Wf = si.bf16_bits_to_f32(c1_weights["pred_w"]).astype(np.float64)
    tokens, parents = si.random_tokens(c1, 8, 11), si.tree_template(8)
    om = oracle.Oracle(c1, c1_weights, max_ctx=256, kv_bf16=False, masked=True)
    on = fresh(c1, c1_weights)
    for o in (om, on):
        o.forward(prompt, si.chain_template(prompt.size), 0, 0)
        o.commit(np.arange(prompt.size))
    masked, plain = om.forward(tokens, parents, k, l), on.forward(tokens, parents, k, l)
    n = prompt.size
    # prefix, root and the k pseudo rows at positions n+1..n+k: causal, except that a pseudo row sees no other one
    ids = list(prompt) + [int(tokens[0])] + [0] * k
    L = len(ids)
    vis = np.tril(np.ones((L, L), np.uint8))
    vis[n + 1:, n + 1:] = np.eye(k, dtype=np.uint8)
    ref = hf_logits_with_replaced_rows(hf, ids, l, n + 1, list(Wf), list(np.zeros((k, c1.d))), n, visible=vis)
    assert np.abs(masked["logits"][8:] - ref[n + 1:]).max() < 1e-5
    causal = hf_logits_with_replaced_rows(hf, ids, l, n + 1, list(Wf), list(np.zeros((k, c1.d))), n,
                                          visible=np.tril(np.ones((L, L), np.uint8)))
    assert np.abs(plain["logits"][8:] - causal[n + 1:]).max() < 1e-5            # the explicit causal mask is the default one
    assert np.array_equal(masked["logits"][:9], plain["logits"][:9])          # tree rows and step 1 are the same
    assert not np.array_equal(masked["logits"][9:], plain["logits"][9:])      # steps 2, 3 lost what they saw
    want = plain["mask"].copy()
    want[8:, 8:] = np.eye(k, dtype=np.uint8)
    assert np.array_equal(masked["mask"], want) and np.array_equal(masked["depth"], plain["depth"])


# ---------------------------------------------------------------- P5
def test_p5_tree_rows_independent_of_k_and_maps(c1, c1_weights):
    prompt, tokens, parents = si.prompt(c1), si.random_tokens(c1, 8, 2), si.tree_template(8)
    o = fresh(c1, c1_weights)
    o.prefill(prompt, 0, 0, None)
    a = o.forward(tokens, parents, 0, 0)["logits"]
    b = o.forward(tokens, parents, 3, 1)["logits"]
    w2 = with_maps(c1_weights, np.random.default_rng(0).normal(size=(3, c1.d, c1.d)).astype(np.float32),
                   np.ones((3, c1.d), np.float32))
    o2 = fresh(c1, w2)
    o2.prefill(prompt, 0, 0, None)
    c = o2.forward(tokens, parents, 3, 0)["logits"]
    assert np.array_equal(a, b[:8]) and np.array_equal(a, c[:8])
    assert not np.array_equal(b[8:], c[8:])


# ---------------------------------------------------------------- P4, P6, P7
def run_free(o, c1, prompt, steps, forced, hf_stream=None):
    """Free-running decode with the oracle's own trees; returns emitted tokens and per-step a."""
    parents = si.tree_template(c1.T)
    tp = oracle.tree_prep(parents)
    D = int(tp["depth"].max())
    principal = [0]
    for _ in range(D):
        principal.append(min(u for u in range(c1.T) if parents[u] == principal[-1]))
    r = o.prefill(prompt, c1.k, c1.l, parents)
    tokens, emitted, accs = r["next_tokens"].copy(), [r["root"]], []
    for _ in range(steps):
        if forced:
            g = o.ar_greedy(int(tokens[0]), D)
            for j in range(1, D + 1):
                v = principal[j]
                sibs = [u for u in range(c1.T) if parents[u] == parents[v] and u != v and tokens[u] == g[j - 1]]
                for u in sibs:
                    tokens[u] = tokens[v]
                tokens[v] = g[j - 1]
        out = o.step(tokens, parents, c1.k, c1.l)
        o.commit(out["path"])
        emitted += out["accepted"].tolist()
        accs.append(out["n_accepted"] - 1)
        tokens = out["next_tokens"].copy()
    return emitted, accs, D


def test_p4_lossless_and_p6_cache_and_p7_forced(c1, c1_weights, hf):
    prompt = si.prompt(c1)
    want = hf_greedy(hf, prompt, 70)
    for forced in (False, True):
        o = fresh(c1, c1_weights)
        emitted, accs, D = run_free(o, c1, prompt, 16, forced)
        assert emitted == want[: len(emitted)]                       # P4 (Eq. 1)
        if forced:
            assert accs == [D] * 16 and len(emitted) == 1 + 16 * (D + 1)   # P7
        # P6: committed cache == from-scratch keys/values over the committed tokens
        n = o.context_len()
        committed = list(prompt) + emitted[: n - prompt.size]
        assert len(committed) == n
        ks, vs = hf_kv(hf, committed)
        for layer in range(c1.L):
            for slot in (0, prompt.size - 1, prompt.size, n - 2, n - 1):
                assert np.abs(o.read_cache(0, layer, 0, slot) - ks[layer][slot]).max() < 1e-5
                assert np.abs(o.read_cache(0, layer, 1, slot) - vs[layer][slot]).max() < 1e-5


def test_p4_lossless_with_arbitrary_trees(c1, c1_weights, hf):
    # any tree contents give the same stream: random tokens, random shapes
    prompt = si.prompt(c1, length=11)
    want = hf_greedy(hf, prompt, 14)
    o = fresh(c1, c1_weights)
    r = o.prefill(prompt, 3, 1, si.tree_template(8))
    emitted, root = [r["root"]], r["root"]
    for step in range(6):
        T = 4 + step
        parents = si.random_tree(3, T, 3, step)
        tokens = si.random_tokens(c1, T, 50 + step)
        tokens[0] = root
        if step % 2 == 0:            # plant the true next token on a child of the root
            tokens[1] = want[len(emitted)]
        out = o.step(tokens, parents, 3, 1)
        o.commit(out["path"])
        emitted += out["accepted"].tolist()
        root = int(out["accepted"][-1])
    assert emitted == want[: len(emitted)]
    assert len(emitted) > 7                                       # the planted tokens were accepted


# ---------------------------------------------------------------- bf16 cache storage
def test_bf16_cache_mode_stores_rounded_keys_and_values(c1, c1_weights, hf):
    """With the bf16 cache, stored rows are exactly bf16 numbers, lie within one bf16 ulp of the
    fp64 decoder's keys/values, the emitted stream is still the greedy stream of Eq. 1 whenever
    the fp64 decoder's top-2 margin is clear, and logits move by far less than the margins."""
    prompt = si.prompt(c1)
    o = fresh(c1, c1_weights, kv_bf16=True)
    emitted, accs, D = run_free(o, c1, prompt, 8, forced=False)
    n = o.context_len()
    committed = list(prompt) + emitted[: n - prompt.size]
    ks, vs = hf_kv(hf, committed)
    for layer in range(c1.L):
        for slot in (0, 7, prompt.size, n - 1):
            for which, ref in ((0, ks), (1, vs)):
                row = o.read_cache(0, layer, which, slot)
                assert not (row.view(np.uint32) & 0xFFFF).any()                 # representable in bf16
                if layer == 0:     # layer-0 keys/values depend on the embeddings only: one rounding apart
                    ulp = np.maximum(np.abs(ref[layer][slot]), 1e-30) * 2.0 ** -8
                    assert (np.abs(row - ref[layer][slot]) <= ulp).all()
                else:              # deeper layers also see the rounded rows of the layers below
                    assert np.abs(row - ref[layer][slot]).max() <= 2e-2 * np.abs(ref[layer][slot]).max()
    want = hf_greedy(hf, prompt, len(emitted))
    ids = list(prompt)
    for i, t in enumerate(emitted):
        lg = hf_logits(hf, ids)[-1]
        top2 = np.sort(lg)[-2:]
        if top2[1] - top2[0] > 0.02:
            assert t == want[i] == int(lg.argmax())
        ids.append(t)
    # same tree, both cache modes: logits differ by rounding noise only
    a, b = fresh(c1, c1_weights, kv_bf16=False), fresh(c1, c1_weights, kv_bf16=True)
    tokens, parents = si.random_tokens(c1, 8, 4), si.tree_template(8)
    for orc in (a, b):
        orc.prefill(prompt, 0, 0, None)
    la, lb = a.forward(tokens, parents, 3, 1)["logits"], b.forward(tokens, parents, 3, 1)["logits"]
    assert 0 < np.abs(la - lb).max() < 2e-2


# ---------------------------------------------------------------- hand-worked verification / next tree
def test_verify_walk_and_ties_hand_example(c1, c1_weights):
    o = fresh(c1, c1_weights)
    V = c1.V
    parents = np.array([-1, 0, 0, 1, 1, 2], np.int32)
    tokens = np.array([9, 5, 5, 7, 3, 7], np.int32)     # duplicate sibling token 5 on nodes 1 and 2
    lg = np.zeros((6, V), np.float32)
    lg[0, 5] = 1.0; lg[0, 900] = 1.0                     # tie 5 vs 900 -> lowest id 5
    lg[1, 3] = 2.0; lg[1, 7] = 1.5                       # node 1 wants 3 -> child 4
    lg[4, 11] = 4.0                                      # bonus 11
    lg[2, 7] = 9.0                                       # never reached: node 1 (lower index) wins the duplicate
    r = o.verify(lg, tokens, parents)
    assert r["best"].tolist()[:2] == [5, 3] and r["best"][4] == 11
    assert r["path"].tolist() == [0, 1, 4] and r["accepted"].tolist() == [5, 3, 11] and r["n_accepted"] == 3
    lg[0, 900] = 1.5                                     # now the root wants 900: nothing accepted
    r = o.verify(lg, tokens, parents)
    assert r["path"].tolist() == [0] and r["accepted"].tolist() == [900]


def test_next_tree_hand_example(c1, c1_weights):
    o = fresh(c1, c1_weights)
    V, T, k = c1.V, 2, 3
    lg = np.zeros((T + k, V), np.float32)
    lg[2, [10, 20, 30]] = [3.0, 2.0, 2.0]                # depth-1 list: 10, 20, 30 (tie -> lower id first)
    lg[3, [40, 41]] = [1.0, 5.0]                          # depth-2 list: 41, 40
    lg[4, 77] = 1.0                                       # depth-3 list: 77, then zeros by ascending id: 0, 1, ...
    parents = si.tree_template(8)                         # depths 0 1 2 3 1 2 2 3, ranks 0 0 0 0 1 1 0 0
    r = o.next_tree(lg, T, k, bonus=99, next_parents=parents)
    assert r["topb_ids"][0, :3].tolist() == [10, 20, 30] and r["topb_ids"][1, :2].tolist() == [41, 40]
    assert r["topb_ids"][2, :3].tolist() == [77, 0, 1]
    assert r["topb_ids"][0, 3:].tolist() == [0, 1, 2, 3, 4]
    assert r["next_tokens"].tolist() == [99, 10, 41, 77, 20, 40, 41, 77]
    with pytest.raises(ValueError):                       # a template deeper than k cannot be filled
        o.next_tree(lg, T, 2, 99, parents)


# ---------------------------------------------------------------- P9
def test_p9_predictor_size_matches_paper_table1():
    with open(os.path.join(GOLDEN, "paper_table1_draft_module_params.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for name, d, k, billions in rows:
        n_params = int(k) * int(d) ** 2
        assert round(n_params / 1e9, 2) == float(billions), name
    assert 3 * si.CONFIGS["c2"].d ** 2 == 50331648 and 3 * si.CONFIGS["c3"].d ** 2 == 78643200


# ---------------------------------------------------------------- RMSNorm gains and grouped-query attention
# The workload configurations have unit gains and (on the tiny shape) as many key/value heads as query heads,
# which would leave the gain factor, the routing of the three gain vectors and the query-head -> kv-head map
# pinned by nothing.  These variants repeat P1, P2, P6 and P8 against the library decoder (the architecture of
# Section 4 "Setup": learned gains in every RMSNorm; grouped-query attention in the larger models).
VARIANTS = {
    "gains": (dict(), True),              # three different seeded gain vectors per layer kind
    "gqa2": (dict(Hkv=2), False),         # 4 query heads on 2 key/value heads
    "gqa1": (dict(Hkv=1), True),          # multi-query, and gains on top
}


@pytest.fixture(scope="module", params=sorted(VARIANTS))
def variant(request):
    over, gains = VARIANTS[request.param]
    shape = si.scaled(si.CONFIGS["c1"], **over)
    weights = si.all_weights(shape, gains=gains)
    return shape, weights, build_hf_llama(shape, weights)


def test_variants_p1_p2_p6_against_the_library_decoder(variant):
    shape, weights, hfv = variant
    prompt = si.prompt(shape, length=19)
    o = fresh(shape, weights)
    r = o.prefill(prompt, 0, 0, None)
    # P1: T = 1, k = 0 stepping is cache-free greedy decoding
    want = hf_greedy(hfv, prompt, 6)
    got, tok, ids = [r["root"]], r["root"], list(prompt)
    one = np.array([-1], np.int32)
    for _ in range(5):
        out = o.step([tok], one, 0, 0)
        ids.append(tok)
        assert np.abs(out["logits"][0] - hf_logits(hfv, ids)[-1]).max() < 1e-5
        o.commit([0])
        tok = int(out["accepted"][0])
        got.append(tok)
    assert got == want
    # P6: the committed cache rows are the keys/values of a from-scratch forward (pins the kv-head layout)
    n = o.context_len()
    ks, vs = hf_kv(hfv, ids)
    for layer in range(shape.L):
        for slot in (0, prompt.size, n - 1):
            assert np.abs(o.read_cache(0, layer, 0, slot) - ks[layer][slot]).max() < 1e-5
            assert np.abs(o.read_cache(0, layer, 1, slot) - vs[layer][slot]).max() < 1e-5
    # P2: every row of a random tree is a causal forward over prefix + its root path
    T = 11
    parents = si.random_tree(5, T, 3, 2)
    tokens = si.random_tokens(shape, T, 3)
    out = o.forward(tokens, parents, 3, 1)
    for v in range(T):
        ref = hf_logits(hfv, ids + [int(tokens[u]) for u in path_to(parents, v)])[-1]
        assert np.abs(out["logits"][v] - ref).max() < 1e-5, v


def test_variants_p8_pseudo_chain(variant):
    shape, weights, hfv = variant
    k, l = 3, 1
    prompt = si.prompt(shape, length=14)
    Wf = si.bf16_bits_to_f32(weights["pred_w"]).astype(np.float64)
    bf = np.zeros((k, shape.d))
    o = fresh(shape, weights)
    o.forward(prompt, si.chain_template(prompt.size), 0, 0)
    o.commit(np.arange(prompt.size))
    tokens, parents = si.random_tokens(shape, 8, 9), si.tree_template(8)
    out = o.forward(tokens, parents, k, l, anchor=0)
    ids = list(prompt) + [int(tokens[0])] + [0] * k
    ref = hf_logits_with_replaced_rows(hfv, ids, l, prompt.size + 1, list(Wf), list(bf), prompt.size)
    assert np.abs(out["logits"][8:] - ref[prompt.size + 1:]).max() < 1e-5


def test_gain_vectors_differ_and_matter(c1):
    """The variant really exercises the gains: the three kinds differ, and the logits move with them."""
    w = si.all_weights(c1, gains=True)
    g = [si.bf16_bits_to_f32(w["layers"][0]["g_attn"]), si.bf16_bits_to_f32(w["layers"][0]["g_mlp"]),
         si.bf16_bits_to_f32(w["g_final"]), si.bf16_bits_to_f32(w["layers"][1]["g_attn"])]
    for i in range(4):
        assert np.abs(g[i] - 1).max() > 0.3
        for j in range(i):
            assert np.abs(g[i] - g[j]).max() > 0.3
    a, b = fresh(c1, w), fresh(c1, si.all_weights(c1))
    la = a.forward(si.prompt(c1, length=5), si.chain_template(5), 0, 0)["logits"]
    lb = b.forward(si.prompt(c1, length=5), si.chain_template(5), 0, 0)["logits"]
    assert np.abs(la - lb).max() > 0.05


# ---------------------------------------------------------------- P13: Eq. 3 on the normalised state (variant)
@pytest.mark.parametrize("layers", [1, (0, 1, 1)])
def test_p13_prenorm_variant_reads_the_anchor_through_the_layers_input_norm(variant, layers):
    """The variant of Eq. 3 that feeds the map the anchor's state after the input RMSNorm of the insertion layer:
    the chain == a library forward whose rows are replaced by W_i input_layernorm(h[anchor]) + b_i (the library's
    own norm module, with non-unit gains in two of the three shapes); the tree rows do not change; and the
    default (raw residual) differs from it."""
    shape, weights, hfv = variant
    k = 3
    prompt = si.prompt(shape, length=12)
    Wf = si.bf16_bits_to_f32(weights["pred_w"]).astype(np.float64)
    bf = np.zeros((k, shape.d))
    o = oracle.Oracle(shape, weights, max_ctx=64, kv_bf16=False, prenorm=True)
    plain = fresh(shape, weights, max_ctx=64)
    for orc in (o, plain):
        orc.forward(prompt, si.chain_template(prompt.size), 0, 0)
        orc.commit(np.arange(prompt.size))
    tokens, parents = si.random_tokens(shape, 8, 9), si.tree_template(8)
    l = layers if np.isscalar(layers) else list(layers)
    out, ref_out = o.forward(tokens, parents, k, l, anchor=0), plain.forward(tokens, parents, k, l, anchor=0)
    ids = list(prompt) + [int(tokens[0])] + [0] * k
    ref = hf_logits_with_replaced_rows(hfv, ids, layers, prompt.size + 1, list(Wf), list(bf), prompt.size, prenorm=True)
    assert np.abs(out["logits"][8:] - ref[prompt.size + 1:]).max() < 1e-5
    assert np.array_equal(out["logits"][:8], ref_out["logits"][:8])
    assert np.abs(out["logits"][8:] - ref_out["logits"][8:]).max() > 1e-3
