"""Lock-step parity harness: the CUDA path (through the C ABI) against the CPU oracle.

Each step both sides get the same tree on the same committed state.  Compared:
  * depth and ancestor mask of every row: bit-exact;
  * logits of all T+k rows: max-abs <= 3e-2 and max-abs / max|oracle row| <= 2e-2;
  * greedy token of a tree row: exact where the oracle's top-2 margin exceeds 0.1;
  * accepted path / tokens / count: exact when every row on the oracle's path has such a margin
    (otherwise the step is counted as ambiguous);
  * the walk and the next tree as integer functions of the CUDA path's own argmax / top-B: exact
    (re-derived with the oracle's walk on one-hot logits and with the template);
  * top-B ids: exact at positions whose neighbouring oracle gaps exceed 0.1; values within tolerance;
  * cache rows after the commit: equal to the oracle's within bf16 rounding.
Then both sides commit the ORACLE's path and take the ORACLE's next tree, so a near-tie never cascades.
"""
from __future__ import annotations

import numpy as np

import oracle
import synth_inputs as si

ABS_TOL, REL_TOL, MARGIN = 3e-2, 2e-2, 0.1


def unpack_mask(words: np.ndarray, M: int) -> np.ndarray:
    """[M][ceil(M/32)] uint32 words -> dense [M][M] 0/1."""
    w = words.astype(np.uint32)
    out = np.zeros((M, M), np.uint8)
    for u in range(M):
        out[:, u] = (w[:, u >> 5] >> np.uint32(u & 31)) & 1
    return out


def principal_chain(parents, depth):
    chain = [0]
    for _ in range(int(depth.max())):
        kids = [u for u in range(len(parents)) if parents[u] == chain[-1]]
        if not kids:
            break
        chain.append(min(kids))
    return chain


def template_next(parents, tp, topb_ids, bonus, k):
    nxt = np.zeros(len(parents), np.int32)
    nxt[0] = bonus
    for v in range(1, len(parents)):
        nxt[v] = topb_ids[tp["depth"][v] - 1][tp["rank"][v]]
    return nxt if k > 0 else np.array([bonus], np.int32)


class Stats:
    def __init__(self):
        self.steps = self.ambiguous = self.rows = self.rows_margin = 0
        self.max_abs = self.max_rel = 0.0
        self.emitted = 0
        self.unsynced_max_abs = None     # deviation of a step on the engine's own prefilled cache (see lockstep_run)

    def as_dict(self):
        return dict(steps=self.steps, ambiguous_steps=self.ambiguous, rows=self.rows, rows_with_margin=self.rows_margin,
                    max_abs=self.max_abs, max_rel=self.max_rel, emitted=self.emitted,
                    unsynced_max_abs=self.unsynced_max_abs)


def compare_step(shape, parents, tokens, k, g, ref, stats: Stats, tp=None, abs_tol=None, chains=False):
    """g: dict of numpy arrays from the CUDA path for ONE sequence; ref: oracle.step() output
    (oracle.step_chains() with chains=True: a chain of k pseudo rows under every node, the candidates
    are those of the chain under the node the walk ended on)."""
    abs_tol = ABS_TOL if abs_tol is None else abs_tol
    T, V = len(parents), shape.V
    M = T * (1 + k) if chains else T + k
    tp = tp or (oracle.tree_prep_chains(parents, k) if chains else oracle.tree_prep(parents, k, 0))
    # (i) integer bookkeeping
    assert np.array_equal(g["depth"], ref["depth"]), "depth mismatch"
    assert np.array_equal(unpack_mask(g["mask"], M), ref["mask"]), "tree mask mismatch"
    # (ii) logits
    d = np.abs(g["logits"].astype(np.float64) - ref["logits"].astype(np.float64))
    row_abs = d.max(axis=1)
    row_rel = row_abs / np.abs(ref["logits"]).max(axis=1)
    stats.max_abs = max(stats.max_abs, float(row_abs.max()))
    stats.max_rel = max(stats.max_rel, float(row_rel.max()))
    assert row_abs.max() <= abs_tol, "logits max-abs %.4g > %.3g (row %d)" % (row_abs.max(), abs_tol, row_abs.argmax())
    assert row_rel.max() <= REL_TOL, "logits rel %.4g > %.3g" % (row_rel.max(), REL_TOL)
    # (iii) greedy tokens where the oracle margin is clear
    part = np.partition(ref["logits"][:T], V - 2, axis=1)
    margin = part[:, V - 1] - part[:, V - 2]
    clear = margin > MARGIN
    stats.rows += T
    stats.rows_margin += int(clear.sum())
    assert np.array_equal(g["best"][clear], ref["best"][clear]), "argmax mismatch on a clear-margin row"
    # (iv) acceptance
    n_ref = ref["n_accepted"]
    decisive = all(clear[v] for v in ref["path"])
    if decisive:
        assert g["n_accepted"] == n_ref, "accepted count %d != %d" % (g["n_accepted"], n_ref)
        assert np.array_equal(g["path"][:n_ref], ref["path"]), "path mismatch"
        assert np.array_equal(g["accepted"][:n_ref], ref["accepted"]), "accepted tokens mismatch"
    else:
        stats.ambiguous += 1
    # the walk as an integer function of the CUDA path's own argmax
    onehot = np.zeros((T, V), np.float32)
    onehot[np.arange(T), g["best"]] = 1.0
    o = oracle.verify(onehot, tokens, parents)
    ng = int(g["n_accepted"])
    assert ng == o["n_accepted"] and np.array_equal(g["path"][:ng], o["path"]) and \
        np.array_equal(g["accepted"][:ng], o["accepted"]), "acceptance walk is not the walk of its own argmax"
    # (v) top-B of the pseudo rows (of the chain under the CUDA path's own end node; compared with the
    # oracle's values of the same rows, which are its candidates too whenever the walks agree)
    g_end = int(g["path"][ng - 1])
    prow = (lambda i: oracle.chain_row(T, g_end, i + 1)) if chains else (lambda i: T + i)
    if k > 0:
        B = g["topb_ids"].shape[1]
        for i in range(k):
            row = ref["logits"][prow(i)]
            order = np.lexsort((np.arange(V), -row))[: B + 1]
            vals = row[order]
            gaps = vals[:-1] - vals[1:]                      # gap after position b
            for b in range(B):
                firm = gaps[b] > MARGIN and (b == 0 or gaps[b - 1] > MARGIN)
                if firm:
                    assert g["topb_ids"][i, b] == order[b], "top-B id mismatch at a firm position"
                gid = int(g["topb_ids"][i, b])
                assert abs(float(g["topb_vals"][i, b]) - float(row[gid])) <= abs_tol, "top-B value off"
                assert float(g["topb_vals"][i, b]) >= float(vals[B - 1]) - 2 * abs_tol, "top-B entry too small"
            gv, gi = g["topb_vals"][i], g["topb_ids"][i]
            assert all(gv[b] > gv[b + 1] or (gv[b] == gv[b + 1] and gi[b] < gi[b + 1]) for b in range(B - 1)), \
                "top-B not ordered by (value desc, id asc)"
            assert np.array_equal(g["topb_ids"][i], np.lexsort((np.arange(V), -g["logits"][prow(i)]))[:B]), \
                "top-B is not the top-B of the CUDA path's own logits"
    # next tree as an integer function of the CUDA path's own top-B and bonus
    want_next = template_next(parents, tp, g["topb_ids"], int(g["accepted"][ng - 1]), k)
    assert np.array_equal(g["next_tokens"][: want_next.size], want_next), "next tree is not the template of its own top-B"
    assert np.array_equal(g["best"], g["logits"][:T].argmax(axis=1)), "best is not the argmax of the CUDA path's own logits"
    stats.steps += 1


def gpu_outputs(out, s, T, k):
    """Slice sequence s of a StepOut into numpy arrays (synchronises)."""
    n_acc = int(out.n_accepted[s].item())
    return dict(depth=out.depth[s].cpu().numpy(), mask=out.mask[s].cpu().numpy().view(np.uint32),
                logits=out.logits[s].cpu().numpy(), best=out.best[s].cpu().numpy(), n_accepted=n_acc,
                path=out.path[s].cpu().numpy(), accepted=out.accepted_tokens[s].cpu().numpy(),
                topb_ids=out.topb_ids[s, :k].cpu().numpy(), topb_vals=out.topb_vals[s, :k].cpu().numpy(),
                next_tokens=out.next_tree_tokens[s].cpu().numpy())


def cache_row(engine, seq, pos):
    """Row of cache position `pos` of slot `seq` inside a (layer, K|V) plane: contiguous, or through the page table
    the engine was given (64 positions per page)."""
    table = getattr(engine, "page_table", None)
    if table is None:
        return seq * engine.cfg.max_ctx + pos
    return int(table[seq, pos // 64]) * 64 + pos % 64


def own_tree_view(g, Ts, T, k):
    """Outputs of a sequence whose own tree has Ts of the T tree rows (firp_step_trees): drop the padding rows
    Ts..T-1 so that the rows are those of an oracle step on the Ts-node tree (tree rows, then the k pseudo rows)."""
    keep = list(range(Ts)) + list(range(T, T + k))
    dense = unpack_mask(g["mask"], T + k)[np.ix_(keep, keep)]
    words = np.zeros((len(keep), (len(keep) + 31) // 32), np.uint32)
    for u in range(len(keep)):
        words[:, u >> 5] |= dense[:, u].astype(np.uint32) << np.uint32(u & 31)
    out = dict(g)
    out.update(depth=g["depth"][keep], mask=words, logits=g["logits"][keep], best=g["best"][:Ts],
               next_tokens=g["next_tokens"][:Ts])
    return out


def read_gpu_cache(engine, seq, layer, which, slot):
    import torch
    s = engine.shape
    cfg = engine.cfg
    kvt = engine.kv.view(torch.bfloat16)
    off = ((layer * 2 + which) * cfg.max_batch * cfg.max_ctx + cache_row(engine, seq, slot)) * s.n_kv
    return kvt[off: off + s.n_kv].float().cpu().numpy()


def check_cache(engine, orc, seq, slots, layers, tol=2e-2):
    for layer in layers:
        for which in (0, 1):
            for slot in slots:
                a = read_gpu_cache(engine, seq, layer, which, slot)
                b = orc.read_cache(seq, layer, which, slot)
                scale = max(1.0, float(np.abs(b).max()))
                assert np.abs(a - b).max() <= tol * scale, "cache row %d layer %d differs" % (slot, layer)


def write_gpu_cache(engine, seq, layer, which, slot0, rows_bits):
    """Copy bf16 bit patterns [count, Hkv*dh] into the engine's cache tensor at positions slot0.. of one
    layer (which: 0 keys, 1 values): plain data movement through torch, no kernel of the library."""
    import torch
    s, cfg = engine.shape, engine.cfg
    kvt = engine.kv.view(torch.int16)
    src = torch.from_numpy(np.ascontiguousarray(rows_bits, np.uint16).view(np.int16)).to(engine.device)
    count = src.shape[0]
    plane0 = (layer * 2 + which) * cfg.max_batch * cfg.max_ctx
    if getattr(engine, "page_table", None) is None:          # contiguous rows
        off = (plane0 + seq * cfg.max_ctx + slot0) * s.n_kv
        kvt[off: off + src.numel()].copy_(src.reshape(-1))
    else:                                                     # scattered through the page table, page by page
        pos = slot0
        while pos < slot0 + count:
            n = min(64 - pos % 64, slot0 + count - pos)
            off = (plane0 + cache_row(engine, seq, pos)) * s.n_kv
            kvt[off: off + n * s.n_kv].copy_(src[pos - slot0: pos - slot0 + n].reshape(-1))
            pos += n


def seed_prefix(engine, orc, shape, seq, n):
    """Give both sides the same committed prefix of n positions WITHOUT a prefill: seeded bf16 key and value rows
    (synth_inputs.cache_rows; N(0, (0.02 sqrt(d))^2), the spread the projections of a unit-RMS row have) are written
    bit for bit into both caches and both committed lengths are set to n.  The oracle's cost per step is then
    linear in n, which is what makes the long contexts checkable against it."""
    std = 0.02 * float(np.sqrt(shape.d))
    for layer in range(shape.L):
        ks, vs = si.cache_rows(shape, seq, layer, n, std, std)
        for which, rows in ((0, ks), (1, vs)):
            orc.write_cache(seq, layer, which, 0, rows)
            write_gpu_cache(engine, seq, layer, which, 0, rows)
    orc.set_context_len(seq, n)
    engine.set_context_len(seq, n)


def sync_prefix_from_oracle(engine, orc, shape, seq, n, sample=12):
    """After both sides have prefilled the same prompt: check the engine's cache rows against the oracle's at
    sampled positions (first and last layer), then overwrite the engine's n prefix rows with the oracle's, bit for
    bit.  Both caches hold bf16, and a key or value whose fp32 pre-image sits next to a rounding boundary may round
    differently on the two sides; over hundreds of rows and tens of layers those one-ulp differences add up to
    logit noise of the size of the parity bound itself, which says nothing about either implementation.  With the
    prefix synchronised, a step is compared on the same committed state, as the lock-step protocol asks."""
    slots = sorted(set(np.linspace(0, n - 1, num=min(sample, n)).astype(int).tolist()))
    check_cache(engine, orc, seq, slots, sorted({0, shape.L - 1}))
    for layer in range(shape.L):
        for which in (0, 1):
            rows = np.stack([orc.read_cache(seq, layer, which, slot) for slot in range(n)])
            bits = (rows.view(np.uint32) >> 16).astype(np.uint16)
            assert not (rows.view(np.uint32) & 0xFFFF).any(), "the oracle's cache rows are not bf16 values"
            write_gpu_cache(engine, seq, layer, which, 0, bits)


def lockstep_run(engine, orc, shape, parents, prompt, steps, forced=False, k=None, l=None, check_cache_rows=True,
                 compare_every=1, seq=0, abs_tol=None, chains=False, forced_steps=(), sync_prefix=False):
    """Prefill both sides, then `steps` lock-step steps (chains: with a chain of k pseudo rows under
    every tree node, firp_step_chains against oracle.step_chains).  sync_prefix: after the prefill has been
    checked (logits, sampled cache rows), one un-synchronised step is compared at twice the bound and its
    deviation reported in Stats.unsynced_max_abs, then the engine's prefix rows are replaced by the oracle's
    (sync_prefix_from_oracle) before the asserted steps.  Returns a Stats."""
    abs_tol = ABS_TOL if abs_tol is None else abs_tol
    import torch
    k = shape.k if k is None else k
    l = shape.l if l is None else l
    T = len(parents)
    dev = engine.device

    # prefill
    d_prompt = torch.from_numpy(np.ascontiguousarray(prompt, np.int32)).to(dev)
    pout = engine.new_out(1, 1, k, T_next=T if k > 0 else 1)
    engine.prefill(seq, d_prompt, k, l, parents if k > 0 else None, pout)
    ref = orc.prefill(prompt, k, l, parents, seq=seq)
    torch.cuda.synchronize()
    plog = pout.logits[0].cpu().numpy()
    dd = np.abs(plog - ref["logits"]).max()
    assert dd <= abs_tol, "prefill logits differ by %.4g" % dd
    part = np.partition(ref["logits"][0], shape.V - 2)
    if part[-1] - part[-2] > MARGIN:
        assert int(pout.accepted_tokens[0, 0].item()) == ref["root"], "prefill root token differs"
    assert engine.context_len(seq) == orc.context_len(seq) == len(prompt)
    unsynced = None
    if sync_prefix:
        n = len(prompt)
        probe = lockstep_steps(engine, orc, shape, parents, ref["next_tokens"].copy(), 1, k=k, l=l, check_cache_rows=False,
                               seq=seq, abs_tol=2 * abs_tol, chains=chains)
        unsynced = probe.max_abs
        orc.set_context_len(seq, n)
        engine.set_context_len(seq, n)
        sync_prefix_from_oracle(engine, orc, shape, seq, n)
    stats = lockstep_steps(engine, orc, shape, parents, ref["next_tokens"].copy(), steps, forced=forced, k=k, l=l,
                           check_cache_rows=check_cache_rows, compare_every=compare_every, seq=seq, abs_tol=abs_tol,
                           chains=chains, forced_steps=forced_steps)
    stats.emitted += 1
    stats.unsynced_max_abs = unsynced
    return stats


def lockstep_steps(engine, orc, shape, parents, tokens, steps, forced=False, k=None, l=None, check_cache_rows=True,
                   compare_every=1, seq=0, abs_tol=None, chains=False, forced_steps=(), device_commit=False):
    """`steps` lock-step steps from the committed state both sides are in, starting with the tree `tokens`.
    forced / forced_steps: all steps, or the listed ones, run in forced-accept mode (the oracle's own greedy
    continuation is planted on the principal chain, so the full depth is accepted and the commit compacts a real
    path).  device_commit: the engine commits the path its own walk found (path = NULL) instead of being told the
    oracle's; this requires a decisive step, and the committed cache rows are compared like any other."""
    abs_tol = ABS_TOL if abs_tol is None else abs_tol
    import torch
    k = shape.k if k is None else k
    l = shape.l if l is None else l
    T = len(parents)
    tp = oracle.tree_prep_chains(parents, k) if chains else oracle.tree_prep(parents, k, 0)
    tp_tree = oracle.tree_prep(parents, 0, 0)
    chain = principal_chain(parents, tp_tree["depth"])
    D = len(chain) - 1        # forced steps plant the greedy continuation on the principal chain (which may end above the deepest node)
    dev = engine.device
    stats = Stats()
    tokens = np.array(tokens, np.int32)
    emitted = []

    out = engine.new_out(1, T, k, chains=chains)
    for step in range(steps):
        force_now = forced or step in forced_steps
        if force_now:
            gcont = orc.ar_greedy(int(tokens[0]), D, seq=seq)
            for j in range(1, D + 1):
                v = chain[j]
                for u in range(T):
                    if parents[u] == parents[v] and u != v and tokens[u] == gcont[j - 1]:
                        tokens[u] = tokens[v]
                tokens[v] = gcont[j - 1]
        d_tokens = torch.from_numpy(np.ascontiguousarray(tokens, np.int32)).to(dev)
        if chains:
            engine.step_chains(d_tokens, parents, k, l, out, seq_ids=[seq])
            ref = orc.step_chains(tokens, parents, k, l, seq=seq)
        else:
            engine.step(d_tokens, parents, k, l, out, seq_ids=[seq])
            ref = orc.step(tokens, parents, k, l, seq=seq)
        g = None
        if step % compare_every == 0 or step == steps - 1 or device_commit:
            g = gpu_outputs(out, 0, T, k)
            compare_step(shape, parents, tokens, k, g, ref, stats, tp, abs_tol, chains=chains)
        if force_now:
            assert ref["n_accepted"] == D + 1, "forced-accept step accepted %d of %d" % (ref["n_accepted"] - 1, D)
        n0 = orc.context_len(seq)
        if device_commit:
            assert g["n_accepted"] == ref["n_accepted"] and np.array_equal(g["path"][: ref["n_accepted"]], ref["path"]), \
                "the device-side commit needs a step on which both walks agree"
            engine.commit(1, seq_ids=[seq])
        else:
            engine.commit(1, seq_ids=[seq], path=[ref["path"]])
        orc.commit(ref["path"], seq=seq)
        n1 = orc.context_len(seq)
        assert engine.context_len(seq) == n1
        if check_cache_rows:
            check_cache(engine, orc, seq, range(n0, n1), sorted({0, shape.L - 1}))
        emitted += ref["accepted"].tolist()
        tokens = ref["next_tokens"].copy()
    stats.emitted = len(emitted)
    return stats


def lockstep_run_batch(engine, orc, shape, parents, prompts, steps, k=None, l=None, abs_tol=None):
    """Several sequences with their own prompts (context lengths) and trees, stepped together by ONE
    firp_step call per step; every sequence is compared with its own oracle step, and both sides commit
    the oracle's paths.  Returns a Stats over all sequences."""
    import torch
    k = shape.k if k is None else k
    l = shape.l if l is None else l
    abs_tol = ABS_TOL if abs_tol is None else abs_tol
    T, n_seq = len(parents), len(prompts)
    dev = engine.device
    tokens = np.zeros((n_seq, T), np.int32)
    for s_i, prompt in enumerate(prompts):
        pout = engine.new_out(1, 1, k, T_next=T)
        engine.prefill(s_i, torch.from_numpy(np.ascontiguousarray(prompt, np.int32)).to(dev), k, l, parents, pout)
        ref = orc.prefill(prompt, k, l, parents, seq=s_i)
        torch.cuda.synchronize()
        dd = np.abs(pout.logits[0].cpu().numpy() - ref["logits"]).max()
        assert dd <= abs_tol, "prefill logits of sequence %d differ by %.4g" % (s_i, dd)
        assert engine.context_len(s_i) == orc.context_len(s_i) == len(prompt)
        tokens[s_i] = ref["next_tokens"]
    return lockstep_steps_batch(engine, orc, shape, parents, tokens, steps, k=k, l=l, abs_tol=abs_tol)


def lockstep_steps_batch(engine, orc, shape, parents, tokens, steps, k=None, l=None, abs_tol=None, check_cache_rows=False):
    """`steps` lock-step steps of n_seq sequences (tokens [n_seq, T]) from the committed state both sides are in."""
    import torch
    k = shape.k if k is None else k
    l = shape.l if l is None else l
    abs_tol = ABS_TOL if abs_tol is None else abs_tol
    tokens = np.array(tokens, np.int32)
    n_seq, T = tokens.shape
    tp = oracle.tree_prep(parents, k, 0)
    dev = engine.device
    stats = Stats()
    out = engine.new_out(n_seq, T, k)
    for step in range(steps):
        d_tokens = torch.from_numpy(np.ascontiguousarray(tokens)).to(dev)
        engine.step(d_tokens, parents, k, l, out, seq_ids=list(range(n_seq)), n_seq=n_seq)
        refs = [orc.step(tokens[s_i], parents, k, l, seq=s_i) for s_i in range(n_seq)]
        for s_i in range(n_seq):
            compare_step(shape, parents, tokens[s_i], k, gpu_outputs(out, s_i, T, k), refs[s_i], stats, tp, abs_tol)
        n0 = [orc.context_len(s_i) for s_i in range(n_seq)]
        engine.commit(n_seq, seq_ids=list(range(n_seq)), path=[r["path"] for r in refs])
        for s_i in range(n_seq):
            orc.commit(refs[s_i]["path"], seq=s_i)
            assert engine.context_len(s_i) == orc.context_len(s_i)
            if check_cache_rows:
                check_cache(engine, orc, s_i, range(n0[s_i], orc.context_len(s_i)), sorted({0, shape.L - 1}))
            stats.emitted += len(refs[s_i]["accepted"])
            tokens[s_i] = refs[s_i]["next_tokens"]
    return stats
