"""CPU oracle of the FIRP draft+verify step -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around firp_oracle.c (the arithmetic lives there, with the
passages of the paper it follows).  Only tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA path never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "firp_oracle.c")
_LIB = os.path.join(_HERE, "_firp_oracle.so")
_lib = None


def compile_source(src: str, out: str) -> str:
    """gcc (OpenMP) a copy of the oracle's C source into the shared object `out`."""
    tmp = out + ".%d.tmp" % os.getpid()
    subprocess.check_call(["gcc", "-O3", "-march=x86-64-v3", "-fopenmp", "-shared", "-fPIC", "-o", tmp, src, "-lm"])
    os.replace(tmp, out)
    return out


def build(force: bool = False) -> str:
    """Compile firp_oracle.c into a shared object next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        compile_source(_SRC, _LIB)
    return _LIB


class _Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("L", "d", "H", "Hkv", "dh", "F", "V", "max_ctx", "n_maps", "n_seq", "kv_bf16")] + \
               [("eps", ctypes.c_float), ("theta", ctypes.c_float)]


_PP = ctypes.POINTER(ctypes.c_void_p)


class _Weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("embed", "lm_head", "g_final", "pred_w", "pred_b")] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "g_attn", "g_mlp")]


def bind(lib):
    """Declare the C signatures on a loaded oracle library (the built one, or a test's altered copy)."""
    i32, vp = ctypes.c_int32, ctypes.c_void_p
    lib.oracle_create.argtypes = [ctypes.POINTER(_Cfg)]
    lib.oracle_create.restype = vp
    lib.oracle_destroy.argtypes = [vp]
    lib.oracle_set_weights.argtypes = [vp, ctypes.POINTER(_Weights)]
    lib.oracle_context_len.argtypes = [vp, i32]
    lib.oracle_context_len.restype = i32
    lib.oracle_set_context_len.argtypes = [vp, i32, i32]
    lib.oracle_tree_prep.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    lib.oracle_tree_prep.restype = i32
    lib.oracle_forward.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.oracle_forward.restype = i32
    lib.oracle_forward_layers.argtypes = [vp, i32, vp, vp, i32, i32, vp, i32, i32, vp, vp, vp, i32, vp, vp]
    lib.oracle_forward_layers.restype = i32
    lib.oracle_forward_chains.argtypes = [vp, i32, vp, vp, i32, i32, vp, i32, vp, vp, vp, vp]
    lib.oracle_forward_chains.restype = i32
    lib.oracle_tree_prep_chains.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    lib.oracle_tree_prep_chains.restype = i32
    lib.oracle_set_masked.argtypes = [vp, i32]
    lib.oracle_set_prenorm.argtypes = [vp, i32]
    lib.oracle_mask_pseudo.argtypes = [vp, i32, i32]
    lib.oracle_verify.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
    lib.oracle_verify.restype = i32
    lib.oracle_next_tree.argtypes = [vp, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp]
    lib.oracle_next_tree.restype = i32
    lib.oracle_commit.argtypes = [vp, i32, vp, i32]
    lib.oracle_commit.restype = i32
    lib.oracle_read_cache.argtypes = [vp, i32, i32, i32, i32, vp]
    lib.oracle_write_cache.argtypes = [vp, i32, i32, i32, i32, i32, vp]
    return lib


def _get_lib():
    global _lib
    if _lib is None:
        _lib = bind(ctypes.CDLL(build()))
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def tree_prep(parents, k: int = 0, anchor: int = 0):
    """depth[T+k], dense mask[(T+k),(T+k)] (1 = visible), rank[T], extended parents[T+k]."""
    parents = _i32(parents)
    T = parents.size
    M = T + k
    ext = np.zeros(M, np.int32); depth = np.zeros(M, np.int32)
    mask = np.zeros((M, M), np.uint8); rank = np.zeros(T, np.int32)
    rc = _get_lib().oracle_tree_prep(_ptr(parents), T, k, anchor, _ptr(ext), _ptr(depth), _ptr(mask), _ptr(rank))
    if rc != 0:
        raise ValueError("malformed tree")
    return dict(ext_parent=ext, depth=depth, mask=mask, rank=rank)


def tree_prep_chains(parents, k: int):
    """The same for a chain of k pseudo rows under every node: M = T*(1+k) rows, chain row i
    (1-based) of node v at row T + (i-1)*T + v."""
    parents = _i32(parents)
    T = parents.size
    M = T * (1 + k)
    ext = np.zeros(M, np.int32); depth = np.zeros(M, np.int32)
    mask = np.zeros((M, M), np.uint8); rank = np.zeros(T, np.int32)
    rc = _get_lib().oracle_tree_prep_chains(_ptr(parents), T, k, _ptr(ext), _ptr(depth), _ptr(mask), _ptr(rank))
    if rc != 0:
        raise ValueError("malformed tree")
    return dict(ext_parent=ext, depth=depth, mask=mask, rank=rank)


def chain_row(T: int, v: int, i: int) -> int:
    """Row of chain step i (1-based) of tree node v in the every-node-chains layout."""
    return T + (i - 1) * T + v


def verify(logits, tokens, parents):
    """Greedy acceptance walk over the tree rows' logits [T][V] (no weights needed)."""
    tokens, parents = _i32(tokens), _i32(parents)
    T = tokens.size
    logits = np.ascontiguousarray(logits, np.float32)
    V = logits.shape[1]
    best = np.zeros(T, np.int32); path = np.zeros(T, np.int32); acc = np.zeros(T, np.int32)
    n_out = _get_lib().oracle_verify(_ptr(logits), _ptr(tokens), _ptr(parents), T, V, _ptr(best), _ptr(path), _ptr(acc))
    return dict(best=best, path=path[:n_out].copy(), accepted=acc[:n_out].copy(), n_accepted=n_out)


def next_tree(logits, T: int, k: int, bonus: int, next_parents, B: int = 8):
    """Top-B of the pseudo rows (rows T..T+k-1 of logits) and the next tree on a template."""
    next_parents = _i32(next_parents)
    logits = np.ascontiguousarray(logits, np.float32)
    V = logits.shape[1]
    ids = np.zeros((max(k, 1), B), np.int32); vals = np.zeros((max(k, 1), B), np.float32)
    nxt = np.zeros(next_parents.size, np.int32)
    rc = _get_lib().oracle_next_tree(_ptr(logits), T, k, V, B, int(bonus), _ptr(next_parents), next_parents.size,
                                     _ptr(ids), _ptr(vals), _ptr(nxt))
    if rc != 0:
        raise ValueError("template deeper than k or wider than B")
    return dict(topb_ids=ids[:k], topb_vals=vals[:k], next_tokens=nxt)


class Oracle:
    """Oracle state for n_seq independent sequences of one decoder shape.

    `weights` is the dict synth_inputs.all_weights() returns (bf16 bits as numpy
    uint16); the arrays are referenced, not copied, and must stay alive.
    kv_bf16: the KV cache stores bf16 (the workload's storage format: keys/values are
    rounded once when stored); False keeps fp32 rows, for comparisons with an fp64 decoder.
    """

    def __init__(self, shape, weights, max_ctx: int, n_seq: int = 1, top_b: int = 8, kv_bf16: bool = True,
                 masked: bool = False, prenorm: bool = False):
        """masked: the "Masked" setting of Section 4.3 (a pseudo row sees no other pseudo row).
        prenorm: Eq. 3 reads the anchor's state through the input RMSNorm of the insertion layer."""
        self.lib = _get_lib()
        self.shape, self.weights, self.top_b = shape, weights, top_b
        s = shape
        n_maps = int(weights["pred_w"].shape[0]) if weights.get("pred_w") is not None else 0
        self.cfg = _Cfg(L=s.L, d=s.d, H=s.H, Hkv=s.Hkv, dh=s.dh, F=s.F, V=s.V, max_ctx=max_ctx,
                        n_maps=n_maps, n_seq=n_seq, kv_bf16=int(kv_bf16), eps=s.eps, theta=s.theta)
        self.h = self.lib.oracle_create(ctypes.byref(self.cfg))
        if not self.h:
            raise MemoryError("oracle cache allocation failed")
        self.max_ctx = max_ctx
        self._keep = []
        w = _Weights()
        for name in ("embed", "lm_head", "g_final"):
            setattr(w, name, _ptr(weights[name]))
        w.pred_w = _ptr(weights["pred_w"]) if n_maps else None
        w.pred_b = _ptr(weights["pred_b"]) if (n_maps and weights.get("pred_b") is not None) else None
        nq, nkv, F = s.n_q, s.n_kv, s.F

        def per_layer(fn):
            views = [np.ascontiguousarray(fn(lw)) for lw in weights["layers"]]
            for v, lw in zip(views, weights["layers"]):
                assert v.dtype == np.uint16
            arr = (ctypes.c_void_p * s.L)(*[v.ctypes.data for v in views])
            self._keep += [views, arr]
            return ctypes.cast(arr, _PP)

        w.wq = per_layer(lambda lw: lw["wqkv"][:nq])
        w.wk = per_layer(lambda lw: lw["wqkv"][nq:nq + nkv])
        w.wv = per_layer(lambda lw: lw["wqkv"][nq + nkv:])
        w.wo = per_layer(lambda lw: lw["wo"])
        w.wgate = per_layer(lambda lw: lw["wgu"][:F])
        w.wup = per_layer(lambda lw: lw["wgu"][F:])
        w.wdown = per_layer(lambda lw: lw["wd"])
        w.g_attn = per_layer(lambda lw: lw["g_attn"])
        w.g_mlp = per_layer(lambda lw: lw["g_mlp"])
        self._w = w
        self.lib.oracle_set_weights(self.h, ctypes.byref(w))
        self.lib.oracle_set_masked(self.h, int(masked))
        self.lib.oracle_set_prenorm(self.h, int(prenorm))

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.oracle_destroy(self.h)
            self.h = None

    # -- state ---------------------------------------------------------------
    def context_len(self, seq: int = 0) -> int:
        return self.lib.oracle_context_len(self.h, seq)

    def set_context_len(self, seq: int, n: int) -> None:
        """Rewind (or reset with n = 0) the committed length; rows >= n become scratch."""
        self.lib.oracle_set_context_len(self.h, seq, n)

    def read_cache(self, seq: int, layer: int, which: int, slot: int) -> np.ndarray:
        out = np.zeros(self.shape.n_kv, np.float32)
        self.lib.oracle_read_cache(self.h, seq, layer, which, slot, _ptr(out))
        return out

    def write_cache(self, seq: int, layer: int, which: int, slot0: int, rows_bf16: np.ndarray) -> None:
        """Overwrite cache rows slot0.. of one layer (which: 0 keys, 1 values) with bf16 bit patterns
        [count, Hkv*dh]: a seeded stand-in for a committed prefix, written into both implementations."""
        rows = np.ascontiguousarray(rows_bf16, dtype=np.uint16)
        assert rows.ndim == 2 and rows.shape[1] == self.shape.n_kv and slot0 + rows.shape[0] <= self.max_ctx
        self.lib.oracle_write_cache(self.h, seq, layer, which, slot0, rows.shape[0], _ptr(rows))

    # -- the step ------------------------------------------------------------
    def forward(self, tokens, parents, k: int, l, anchor: int = 0, seq: int = 0,
                logit_row0: int = 0, want_h_at_l: bool = False):
        """l: one insertion layer for all k prediction steps, or a non-decreasing sequence of k
        layers t_1..t_k (Section 3.3); with a sequence, want_h_at_l returns `h_ins` [k, d], every
        pseudo row as it was appended, instead of the residual stream at one layer."""
        tokens, parents = _i32(tokens), _i32(parents)
        if not np.isscalar(l):
            return self._forward_layers(tokens, parents, k, _i32(l), anchor, seq, logit_row0, want_h_at_l)
        T = tokens.size
        M = T + k
        s = self.shape
        logits = np.zeros((M, s.V), np.float32)
        depth = np.zeros(M, np.int32)
        mask = np.zeros((M, M), np.uint8)
        h_at_l = np.zeros((M, s.d), np.float32) if want_h_at_l else None
        rc = self.lib.oracle_forward(self.h, seq, _ptr(tokens), _ptr(parents), T, k, l, anchor, logit_row0,
                                     _ptr(logits), _ptr(depth), _ptr(mask), _ptr(h_at_l))
        if rc != 0:
            raise ValueError("oracle_forward failed: %d" % rc)
        out = dict(logits=logits, depth=depth, mask=mask, pos=depth + self.context_len(seq))
        if want_h_at_l:
            out["h_at_l"] = h_at_l
        return out

    def _forward_layers(self, tokens, parents, k, layers, anchor, seq, logit_row0, want_h_ins):
        if layers.size != k:
            raise ValueError("need one insertion layer per prediction step")
        T = tokens.size
        M = T + k
        s = self.shape
        logits = np.zeros((M, s.V), np.float32)
        depth = np.zeros(M, np.int32)
        mask = np.zeros((M, M), np.uint8)
        h_ins = np.zeros((k, s.d), np.float32) if want_h_ins else None
        rc = self.lib.oracle_forward_layers(self.h, seq, _ptr(tokens), _ptr(parents), T, k, _ptr(layers), anchor,
                                            logit_row0, _ptr(logits), _ptr(depth), _ptr(mask), -1, None, _ptr(h_ins))
        if rc != 0:
            raise ValueError("oracle_forward_layers failed: %d" % rc)
        out = dict(logits=logits, depth=depth, mask=mask, pos=depth + self.context_len(seq))
        if want_h_ins:
            out["h_ins"] = h_ins
        return out

    def forward_chains(self, tokens, parents, k: int, l, seq: int = 0, logit_row0: int = 0, want_h_ins: bool = False):
        """The step with a chain of k pseudo rows under every tree node (rows as in tree_prep_chains);
        l: one insertion layer or one per prediction step."""
        tokens, parents = _i32(tokens), _i32(parents)
        layers = _i32([l] * k) if np.isscalar(l) else _i32(l)
        if layers.size != k:
            raise ValueError("need one insertion layer per prediction step")
        T = tokens.size
        M = T * (1 + k)
        s = self.shape
        logits = np.zeros((M, s.V), np.float32)
        depth = np.zeros(M, np.int32)
        mask = np.zeros((M, M), np.uint8)
        h_ins = np.zeros((T * k, s.d), np.float32) if want_h_ins else None
        rc = self.lib.oracle_forward_chains(self.h, seq, _ptr(tokens), _ptr(parents), T, k, _ptr(layers), logit_row0,
                                            _ptr(logits), _ptr(depth), _ptr(mask), _ptr(h_ins))
        if rc != 0:
            raise ValueError("oracle_forward_chains failed: %d" % rc)
        out = dict(logits=logits, depth=depth, mask=mask, pos=depth + self.context_len(seq))
        if want_h_ins:
            out["h_ins"] = h_ins
        return out

    def step_chains(self, tokens, parents, k: int, l, seq: int = 0, next_parents=None):
        """Forward with a chain under every node + greedy verification + the next tree read from the
        chain of the node the walk ended on (its row i gives the candidates of depth i).  Does not commit."""
        tokens, parents = _i32(tokens), _i32(parents)
        T = tokens.size
        out = self.forward_chains(tokens, parents, k, l, seq)
        out.update(self.verify(out["logits"][:T], tokens, parents))
        end = int(out["path"][-1])
        bonus = int(out["accepted"][-1])
        rows = [chain_row(T, end, i) for i in range(1, k + 1)]
        picked = np.concatenate([out["logits"][:T], out["logits"][rows]]) if k > 0 else out["logits"][:T]
        if next_parents is None:
            next_parents = parents if k > 0 else np.array([-1], np.int32)
        out.update(self.next_tree(picked, T, k, bonus, next_parents))
        out["end_node"] = end
        return out

    def verify(self, logits, tokens, parents):
        return verify(logits, tokens, parents)

    def next_tree(self, logits, T: int, k: int, bonus: int, next_parents):
        return next_tree(logits, T, k, bonus, next_parents, self.top_b)

    def step(self, tokens, parents, k: int, l: int, seq: int = 0, anchor: int = 0, next_parents=None,
             want_h_at_l: bool = False):
        """Forward + greedy verification + next tree.  Does not commit."""
        tokens, parents = _i32(tokens), _i32(parents)
        T = tokens.size
        out = self.forward(tokens, parents, k, l, anchor, seq, want_h_at_l=want_h_at_l)
        out.update(self.verify(out["logits"][:T], tokens, parents))
        bonus = int(out["accepted"][-1])
        if next_parents is None:
            next_parents = parents if k > 0 else np.array([-1], np.int32)
        out.update(self.next_tree(out["logits"], T, k, bonus, next_parents))
        return out

    def commit(self, path, seq: int = 0) -> None:
        path = _i32(path)
        rc = self.lib.oracle_commit(self.h, seq, _ptr(path), path.size)
        if rc != 0:
            raise ValueError("oracle_commit failed: %d" % rc)

    def prefill(self, prompt, k: int, l: int, next_parents, seq: int = 0):
        """Chain tree over the prompt on an empty cache, anchor = last prompt token
        (the plain 'n + k hidden states' picture of Section 3.2); commits all P rows.
        Returns the first root token and the first draft tree."""
        prompt = _i32(prompt)
        P = prompt.size
        self.set_context_len(seq, 0)
        chain = np.arange(-1, P - 1, dtype=np.int32)
        out = self.forward(prompt, chain, k, l, anchor=P - 1, seq=seq, logit_row0=P - 1)
        root = int(np.argmax(out["logits"][P - 1]))
        self.commit(np.arange(P, dtype=np.int32), seq)
        nt = self.next_tree(out["logits"], P, k, root, next_parents if k > 0 else np.array([-1], np.int32))
        return dict(root=root, logits=out["logits"][P - 1:], **nt)

    def ar_greedy(self, root: int, count: int, seq: int = 0, l: int = 0):
        """Greedy continuation g_1..g_count after the committed tokens + root, by T=1,k=0
        steps; the committed length is restored afterwards."""
        n0 = self.context_len(seq)
        one = np.array([-1], np.int32)
        tok, outs = int(root), []
        for _ in range(count):
            o = self.step(np.array([tok], np.int32), one, 0, l, seq=seq)
            self.commit(np.array([0], np.int32), seq)
            tok = int(o["accepted"][-1])
            outs.append(tok)
        self.set_context_len(seq, n0)
        return np.array(outs, np.int32)
