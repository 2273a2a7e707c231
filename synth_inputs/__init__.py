"""Seeded synthetic inputs for the FIRP draft+verify step.

This module produces *data only*: decoder shapes, bf16 weight tensors, prompts,
context lengths and draft-tree templates.  It contains none of the method's
arithmetic, so both the CPU oracle's tests and the CUDA path may use it without
sharing any computation.

Recipe (all counter-based, see gen.c for the bit-level definition):
  * weight matrices  ~ N(0, std=0.02), rounded once to bf16 (RNE)
  * predictor maps   ~ N(0, variance=1/d)  (std d^-1/2), bias = 0
  * RMSNorm gains    = 1.0 (the workload configurations); `gains=True` draws three kinds of
                       non-unit gains, 1 + 0.25 N(0,1), each from a stream of its own
  * prompts          = uniform token ids in [0, V)
  * tree templates   = the first T nodes of a per-depth-width product tree,
                       ordered by (sum of sibling ranks, depth, rank tuple)
Tensors are returned as numpy uint16 arrays holding bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import itertools
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "_synth_gen.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into a shared object next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _get_lib():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64 = ctypes.c_uint64
        lib.synth_normal_bf16.argtypes = [u64, u64, u64, u64, ctypes.c_double, ctypes.c_void_p]
        lib.synth_normal_bf16.restype = None
        lib.synth_uniform_i32.argtypes = [u64, u64, u64, u64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
        lib.synth_uniform_i32.restype = None
        _lib = lib
    return _lib


# ----------------------------------------------------------------------------
# raw streams
# ----------------------------------------------------------------------------
def normal_bf16(seed: int, stream: int, count: int, std: float, first: int = 0, out: np.ndarray | None = None) -> np.ndarray:
    """bf16 bits of std * N(0,1) for elements [first, first+count) of a stream."""
    if out is None:
        out = np.empty(count, dtype=np.uint16)
    assert out.dtype == np.uint16 and out.size == count and out.flags["C_CONTIGUOUS"]
    _get_lib().synth_normal_bf16(seed, stream, first, count, float(std), out.ctypes.data)
    return out


def uniform_i32(seed: int, stream: int, count: int, lo: int, hi: int, first: int = 0) -> np.ndarray:
    """Uniform int32 in [lo, hi) for elements [first, first+count) of a stream."""
    out = np.empty(count, dtype=np.int32)
    _get_lib().synth_uniform_i32(seed, stream, first, count, lo, hi, out.ctypes.data)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


BF16_ONE = np.uint16(0x3F80)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 bit patterns (round to nearest even; finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> 16) & np.uint32(1))) >> 16).astype(np.uint16)


def gain_vector(shape: "Shape", kind: str, index: int = 0) -> np.ndarray:
    """A non-unit RMSNorm gain, 1 + 0.25 N(0,1), as bf16 bits; kind = g_attn | g_mlp | g_final."""
    noise = bf16_bits_to_f32(normal_bf16(shape.seed, stream_id(kind, index), shape.d, 0.25))
    return f32_to_bf16_bits(np.float32(1.0) + noise)

# stream ids: kind + 32 * (index + 1); index = layer or map number (0 for globals)
_KIND = dict(embed=1, lm_head=2, pred_w=3, wq=4, wk=5, wv=6, wo=7, wgate=8, wup=9, wdown=10,
             g_attn=11, g_mlp=12, g_final=13, prompt=20, ctxlen=21, tokens=22, cache_k=23, cache_v=24)


def stream_id(kind: str, index: int = 0) -> int:
    return _KIND[kind] + 32 * (index + 1)


# ----------------------------------------------------------------------------
# shapes and the benchmark configurations
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class Shape:
    name: str
    L: int          # decoder layers
    d: int          # model width
    H: int          # query heads
    Hkv: int        # key/value heads
    dh: int         # head dim
    F: int          # SwiGLU hidden width
    V: int          # vocabulary
    seed: int
    k: int = 3      # pseudo hidden states (future positions)
    l: int = 0      # insertion layer (0-based: input of layer l)
    T: int = 1      # tree rows, root included
    prompt_len: int = 1
    steps: int = 1
    batch: int = 1
    eps: float = 1e-5
    theta: float = 1e4
    top_b: int = 8

    @property
    def n_q(self): return self.H * self.dh
    @property
    def n_kv(self): return self.Hkv * self.dh
    @property
    def n_qkv(self): return (self.H + 2 * self.Hkv) * self.dh

    def weight_bytes(self, k: int | None = None) -> int:
        k = self.k if k is None else k
        per_layer = self.n_qkv * self.d + self.d * self.n_q + 3 * self.d * self.F
        return 2 * (self.L * per_layer + self.V * self.d + k * self.d * self.d)


CONFIGS = {
    "c1": Shape("c1-tiny", L=2, d=256, H=4, Hkv=4, dh=64, F=688, V=1024, seed=0, k=3, l=1, T=8,
                prompt_len=32, steps=16),
    "c2": Shape("c2-llama2-7b", L=32, d=4096, H=32, Hkv=32, dh=128, F=11008, V=32000, seed=1, k=3, l=16, T=32,
                prompt_len=512, steps=128),
    "c3": Shape("c3-llama2-13b", L=40, d=5120, H=40, Hkv=40, dh=128, F=13824, V=32000, seed=2, k=3, l=20, T=64,
                prompt_len=1024, steps=128),
    "c5": Shape("c5-34b-gqa", L=48, d=8192, H=64, Hkv=8, dh=128, F=22016, V=32000, seed=3, k=3, l=24, T=32,
                prompt_len=4096, steps=64, batch=4),
}
# Sweep (config 4): the c2 weights with these tree sizes x committed context lengths, 64 steps per point.
C4_TREE_SIZES = (1, 8, 16, 32, 64, 128)
C4_CONTEXTS = (128, 2048, 8192)


def c4_point(T: int, n_ctx: int) -> Shape:
    base = CONFIGS["c2"]
    return replace(base, name="c4-T%d-n%d" % (T, n_ctx), T=T, k=(0 if T == 1 else 3), prompt_len=n_ctx, steps=64)


def scaled(shape: Shape, **kw) -> Shape:
    """A copy of a shape with fields overridden (reduced-depth cases for tests)."""
    return replace(shape, **kw)


# ----------------------------------------------------------------------------
# weights
# ----------------------------------------------------------------------------
def layer_weights(shape: Shape, layer: int, gains: bool = False) -> dict:
    """bf16 bits of one decoder layer.

    wqkv [(H+2Hkv)*dh, d]: q rows, then k rows, then v rows (each its own stream);
    wo [d, H*dh]; wgu [2F, d]: gate rows then up rows; wd [d, F]; gains = 1
    unless `gains` asks for the seeded non-unit ones.  All matrices are [out, in] row-major.
    """
    s = shape
    wqkv = np.empty((s.n_qkv, s.d), dtype=np.uint16)
    normal_bf16(s.seed, stream_id("wq", layer), s.n_q * s.d, 0.02, out=wqkv[: s.n_q].reshape(-1))
    normal_bf16(s.seed, stream_id("wk", layer), s.n_kv * s.d, 0.02, out=wqkv[s.n_q: s.n_q + s.n_kv].reshape(-1))
    normal_bf16(s.seed, stream_id("wv", layer), s.n_kv * s.d, 0.02, out=wqkv[s.n_q + s.n_kv:].reshape(-1))
    wo = normal_bf16(s.seed, stream_id("wo", layer), s.d * s.n_q, 0.02).reshape(s.d, s.n_q)
    wgu = np.empty((2 * s.F, s.d), dtype=np.uint16)
    normal_bf16(s.seed, stream_id("wgate", layer), s.F * s.d, 0.02, out=wgu[: s.F].reshape(-1))
    normal_bf16(s.seed, stream_id("wup", layer), s.F * s.d, 0.02, out=wgu[s.F:].reshape(-1))
    wd = normal_bf16(s.seed, stream_id("wdown", layer), s.d * s.F, 0.02).reshape(s.d, s.F)
    ones = np.full(s.d, BF16_ONE, dtype=np.uint16)
    g_attn = gain_vector(s, "g_attn", layer) if gains else ones.copy()
    g_mlp = gain_vector(s, "g_mlp", layer) if gains else ones.copy()
    return dict(wqkv=wqkv, wo=wo, wgu=wgu, wd=wd, g_attn=g_attn, g_mlp=g_mlp)


def global_weights(shape: Shape, n_maps: int | None = None, gains: bool = False) -> dict:
    """embed [V,d], lm_head [V,d] (untied), g_final [d], pred_w [k,d,d], pred_b [k,d] (zeros)."""
    s = shape
    k = s.k if n_maps is None else n_maps
    embed = normal_bf16(s.seed, stream_id("embed"), s.V * s.d, 0.02).reshape(s.V, s.d)
    lm_head = normal_bf16(s.seed, stream_id("lm_head"), s.V * s.d, 0.02).reshape(s.V, s.d)
    pred_w = np.empty((max(k, 1), s.d, s.d), dtype=np.uint16)
    for i in range(k):
        normal_bf16(s.seed, stream_id("pred_w", i), s.d * s.d, s.d ** -0.5, out=pred_w[i].reshape(-1))
    pred_w = pred_w[:k]
    pred_b = np.zeros((k, s.d), dtype=np.uint16)
    g_final = gain_vector(s, "g_final") if gains else np.full(s.d, BF16_ONE, dtype=np.uint16)
    return dict(embed=embed, lm_head=lm_head, g_final=g_final, pred_w=pred_w, pred_b=pred_b)


def all_weights(shape: Shape, gains: bool = False) -> dict:
    """{'layers': [layer dicts], **globals}; host memory = shape.weight_bytes().
    gains: non-unit RMSNorm gains, different for the attention, MLP and final norms."""
    w = global_weights(shape, gains=gains)
    w["layers"] = [layer_weights(shape, i, gains) for i in range(shape.L)]
    return w


def cache_rows(shape: Shape, seq: int, layer: int, n: int, std_k: float = 1.0, std_v: float = 0.5) -> tuple:
    """Seeded key and value rows for cache positions 0..n-1 of one layer, as bf16 bits [n, Hkv*dh]:
    a stand-in for the committed prefix of a long context (data only; nobody computed them)."""
    idx = seq * 4096 + layer
    ks = normal_bf16(shape.seed, stream_id("cache_k", idx), n * shape.n_kv, std_k).reshape(n, shape.n_kv)
    vs = normal_bf16(shape.seed, stream_id("cache_v", idx), n * shape.n_kv, std_v).reshape(n, shape.n_kv)
    return ks, vs


# ----------------------------------------------------------------------------
# prompts, context lengths, tokens
# ----------------------------------------------------------------------------
def prompt(shape: Shape, seq: int = 0, length: int | None = None) -> np.ndarray:
    n = shape.prompt_len if length is None else length
    return uniform_i32(shape.seed, stream_id("prompt", seq), n, 0, shape.V)


def context_lengths(shape: Shape, lo: int = 256, hi: int = 4096) -> np.ndarray:
    """Per-sequence committed context lengths, uniform in [lo, hi] (config 5)."""
    return uniform_i32(shape.seed, stream_id("ctxlen"), shape.batch, lo, hi + 1)


def random_tokens(shape: Shape, count: int, stream_index: int = 0) -> np.ndarray:
    return uniform_i32(shape.seed, stream_id("tokens", stream_index), count, 0, shape.V)


# ----------------------------------------------------------------------------
# draft-tree templates
# ----------------------------------------------------------------------------
TREE_WIDTHS = {1: (), 8: (2, 2, 1), 16: (3, 2, 2), 32: (4, 3, 2), 64: (5, 4, 3), 128: (8, 5, 3)}


def tree_template(T: int, widths: tuple | None = None) -> np.ndarray:
    """parents[T] (int32) of a static draft tree; parents[0] = -1 and parents[v] < v.

    Nodes are rank tuples (r_1..r_j), r_i < widths[i-1]; the full product tree is
    ordered by (sum of ranks, depth, tuple) and cut to its first T nodes, root first.
    The cut is prefix-closed and each parent's children carry ranks 0..c-1 in index order.
    """
    if widths is None:
        widths = TREE_WIDTHS[T]
    nodes = [()]
    for depth in range(1, len(widths) + 1):
        nodes += list(itertools.product(*[range(w) for w in widths[:depth]]))
    nodes.sort(key=lambda t: (sum(t), len(t), t))
    if T > len(nodes):
        raise ValueError("tree of %d nodes does not fit widths %r" % (T, widths))
    nodes = nodes[:T]
    index = {t: i for i, t in enumerate(nodes)}
    parents = np.array([-1] + [index[t[:-1]] for t in nodes[1:]], dtype=np.int32)
    assert all(parents[v] < v for v in range(1, T))
    return parents


def chain_template(T: int) -> np.ndarray:
    return np.arange(-1, T - 1, dtype=np.int32)


def random_tree(seed: int, T: int, max_depth: int, stream_index: int = 0, max_children: int = 8) -> np.ndarray:
    """A random tree with parents[v] < v, depth <= max_depth and at most max_children per node."""
    draws = uniform_i32(seed, stream_id("tokens", 1000 + stream_index), 4 * T, 0, 1 << 30)
    parents = np.full(T, -1, dtype=np.int32)
    depth = np.zeros(T, dtype=np.int32)
    kids = np.zeros(T, dtype=np.int32)
    for v in range(1, T):
        ok = lambda p: depth[p] < max_depth and kids[p] < max_children
        cands = [int(draws[4 * v + t] % v) for t in range(4)]
        p = next((c for c in cands if ok(c)), None)
        if p is None:
            p = next((c for c in range(v) if ok(c)), None)
        if p is None:
            raise ValueError("no room for %d nodes under depth %d / %d children" % (T, max_depth, max_children))
        parents[v] = p
        depth[v] = depth[p] + 1
        kids[p] += 1
    return parents
