"""ctypes binding of libfirp_b200.so (see include/firp.h for the contract of every call)."""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libfirp_b200.so")
_lib = None

i32, vp, sz = ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t


class FirpError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("firp error %d: %s" % (code, msg))
        self.code = code


FIRP_OK, FIRP_ERR_BAD_ARG, FIRP_ERR_BAD_TREE, FIRP_ERR_CAPACITY, FIRP_ERR_CUDA, FIRP_ERR_STATE = 0, -1, -2, -3, -4, -5
FIRP_ERR_DEVICE_TIMEOUT = -6


class ModelCfg(ctypes.Structure):
    _fields_ = [(n, i32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)] + \
               [(n, i32) for n in ("max_batch", "max_ctx", "max_tree", "max_k", "max_depth", "top_b", "max_rows")]


_PP = ctypes.POINTER(vp)


class Weights(ctypes.Structure):
    _fields_ = [(n, vp) for n in ("embed", "lm_head", "g_final", "pred_w", "pred_b")] + [("n_maps", i32)] + \
               [(n, _PP) for n in ("wqkv", "wo", "wgu", "wd", "g_attn", "g_mlp")]


class StepOutC(ctypes.Structure):
    _fields_ = [(n, vp) for n in ("accepted_tokens", "n_accepted", "path", "next_tree_tokens", "best", "topb_ids",
                                  "topb_vals", "logits", "depth", "mask")]


EXPORTS = ("firp_create", "firp_destroy", "firp_last_error", "firp_workspace_bytes", "firp_kv_bytes",
           "firp_bind_buffers", "firp_init_weights", "firp_prefill", "firp_step", "firp_kv_commit",
           "firp_context_len", "firp_set_context_len", "firp_last_launch_count", "firp_profile_enable",
           "firp_profile_read", "firp_kernel_class_name", "firp_topb_static", "firp_prefill_layers", "firp_step_layers", "firp_step_chains", "firp_set_pseudo_masked",
           "firp_set_fused", "firp_set_wait_limit_us", "firp_selftest_wait", "firp_set_pred_prenorm", "firp_set_kv_pages",
           "firp_set_activation_planes", "firp_set_attention_planes", "firp_set_attention_kernel", "firp_step_trees")


def lib_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libfirp_b200.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("libfirp_b200.so is missing: run `python -m paper_2410_20488_b200.build` "
                          "(or __graft_entry__.build()); the FIRP step has no CPU fallback")
    lib = ctypes.CDLL(_LIB_PATH)
    lib.firp_create.argtypes = [ctypes.POINTER(ModelCfg), ctypes.POINTER(vp)]
    lib.firp_destroy.argtypes = [vp]
    lib.firp_destroy.restype = None
    lib.firp_last_error.argtypes = [vp]
    lib.firp_last_error.restype = ctypes.c_char_p
    lib.firp_workspace_bytes.argtypes = [vp]
    lib.firp_workspace_bytes.restype = sz
    lib.firp_kv_bytes.argtypes = [vp]
    lib.firp_kv_bytes.restype = sz
    lib.firp_bind_buffers.argtypes = [vp, vp, vp, vp]
    lib.firp_init_weights.argtypes = [vp, ctypes.POINTER(Weights)]
    lib.firp_prefill.argtypes = [vp, i32, vp, i32, i32, i32, vp, i32, ctypes.POINTER(StepOutC), vp]
    lib.firp_step.argtypes = [vp, i32, vp, vp, vp, i32, i32, i32, ctypes.POINTER(StepOutC), vp]
    lib.firp_prefill_layers.argtypes = [vp, i32, vp, i32, i32, vp, vp, i32, ctypes.POINTER(StepOutC), vp]
    lib.firp_step_layers.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp, ctypes.POINTER(StepOutC), vp]
    lib.firp_step_chains.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp, ctypes.POINTER(StepOutC), vp]
    lib.firp_step_trees.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, vp, ctypes.POINTER(StepOutC), vp]
    lib.firp_set_pseudo_masked.argtypes = [vp, i32]
    lib.firp_set_fused.argtypes = [vp, i32]
    lib.firp_set_attention_planes.argtypes = [vp, i32, i32]
    lib.firp_set_attention_kernel.argtypes = [vp, i32]
    lib.firp_set_activation_planes.argtypes = [vp, i32, i32, i32, i32, i32]
    lib.firp_set_kv_pages.argtypes = [vp, vp, vp]
    lib.firp_set_pred_prenorm.argtypes = [vp, i32]
    lib.firp_set_wait_limit_us.argtypes = [vp, ctypes.c_int64]
    lib.firp_selftest_wait.argtypes = [vp, vp]
    lib.firp_kv_commit.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.firp_context_len.argtypes = [vp, i32, ctypes.POINTER(i32), vp]
    lib.firp_set_context_len.argtypes = [vp, i32, i32, vp]
    lib.firp_last_launch_count.argtypes = [vp]
    lib.firp_profile_enable.argtypes = [vp, i32]
    lib.firp_profile_read.argtypes = [vp, vp, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_float)]
    lib.firp_kernel_class_name.argtypes = [i32]
    lib.firp_kernel_class_name.restype = ctypes.c_char_p
    lib.firp_topb_static.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    for name in EXPORTS:
        if name not in ("firp_destroy", "firp_last_error", "firp_workspace_bytes", "firp_kv_bytes",
                        "firp_kernel_class_name"):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(ctx, rc):
    if rc != 0:
        msg = load_library().firp_last_error(ctx)
        raise FirpError(rc, msg.decode() if msg else "")


# ---- thin functions with the names of the C ABI ---------------------------
def firp_create(cfg: ModelCfg):
    ctx = vp()
    rc = load_library().firp_create(ctypes.byref(cfg), ctypes.byref(ctx))
    if rc != 0:
        raise FirpError(rc, "firp_create rejected the configuration")
    return ctx


def firp_destroy(ctx):
    load_library().firp_destroy(ctx)


def firp_last_error(ctx) -> str:
    return load_library().firp_last_error(ctx).decode()


def firp_workspace_bytes(ctx) -> int:
    return load_library().firp_workspace_bytes(ctx)


def firp_kv_bytes(ctx) -> int:
    return load_library().firp_kv_bytes(ctx)


def firp_bind_buffers(ctx, workspace_ptr: int, kv_ptr: int, stream: int = 0):
    _check(ctx, load_library().firp_bind_buffers(ctx, workspace_ptr, kv_ptr, stream))


def firp_init_weights(ctx, w: Weights):
    _check(ctx, load_library().firp_init_weights(ctx, ctypes.byref(w)))


def _host_i32(a):
    if a is None:
        return None, None
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, arr.ctypes.data


def firp_prefill(ctx, seq: int, d_prompt_ptr: int, P: int, k: int, l: int, next_parents, out: StepOutC, stream: int = 0):
    arr, ptr = _host_i32(next_parents)
    _check(ctx, load_library().firp_prefill(ctx, seq, d_prompt_ptr, P, k, l, ptr, 0 if arr is None else arr.size,
                                            ctypes.byref(out) if out is not None else None, stream))


def firp_prefill_layers(ctx, seq: int, d_prompt_ptr: int, P: int, k: int, layers, next_parents, out: StepOutC,
                        stream: int = 0):
    arr, ptr = _host_i32(next_parents)
    lay, lay_ptr = _host_i32(layers)
    if lay is None or lay.size != k:
        raise ValueError("need one insertion layer per prediction step")
    _check(ctx, load_library().firp_prefill_layers(ctx, seq, d_prompt_ptr, P, k, lay_ptr, ptr, 0 if arr is None else arr.size,
                                                   ctypes.byref(out) if out is not None else None, stream))


def firp_step_layers(ctx, n_seq: int, seq_ids, d_tokens_ptr: int, tree_parents, T: int, k: int, layers, out: StepOutC,
                     stream: int = 0):
    ids, ids_ptr = _host_i32(seq_ids)
    par, par_ptr = _host_i32(tree_parents)
    lay, lay_ptr = _host_i32(layers)
    if lay is None or lay.size != k:
        raise ValueError("need one insertion layer per prediction step")
    _check(ctx, load_library().firp_step_layers(ctx, n_seq, ids_ptr, d_tokens_ptr, par_ptr, T, k, lay_ptr,
                                                ctypes.byref(out) if out is not None else None, stream))


def firp_step(ctx, n_seq: int, seq_ids, d_tokens_ptr: int, tree_parents, T: int, k: int, l: int, out: StepOutC,
              stream: int = 0):
    ids, ids_ptr = _host_i32(seq_ids)
    par, par_ptr = _host_i32(tree_parents)
    _check(ctx, load_library().firp_step(ctx, n_seq, ids_ptr, d_tokens_ptr, par_ptr, T, k, l,
                                         ctypes.byref(out) if out is not None else None, stream))


def firp_step_chains(ctx, n_seq: int, seq_ids, d_tokens_ptr: int, tree_parents, T: int, k: int, layers, out: StepOutC,
                     stream: int = 0):
    """A chain of k pseudo rows under every tree node; layers: one insertion layer per prediction step."""
    ids, ids_ptr = _host_i32(seq_ids)
    par, par_ptr = _host_i32(tree_parents)
    lay, lay_ptr = _host_i32(layers)
    if k > 0 and (lay is None or lay.size != k):
        raise ValueError("need one insertion layer per prediction step")
    _check(ctx, load_library().firp_step_chains(ctx, n_seq, ids_ptr, d_tokens_ptr, par_ptr, T, k, lay_ptr,
                                                ctypes.byref(out) if out is not None else None, stream))


def firp_step_trees(ctx, n_seq: int, seq_ids, d_tokens_ptr: int, tree_parents, tree_sizes, T: int, k: int, layers,
                    out: StepOutC, stream: int = 0):
    """A tree per sequence: tree_parents host [n_seq][T], tree_sizes host [n_seq] (see firp.h)."""
    ids, ids_ptr = _host_i32(seq_ids)
    par, par_ptr = _host_i32(tree_parents)
    siz, siz_ptr = _host_i32(tree_sizes)
    lay, lay_ptr = _host_i32(layers)
    if par is None or par.size != n_seq * T or siz is None or siz.size != n_seq:
        raise ValueError("tree_parents must be [n_seq][T] and tree_sizes [n_seq]")
    _check(ctx, load_library().firp_step_trees(ctx, n_seq, ids_ptr, d_tokens_ptr, par_ptr, siz_ptr, T, k, lay_ptr,
                                               ctypes.byref(out) if out is not None else None, stream))


def firp_set_pseudo_masked(ctx, masked: bool):
    """Section 4.3 "Masked" ablation: pseudo rows do not see one another."""
    _check(ctx, load_library().firp_set_pseudo_masked(ctx, int(bool(masked))))


def firp_set_pred_prenorm(ctx, on: bool):
    """Eq. 3 on the anchor's state after the insertion layer's input RMSNorm (variant) instead of the raw residual."""
    _check(ctx, load_library().firp_set_pred_prenorm(ctx, int(bool(on))))


def firp_set_kv_pages(ctx, page_table, stream: int = 0):
    """page_table: host int32 [max_batch][max_ctx / 64] (physical page of every logical page), or None for
    contiguous rows."""
    arr, ptr = _host_i32(page_table)
    _check(ctx, load_library().firp_set_kv_pages(ctx, ptr, stream))


def firp_set_activation_planes(ctx, qkv=2, o=2, gate_up=2, down=2, lm_head=2):
    """bf16 planes of the activations per GEMM class (1 = plain bf16; see firp.h)."""
    _check(ctx, load_library().firp_set_activation_planes(ctx, qkv, o, gate_up, down, lm_head))


def firp_set_attention_planes(ctx, q_planes=2, p_planes=2):
    _check(ctx, load_library().firp_set_attention_planes(ctx, q_planes, p_planes))


def firp_set_attention_kernel(ctx, tensor_core=None):
    """True: the tcgen05 kernel, False: the mma.sync kernel, None: chosen per step (the default)."""
    _check(ctx, load_library().firp_set_attention_kernel(ctx, -1 if tensor_core is None else (1 if tensor_core else 0)))


def firp_set_fused(ctx, on: bool):
    """Run the layers of small steps as one persistent kernel (default) or one kernel per operation."""
    _check(ctx, load_library().firp_set_fused(ctx, int(bool(on))))


def firp_set_wait_limit_us(ctx, usec: int):
    """Bound of every device-side wait in microseconds (0: the default of 2 s)."""
    _check(ctx, load_library().firp_set_wait_limit_us(ctx, int(usec)))


def firp_selftest_wait(ctx, stream: int = 0):
    """Enqueue the bounded wait that nothing satisfies (see firp.h); the next firp_context_len reports it."""
    _check(ctx, load_library().firp_selftest_wait(ctx, stream))


def firp_kv_commit(ctx, n_seq: int, seq_ids=None, path=None, path_len=None, stream: int = 0):
    ids, ids_ptr = _host_i32(seq_ids)
    p, p_ptr = _host_i32(path)
    ln, ln_ptr = _host_i32(path_len)
    _check(ctx, load_library().firp_kv_commit(ctx, n_seq, ids_ptr, p_ptr, ln_ptr, stream))


def firp_context_len(ctx, seq: int, stream: int = 0) -> int:
    n = i32(0)
    _check(ctx, load_library().firp_context_len(ctx, seq, ctypes.byref(n), stream))
    return n.value


def firp_set_context_len(ctx, seq: int, n: int, stream: int = 0):
    _check(ctx, load_library().firp_set_context_len(ctx, seq, n, stream))


def firp_last_launch_count(ctx) -> int:
    return load_library().firp_last_launch_count(ctx)


def firp_profile_enable(ctx, on: bool):
    _check(ctx, load_library().firp_profile_enable(ctx, 1 if on else 0))


def firp_kernel_class_name(c: int):
    name = load_library().firp_kernel_class_name(c)
    return name.decode() if name else None


def firp_profile_read(ctx, stream: int = 0) -> dict:
    """{class name: (launches, total microseconds)} since the last read; synchronises the stream."""
    n = 64
    launches, usec = (i32 * n)(), (ctypes.c_float * n)()
    rc = load_library().firp_profile_read(ctx, stream, n, launches, usec)
    if rc < 0:
        _check(ctx, rc)
    return {firp_kernel_class_name(c): (int(launches[c]), float(usec[c])) for c in range(rc)}


def firp_topb_static(d_logits_ptr: int, rows: int, vocab: int, b: int, d_ids_ptr: int, d_vals_ptr: int, stream: int = 0):
    """Top-b of `rows` rows of device logits into caller-owned device arrays; allocates nothing (the
    candidate scratch is a fixed array inside the library).  Raises FirpError on a bad argument or when
    rows * ceil(vocab / 2048) exceeds the built-in scratch."""
    rc = load_library().firp_topb_static(d_logits_ptr, rows, vocab, b, d_ids_ptr, d_vals_ptr, stream)
    if rc != 0:
        raise FirpError(rc, "firp_topb_static rejected the call (see stderr)")


# ---- convenience: device memory through torch, nothing else ---------------
class StepOut:
    """Device output buffers of one step (torch tensors) and their C view."""

    def __init__(self, torch, device, n_seq, T, k, V, S, B, T_next=None, want_logits=True, chains=False):
        T_next = T if T_next is None else T_next
        M = T * (1 + k) if chains else T + k          # rows per sequence
        z = lambda *shape, dt=torch.int32: torch.zeros(*shape, dtype=dt, device=device)
        self.accepted_tokens, self.n_accepted, self.path = z(n_seq, S), z(n_seq), z(n_seq, S)
        self.next_tree_tokens, self.best = z(n_seq, max(T_next, 1)), z(n_seq, T)
        self.topb_ids, self.topb_vals = z(n_seq, max(k, 1), B), z(n_seq, max(k, 1), B, dt=torch.float32)
        self.logits = z(n_seq, M, V, dt=torch.float32) if want_logits else None
        self.depth = z(n_seq, M)
        self.mask = z(n_seq, M, (M + 31) // 32)
        self.c = StepOutC(**{n: (getattr(self, n).data_ptr() if getattr(self, n) is not None else None)
                             for n, _ in StepOutC._fields_})


class FirpEngine:
    """Owns a context plus the torch tensors backing its workspace, KV cache and weights."""

    def __init__(self, shape, weights, max_ctx, max_batch=1, max_tree=None, max_k=None, max_depth=None, top_b=8,
                 device="cuda:0", max_rows=0):
        import torch
        self.torch, self.device, self.shape = torch, torch.device(device), shape
        s = shape
        max_tree = s.T if max_tree is None else max_tree
        max_k = s.k if max_k is None else max_k
        max_depth = max(max_k, 1) if max_depth is None else max_depth
        self.cfg = ModelCfg(n_layers=s.L, d_model=s.d, n_heads=s.H, n_kv_heads=s.Hkv, head_dim=s.dh, d_ffn=s.F,
                            vocab=s.V, rms_eps=s.eps, rope_theta=s.theta, max_batch=max_batch, max_ctx=max_ctx,
                            max_tree=max_tree, max_k=max_k, max_depth=max_depth, top_b=top_b, max_rows=max_rows)
        self.S, self.B = max_depth + 1, top_b
        self.page_table = None
        self.ctx = firp_create(self.cfg)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(firp_workspace_bytes(self.ctx), dtype=torch.uint8, device=self.device)
            self.kv = torch.zeros(firp_kv_bytes(self.ctx), dtype=torch.uint8, device=self.device)
            firp_bind_buffers(self.ctx, self.workspace.data_ptr(), self.kv.data_ptr(), self.stream)
            self._upload(weights)

    @property
    def stream(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def _dev(self, bits):
        t = self.torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
        return t.to(self.device)

    def _upload(self, weights):
        L = self.shape.L
        self.w_tensors = {n: self._dev(weights[n]) for n in ("embed", "lm_head", "g_final")}
        n_maps = int(weights["pred_w"].shape[0]) if weights.get("pred_w") is not None else 0
        if n_maps:
            self.w_tensors["pred_w"] = self._dev(weights["pred_w"])
            if weights.get("pred_b") is not None:
                self.w_tensors["pred_b"] = self._dev(weights["pred_b"])
        self.layer_tensors = [{n: self._dev(lw[n]) for n in ("wqkv", "wo", "wgu", "wd", "g_attn", "g_mlp")}
                              for lw in weights["layers"]]
        w = Weights()
        for n in ("embed", "lm_head", "g_final", "pred_w", "pred_b"):
            setattr(w, n, self.w_tensors[n].data_ptr() if n in self.w_tensors else None)
        w.n_maps = n_maps
        self._arrays = []
        for n in ("wqkv", "wo", "wgu", "wd", "g_attn", "g_mlp"):
            arr = (vp * L)(*[lt[n].data_ptr() for lt in self.layer_tensors])
            self._arrays.append(arr)
            setattr(w, n, ctypes.cast(arr, _PP))
        self.w = w
        firp_init_weights(self.ctx, w)

    def new_out(self, n_seq, T, k, T_next=None, want_logits=True, chains=False) -> StepOut:
        return StepOut(self.torch, self.device, n_seq, T, k, self.shape.V, self.S, self.B, T_next, want_logits, chains)

    def prefill(self, seq, d_prompt, k, l, next_parents, out: StepOut):
        """l: one insertion layer, or a sequence of k layers (one per prediction step)."""
        fn = firp_prefill if np.isscalar(l) else firp_prefill_layers
        fn(self.ctx, seq, d_prompt.data_ptr(), d_prompt.numel(), k, l, next_parents,
           out.c if out is not None else None, self.stream)

    def step(self, d_tokens, parents, k, l, out: StepOut, seq_ids=None, n_seq=1):
        """l: one insertion layer, or a sequence of k layers (one per prediction step)."""
        T = len(parents)
        fn = firp_step if np.isscalar(l) else firp_step_layers
        fn(self.ctx, n_seq, seq_ids, d_tokens.data_ptr(), parents, T, k, l, out.c if out is not None else None, self.stream)

    def step_chains(self, d_tokens, parents, k, l, out: StepOut, seq_ids=None, n_seq=1):
        """The step with a chain of k pseudo rows under every tree node (out from new_out(..., chains=True));
        l: one insertion layer, or one per prediction step."""
        layers = [l] * k if np.isscalar(l) else l
        firp_step_chains(self.ctx, n_seq, seq_ids, d_tokens.data_ptr(), parents, len(parents), k, layers,
                         out.c if out is not None else None, self.stream)

    def step_trees(self, d_tokens, tree_parents, tree_sizes, k, l, out: StepOut, seq_ids=None):
        """A tree per sequence: tree_parents [n_seq][T] (host), tree_sizes [n_seq]; d_tokens [n_seq][T]."""
        par = np.ascontiguousarray(tree_parents, np.int32)
        n_seq, T = par.shape
        layers = [l] * k if np.isscalar(l) else l
        firp_step_trees(self.ctx, n_seq, seq_ids, d_tokens.data_ptr(), par, tree_sizes, T, k, layers,
                        out.c if out is not None else None, self.stream)

    def set_pseudo_masked(self, masked: bool):
        firp_set_pseudo_masked(self.ctx, masked)

    def set_pred_prenorm(self, on: bool):
        firp_set_pred_prenorm(self.ctx, on)

    def set_kv_pages(self, page_table):
        """Scatter the cache over pages of 64 positions (None: contiguous); remembered for the test harness."""
        firp_set_kv_pages(self.ctx, page_table, self.stream)
        self.page_table = None if page_table is None else np.ascontiguousarray(page_table, np.int32).reshape(self.cfg.max_batch, -1)

    def set_activation_planes(self, qkv=2, o=2, gate_up=2, down=2, lm_head=2):
        firp_set_activation_planes(self.ctx, qkv, o, gate_up, down, lm_head)

    def set_attention_planes(self, q_planes=2, p_planes=2):
        firp_set_attention_planes(self.ctx, q_planes, p_planes)

    def set_attention_kernel(self, tensor_core=None):
        firp_set_attention_kernel(self.ctx, tensor_core)

    def set_fused(self, on: bool):
        firp_set_fused(self.ctx, on)

    def set_wait_limit_us(self, usec: int):
        firp_set_wait_limit_us(self.ctx, usec)

    def selftest_wait(self):
        firp_selftest_wait(self.ctx, self.stream)

    def commit(self, n_seq=1, seq_ids=None, path=None, path_len=None):
        if path is not None:
            p = np.zeros((n_seq, self.S), np.int32)
            for s_i in range(n_seq):
                row = np.asarray(path[s_i], np.int32)
                p[s_i, : row.size] = row
            path_len = np.array([len(path[s_i]) for s_i in range(n_seq)], np.int32)
            path = p
        firp_kv_commit(self.ctx, n_seq, seq_ids, path, path_len, self.stream)

    def context_len(self, seq=0) -> int:
        return firp_context_len(self.ctx, seq, self.stream)

    def set_context_len(self, seq, n):
        firp_set_context_len(self.ctx, seq, n, self.stream)

    def launches(self) -> int:
        return firp_last_launch_count(self.ctx)

    def profile(self, on: bool):
        firp_profile_enable(self.ctx, on)

    def profile_read(self) -> dict:
        return firp_profile_read(self.ctx, self.stream)

    def close(self):
        if self.ctx:
            firp_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
