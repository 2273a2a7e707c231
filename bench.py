#!/usr/bin/env python
"""Benchmark of the FIRP draft+verify step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

One "step" = one pass of the whole hot path: firp_step (tree prep, embedding, all decoder layers
with the pseudo hidden states inserted at layer l, lm-head, top-B, acceptance walk, next tree)
followed by firp_kv_commit, on the Llama-2-7B-shaped synthetic workload (T = 32, k = 3, l = 16,
512 committed tokens, random bf16 weights from the seeded generator).  Prints ONE JSON line.

N > 1 runs N independent replicas (the step does not shard; there is no collective): every rank
steps its own sequence on its own GPU, the job's value is the sum of the units over the maximum
of the device times.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verify+draft step: accepted tokens/s (step latency in ms_per_step), Llama-2-7B shape; HBM GB/s vs peak"
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", help="c1 | c2 | c3 | c4:T:n (sweep point on the c2 weights)")
    ap.add_argument("--layers", type=int, default=0, help="debug only: truncate the decoder (marks the line invalid)")
    ap.add_argument("--insert-layers", default="", help="one insertion layer per prediction step, e.g. 15,20,25 "
                    "(the paper's 7B setting); default: the workload's single layer l")
    ap.add_argument("--chains", action="store_true", help="a chain of k pseudo rows under every tree node "
                    "(firp_step_chains; T (1 + k) rows) instead of the workload's single chain")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-kernel-times", action="store_true", help="skip the per-kernel event-timed pass")
    ap.add_argument("--fused", type=int, default=-1, choices=[-1, 0, 1], help="1: the decoder layers of a step as one persistent "
                    "kernel, 0: one kernel per operation, -1: the library's default")
    ap.add_argument("--attention", default="auto", choices=["auto", "tc", "mma"], help="tree attention at head_dim 128: chosen per "
                    "step (the library's default), the tcgen05 kernel or the mma.sync one")
    ap.add_argument("--no-forced", action="store_true", help="skip the forced-accept run")
    ap.add_argument("--sweep", action="store_true", help="config-4 sweep on the c2 weights: T x context, one JSON line per point")
    return ap.parse_args()


# One insertion layer per prediction step (--insert-layers), or None: the workload's single layer l.
INSERT_LAYERS = None
# A chain of pseudo rows under every tree node (--chains) instead of one chain under the root.
CHAINS = False


def ins_l(shape):
    """What the step and prefill calls get as `l`: the per-step layers if given, else shape.l."""
    return list(INSERT_LAYERS) if INSERT_LAYERS else shape.l


def pick_shape(name: str, layers: int):
    import synth_inputs as si
    if name.startswith("c4:"):
        _, T, n = name.split(":")
        shape = si.c4_point(int(T), int(n))
    else:
        shape = si.CONFIGS[name]
    if layers:
        shape = si.scaled(shape, L=layers, l=min(shape.l, layers - 1), name=shape.name + "-L%d" % layers)
    return shape


def algorithmic_bytes(shape, n_ctx: float, batch: int = 1) -> dict:
    """Bytes one step must move: every weight once, the KV cache read once per layer, the new
    rows' KV written once, the embedding rows (logits stay on the device and are not exported)."""
    s = shape
    weights = s.weight_bytes()
    kv_row = 2 * 2 * s.n_kv * batch               # K and V, bf16, every sequence
    kv_read = kv_write = 0
    for j in range(s.L):
        per_step = s.T if CHAINS else 1            # pseudo rows one prediction step adds
        alive = sum(1 for t in INSERT_LAYERS if t <= j) if INSERT_LAYERS else (s.k if j >= s.l else 0)
        M = s.T + per_step * alive
        kv_read += kv_row * (n_ctx + M)
        kv_write += kv_row * M
    return dict(weights=weights, kv_read=kv_read, kv_write=kv_write, embed=2 * s.T * s.d * batch,
                total=weights + kv_read + kv_write + 2 * s.T * s.d * batch)


def class_bytes(shape, n_ctx: float) -> dict:
    """Algorithmic bytes per launch of each kernel class that streams from HBM: the weight matrix
    (read once) for the GEMMs and the Eq. 3 maps, the K and V planes of one layer for the attention."""
    s = shape
    M = s.T + s.k
    ab = algorithmic_bytes(s, n_ctx)
    return dict(gemm_qkv=2 * s.n_qkv * s.d, gemm_o=2 * s.d * s.n_q, gemm_gate_up=2 * 2 * s.F * s.d,
                gemm_down=2 * s.d * s.F, gemm_lm_head=2 * s.V * s.d, pseudo_proj=2 * s.k * s.d * s.d,
                tree_attention=2 * 2 * s.n_kv * (n_ctx + M),
                # the persistent kernel runs every layer, Eq. 3 and the lm-head: all weights once, the cache once
                fused_decoder_layers=ab["weights"] - 2 * s.V * s.d + ab["kv_read"] + ab["kv_write"])


def ncu_traffic(workload: str):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of each kernel class, from the ncu
    capture summarised in profiles/ncu_traffic.json; valid only for the kernel sources whose digest is recorded
    with it (a changed kernel reports traffic = null until it is captured again)."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "ncu_traffic.json"))).get(workload)
    except (OSError, ValueError):
        return None
    if not rec or rec.get("digest") != kernel_source_digest():
        return None
    return rec.get("per_launch", {})


def kernel_source_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2410_20488_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")) and name != "firp_api.cu":       # device code only (firp_api.cu is host code)
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def kernel_times(eng, shape, parents, tokens, out, steps, n_ctx, peak_gbs, peak_kind, seq_ids=None, step_fn=None):
    """Second, separately timed pass: the library brackets every launch with CUDA events on the
    launching stream; per class: launches, average duration, share of the summed kernel time and,
    for the HBM-streaming classes, achieved GB/s = algorithmic bytes per launch / average duration."""
    seq_ids = seq_ids or [0]
    step_fn = step_fn or eng.step
    eng.profile(True)
    for _ in range(steps):
        step_fn(tokens, parents, shape.k, ins_l(shape), out, seq_ids=seq_ids, n_seq=len(seq_ids))
        eng.commit(len(seq_ids), seq_ids=seq_ids)
        tokens = out.next_tree_tokens
    prof = eng.profile_read()
    eng.profile(False)
    total = sum(us for _, us in prof.values()) or 1.0
    cb = class_bytes(shape, n_ctx)
    kernels = {}
    for name, (n, us) in prof.items():
        if n == 0:
            continue
        k = dict(launches_per_step=n / steps, avg_us=us / n, share=us / total)
        if name in cb:
            k["bytes_per_launch"] = cb[name]
            k["achieved_gbs"] = cb[name] / (us / n * 1e-6) / 1e9
            k["frac_of_peak"] = k["achieved_gbs"] / peak_gbs
        kernels[name] = k
    top = max((n for n in kernels if n in cb), key=lambda n: kernels[n]["share"])
    t = kernels[top]
    rec = None if CHAINS else ncu_traffic(shape.name)      # the capture is of the 35-row step
    traffic = rec.get(top) if rec else None
    roofline = dict(bound="hbm", kernel=top, achieved=t["achieved_gbs"], peak=peak_gbs, unit="GB/s",
                    frac=t["frac_of_peak"], traffic=traffic, peak_kind="%s copy bandwidth" % peak_kind,
                    avg_us=t["avg_us"], share_of_kernel_time=t["share"], bytes_per_launch=t["bytes_per_launch"],
                    note="dominant kernel class, event-bracketed launches (bracketing serialises launches that "
                         "overlap in the timed run)")
    return dict(roofline=roofline, kernels=kernels, profiled_steps=steps, sum_kernel_ms_per_step=total / steps / 1e3)


def aggregate_over_ranks(ms: float, units: float, device=None):
    """Whole-job figures of N independent replicas: the slowest rank's device time and the units of all
    ranks.  With one process (no process group) the inputs come back unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), float(units)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(suffix=".csv")
        self.f = open(self.path, "w")
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self) -> dict:
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.p.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        try:
            for ln in open(self.path):
                c = [x.strip() for x in ln.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def eng_fused(args) -> bool:
    """What --fused selects; -1 is the library's default."""
    return LIB_DEFAULT_FUSED if args.fused < 0 else bool(args.fused)


LIB_DEFAULT_FUSED = False


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def time_oracle(shape, weights, steps: int, warmup: int, n_ctx: int | None = None):
    """The CPU oracle, as it stands, on a bounded sample: `steps` full draft+verify steps (all layers, T + k rows)
    on the workload's own committed context length.  The context is not prefilled (the oracle's prefill grows with
    the square of the context): its cache rows are seeded values (synth_inputs.cache_rows), so a step costs what a
    step on a real context of that length costs."""
    import oracle
    import synth_inputs as si
    n_ctx = shape.prompt_len if n_ctx is None else n_ctx
    parents = si.tree_template(shape.T)
    rows = shape.T * (1 + shape.k) if CHAINS else shape.T + shape.k
    orc = oracle.Oracle(shape, weights, max_ctx=n_ctx + (steps + warmup + 1) * (shape.k + 1) + rows + 8)
    std = 0.02 * float(np.sqrt(shape.d))
    for layer in range(shape.L):
        ks, vs = si.cache_rows(shape, 0, layer, n_ctx, std, std)
        orc.write_cache(0, layer, 0, 0, ks)
        orc.write_cache(0, layer, 1, 0, vs)
    orc.set_context_len(0, n_ctx)
    tokens = si.random_tokens(shape, shape.T, 9)
    emitted, t_total = 0, 0.0
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        out = (orc.step_chains if CHAINS else orc.step)(tokens, parents, shape.k, ins_l(shape))
        orc.commit(out["path"])
        dt = time.perf_counter() - t0
        if i >= warmup:
            t_total += dt
            emitted += int(out["n_accepted"])
        tokens = out["next_tokens"]
    return emitted / t_total, t_total / steps * 1e3


def run_forced(eng, shape, parents, tokens, outs, K, dev, step_fn):
    """Forced-accept throughput (every step accepts the full depth D of the tree and emits D + 1 tokens, so every
    commit compacts a real path), without the oracle: the greedy continuation of the committed sequence is first
    produced on the device by plain T = 1, k = 0 steps, the context is rewound, and each timed step then gets that
    continuation planted on the principal chain (root -> lowest-index child -> ...) of its tree.  A near-tie that
    the two passes resolve differently would show as tokens_per_step < D + 1; nothing is assumed, the emitted
    tokens are counted from the growth of the committed context."""
    import torch
    T = shape.T
    chain = [0]
    while True:
        kids = [u for u in range(T) if parents[u] == chain[-1]]
        if not kids:
            break
        chain.append(min(kids))
    D = len(chain) - 1
    n0 = eng.context_len(0)
    need = K * (D + 1) + D + 1
    one = np.array([-1], np.int32)
    o1 = eng.new_out(1, 1, 0, T_next=1, want_logits=False)
    stream = torch.empty(need + 1, dtype=torch.int32, device=dev)
    tok = tokens[0, :1].clone()
    stream[0] = tok[0]
    for i in range(need):
        eng.step(tok, one, 0, 0, o1)
        eng.commit(1)
        tok = o1.accepted_tokens[0, :1].clone()
        stream[i + 1] = tok[0]
    eng.set_context_len(0, n0)                       # rewind to the committed prefix (synchronises)
    idx = torch.tensor(chain[1:], dtype=torch.long, device=dev)

    def forced_steps(count):
        cur = tokens.clone()
        p = 0
        for i in range(count):
            cur[0, 0] = stream[p]
            cur[0, idx] = stream[p + 1: p + 1 + D]
            o = outs[i & 1]
            step_fn(cur, parents, shape.k, ins_l(shape), o, seq_ids=[0], n_seq=1)
            eng.commit(1, seq_ids=[0])
            cur = o.next_tree_tokens.clone()
            p += D + 1

    forced_steps(3)                                  # untimed: the same loop (the first use of torch's indexing kernels costs ~30 ms)
    eng.set_context_len(0, n0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    forced_steps(K)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    emitted = eng.context_len(0) - n0
    return dict(tokens_per_s=emitted / (ms * 1e-3), tokens_per_step=emitted / K, ms_per_step=ms / K, steps=K, depth=D,
                note="device-resident; the timed region also holds the three small torch kernels per step that plant the chain; "
                     "a near-tie that the T = 1 pass and the tree pass resolve differently desynchronises every later step")


def load_weights(shape, local_rank: int, world: int):
    """Rank-local generation of the seeded weights (every rank needs the same tensors)."""
    import synth_inputs as si
    if world > 1:
        os.environ.setdefault("OMP_NUM_THREADS", str(max(1, host_cores() // world)))
    return si.all_weights(shape)


def run_reference(args, shape):
    """The reference arm of this tier is the CPU oracle, timed on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import synth_inputs as si
    weights = si.all_weights(shape)
    steps, warmup = max(1, min(args.steps, 3)), min(args.warmup, 1)
    tps, ms = time_oracle(shape, weights, steps, warmup)
    sample = "%d oracle steps (+%d warm-up) of T=%d,k=%d,l=%s over all %d layers on a %d-token context (seeded cache rows, no prefill)" % (
        steps, warmup, shape.T, shape.k, ins_l(shape), shape.L, shape.prompt_len)
    line = dict(metric=METRIC, value=tps, unit=UNIT, n_gpus=args.gpus, steps=steps, warmup=warmup, ms_per_step=ms,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32 storage, f64 accumulation",
                data="synthetic", impl="reference",
                config=dict(workload=shape.name, T=shape.T, k=shape.k, l=ins_l(shape), context_start=shape.prompt_len,
                            batch=1, sample="a few oracle steps on the workload's %d-token context" % shape.prompt_len),
                cpu_baseline=dict(value=tps, unit=UNIT, cores=host_cores(), kind="oracle", sample=sample),
                e2e=dict(value=tps, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def run_sweep(args, shape, weights, dev, rank):
    """Config 4: tree size x committed context on the c2 weights, `--steps` steps per point (default 64 there),
    device-resident timing only.  One engine serves every point; one JSON line per point."""
    import torch
    import synth_inputs as si
    from paper_2410_20488_b200 import FirpEngine
    K, W = args.steps, max(args.warmup, 3)
    eng = FirpEngine(shape, weights, max_ctx=max(si.C4_CONTEXTS) + (K + W + 2) * 4 + 128 + 3 + 64, max_tree=128, max_k=3,
                     max_depth=3, device=str(dev))
    if args.fused >= 0:
        eng.set_fused(bool(args.fused))
    eng.set_attention_kernel({"auto": None, "tc": True, "mma": False}[args.attention])
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    peak_gbs = peaks.get("hbm_gbs", 6650.0)
    for n_ctx in si.C4_CONTEXTS:
        prompt = torch.from_numpy(si.prompt(shape, length=n_ctx)).to(dev)
        for T in si.C4_TREE_SIZES:
            pt = si.c4_point(T, n_ctx)
            parents = si.tree_template(T)
            T_next = T if pt.k > 0 else 1
            pout = eng.new_out(1, 1, pt.k, T_next=T_next, want_logits=False)
            eng.prefill(0, prompt, pt.k, pt.l, parents if pt.k > 0 else None, pout)
            outs = [eng.new_out(1, T, pt.k, want_logits=False) for _ in range(2)]
            tokens = pout.next_tree_tokens
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_w = n_ctx
            for i in range(W + K):
                if i == W:
                    n_w = eng.context_len(0)        # synchronises
                    ev0.record()
                o = outs[i & 1]
                eng.step(tokens, parents, pt.k, pt.l, o)
                eng.commit(1)
                tokens = o.next_tree_tokens
            ev1.record()
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1) / K
            n_end = eng.context_len(0)
            ab = algorithmic_bytes(pt, 0.5 * (n_ctx + n_end))
            gbs = ab["total"] / (ms * 1e-3) / 1e9
            print(json.dumps(dict(workload=pt.name, T=T, k=pt.k, context=n_ctx, steps=K, ms_per_step=ms,
                                  tokens_per_s=(n_end - n_w) / (ms * K * 1e-3), bytes_per_step=ab["total"],
                                  achieved_gbs=gbs, frac_of_measured_peak=gbs / peak_gbs, frac_of_8tbs=gbs / 8000.0,
                                  layers_as="one persistent kernel where a step has at most 48 rows" if eng_fused(args) else "one kernel per operation")),
                  flush=True)
    eng.close()


def main():
    args = parse()
    shape = pick_shape(args.workload, args.layers)
    if args.insert_layers:
        global INSERT_LAYERS
        INSERT_LAYERS = [int(t) for t in args.insert_layers.split(",")]
        if len(INSERT_LAYERS) != shape.k or INSERT_LAYERS != sorted(INSERT_LAYERS) or not all(0 <= t < shape.L for t in INSERT_LAYERS):
            raise SystemExit("--insert-layers needs k non-decreasing layers inside the decoder")
    global CHAINS
    CHAINS = bool(args.chains)
    if args.impl == "reference":
        return run_reference(args, shape)

    import torch
    import torch.distributed as dist
    import synth_inputs as si
    from paper_2410_20488_b200 import FirpEngine, build as firp_build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the FIRP step has no CPU fallback")
    if rank == 0:
        firp_build.build()
    if world > 1:
        dist.barrier()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)

    K, W = args.steps, max(args.warmup, 3)
    weights = load_weights(shape, local_rank, world)
    if args.sweep:
        return run_sweep(args, shape, weights, dev, rank)
    parents = si.tree_template(shape.T)
    B = shape.batch
    S = max(shape.k, 1) + 1
    total_steps = 4 * (K + W) + 32
    if B > 1:       # config 5: every sequence has its own committed context length, uniform in [256, 4096]
        lengths = [int(n) for n in si.context_lengths(shape)]
    else:
        lengths = [shape.prompt_len]
    chains = bool(args.chains)
    rows_per_seq = shape.T * (1 + shape.k) if chains else shape.T + shape.k
    max_ctx = max(lengths) + total_steps * S + rows_per_seq + 64
    eng = FirpEngine(shape, weights, max_ctx=max_ctx, max_batch=B, device=str(dev), max_rows=B * rows_per_seq if chains else 0)
    if args.fused >= 0:
        eng.set_fused(bool(args.fused))
    eng.set_attention_kernel({"auto": None, "tc": True, "mma": False}[args.attention])
    step_fn = eng.step_chains if chains else eng.step
    T_next = shape.T if shape.k > 0 else 1
    outs = [eng.new_out(B, shape.T, shape.k, want_logits=False, chains=chains) for _ in range(2)]
    first = torch.zeros(B, T_next, dtype=torch.int32, device=dev)
    for b_i, n in enumerate(lengths):
        prompt = torch.from_numpy(si.prompt(shape, seq=rank * B + b_i, length=n)).to(dev)
        pout = eng.new_out(1, 1, shape.k, T_next=T_next, want_logits=False)
        eng.prefill(b_i, prompt, shape.k, ins_l(shape), parents if shape.k > 0 else None, pout)
        first[b_i] = pout.next_tree_tokens[0]
    torch.cuda.synchronize()
    n_start = sum(eng.context_len(b_i) for b_i in range(B)) / B
    seq_ids = list(range(B))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: next tree tokens never leave the GPU -----------------------
    tokens = first
    launches = 0
    def one_step(i, tokens):
        nonlocal launches
        o = outs[i & 1]
        step_fn(tokens, parents, shape.k, ins_l(shape), o, seq_ids=seq_ids, n_seq=B)
        launches += eng.launches()
        eng.commit(B, seq_ids=seq_ids)
        launches += eng.launches()
        return o

    sampler = ClockSampler(local_rank) if rank == 0 else None    # nvidia-smi takes a while to start: the warm-up
    for i in range(W):                                           # steps (same load) are sampled as well
        tokens = one_step(i, tokens).next_tree_tokens
    barrier()
    launches = 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_before = [eng.context_len(b_i) for b_i in range(B)]
    barrier()
    ev0.record()
    for i in range(K):
        tokens = one_step(i, tokens).next_tree_tokens
    ev1.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    ms_total = ev0.elapsed_time(ev1)
    # every commit advances a context by the tokens that step emitted, so the growth counts them exactly
    n_after = [eng.context_len(b_i) for b_i in range(B)]
    emitted = sum(n_after) - sum(n_before)
    n_end = sum(n_after) / B

    # ---- end to end: host buffers in, host results out, every step -------------------------
    e2e = None
    if not args.no_e2e:
        h_tokens = torch.empty(B, T_next, dtype=torch.int32).pin_memory()
        h_tokens.copy_(tokens.cpu())
        d_tokens = torch.empty(B, T_next, dtype=torch.int32, device=dev)
        o = outs[0]
        h_acc = torch.empty(B, S, dtype=torch.int32).pin_memory()
        h_n = torch.empty(B, dtype=torch.int32).pin_memory()
        h_next = torch.empty(B, T_next, dtype=torch.int32).pin_memory()
        e_emitted = 0
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(K):
            d_tokens.copy_(h_tokens, non_blocking=True)
            step_fn(d_tokens, parents, shape.k, ins_l(shape), o, seq_ids=seq_ids, n_seq=B)
            eng.commit(B, seq_ids=seq_ids)
            h_acc.copy_(o.accepted_tokens, non_blocking=True)
            h_n.copy_(o.n_accepted, non_blocking=True)
            h_next.copy_(o.next_tree_tokens, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            e_emitted += int(h_n.sum())
            h_tokens.copy_(h_next)
        e1.record()
        barrier()
        e2e = dict(ms=e0.elapsed_time(e1), emitted=e_emitted, h2d=int(h_tokens.numel() * 4),
                   d2h=int((h_acc.numel() + h_n.numel() + h_next.numel()) * 4))

    # ---- forced-accept mode (a = D every step): rank-local, one sequence --------------------
    forced = None
    if not args.no_forced and shape.k > 0 and B == 1 and not chains:
        forced = run_forced(eng, shape, parents, tokens, outs, K, dev, step_fn)

    # ---- aggregate over ranks: max time, summed units ----------------------------------------
    ms_max, units = aggregate_over_ranks(ms_total, emitted, dev)
    if e2e:
        e_ms_max, e_units = aggregate_over_ranks(e2e["ms"], e2e["emitted"], dev)

    if rank != 0:
        return
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    peak_gbs, peak_kind = (peaks["hbm_gbs"], "measured") if "hbm_gbs" in peaks else (6650.0, "fallback")
    n_mid = 0.5 * (n_start + n_end)

    # ---- per-kernel-class durations (second, separately timed pass with events in the library) ----
    prof = None
    if not args.no_kernel_times:
        prof = kernel_times(eng, shape, parents, tokens, outs[0], min(K, 8), n_end, peak_gbs, peak_kind, seq_ids, step_fn)
    ab = algorithmic_bytes(shape, n_mid, B)
    ms_step = ms_max / K
    step_gbs = ab["total"] / (ms_step * 1e-3) / 1e9
    line = dict(metric=METRIC, value=units / (ms_max * 1e-3), unit=UNIT, n_gpus=world, steps=K, warmup=W,
                ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic", gpu_launches=launches,
                config=dict(workload=shape.name, T=shape.T, k=shape.k, l=ins_l(shape), context_start=n_start,
                            context_end=n_end, batch=B, pseudo_rows="a chain under every node" if chains else "one chain under the root", l2="inputs_larger_than_l2 (%.1f GB of weights per step)" %
                            (ab["weights"] / 1e9), parallelism="replicas x%d" % world,
                            mode="free-running greedy (random weights accept ~0 drafts per step); forced_accept has the a = D case",
                            layers_as="one persistent kernel" if eng_fused(args) else "one kernel per operation"),
                step_latency_us=ms_step * 1e3, tokens_per_step=units / (K * world), tokens_per_step_per_sequence=units / (K * world * B),
                step_hbm=dict(bytes_per_step=ab["total"], weights=ab["weights"], kv_read=ab["kv_read"],
                              achieved_gbs=step_gbs, frac_of_measured_peak=step_gbs / peak_gbs,
                              frac_of_8tbs=step_gbs / 8000.0, peak_gbs=peak_gbs, peak=peak_kind),
                clocks=clocks)
    if args.layers:
        line["invalid"] = "decoder truncated to %d layers (debug run)" % args.layers
    if e2e:
        line["e2e"] = dict(value=e_units / (e_ms_max * 1e-3), unit=UNIT, ms_per_step=e_ms_max / K,
                           h2d_bytes_per_step=e2e["h2d"], d2h_bytes_per_step=e2e["d2h"])
    if forced:
        line["forced_accept"] = forced
    if prof:
        line["roofline"] = prof["roofline"]
        line["kernels"] = prof["kernels"]
        line["kernel_pass"] = dict(steps=prof["profiled_steps"], sum_kernel_ms_per_step=prof["sum_kernel_ms_per_step"])
    else:
        line["roofline"] = dict(bound="hbm", achieved=step_gbs, peak=peak_gbs, unit="GB/s", frac=step_gbs / peak_gbs,
                                traffic=None, note="whole step (all kernels): bytes per step / step time; peak = %s copy bandwidth" % peak_kind)
    if not args.no_cpu_baseline:
        cb_steps = 2 if shape.name.startswith("c2") else 1
        tps, ms = time_oracle(shape, weights, cb_steps, 0)
        line["cpu_baseline"] = dict(value=tps, unit=UNIT, cores=host_cores(), kind="oracle", ms_per_step=ms,
                                    sample="%d oracle steps of T=%d,k=%d,l=%s over all %d layers on a %d-token context "
                                           "(seeded cache rows, no prefill)" % (cb_steps, shape.T, shape.k, ins_l(shape), shape.L, shape.prompt_len))
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
