"""Parity of the CUDA path (through the C ABI) against the CPU oracle, on a B200."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from lockstep import lockstep_run, lockstep_steps, seed_prefix, compare_step, gpu_outputs, Stats

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2410_20488_b200 import build as firp_build
    firp_build.build()
    return torch


def make_pair(shape, weights, max_ctx, masked=False, fused=False, prenorm=False, **kw):
    """fused=True: steps of at most 48 rows run their decoder layers as one persistent kernel (firp_set_fused)."""
    from paper_2410_20488_b200 import FirpEngine
    eng = FirpEngine(shape, weights, max_ctx=max_ctx, **kw)
    eng.set_fused(fused)
    orc = oracle.Oracle(shape, weights, max_ctx=max_ctx, n_seq=kw.get("max_batch", 1), masked=masked, prenorm=prenorm)
    if masked:
        eng.set_pseudo_masked(True)
    if prenorm:
        eng.set_pred_prenorm(True)
    return eng, orc


@pytest.mark.parametrize("fused", [True, False])
def test_c1_greedy_and_forced(torch_cuda, c1, c1_weights, fused):
    parents = si.tree_template(c1.T)
    for forced in (False, True):
        eng, orc = make_pair(c1, c1_weights, 256, fused=fused)
        st = lockstep_run(eng, orc, c1, parents, si.prompt(c1), c1.steps, forced=forced)
        assert st.steps == c1.steps
        if forced:
            assert st.emitted == 1 + c1.steps * 4
        print("c1 forced=%s" % forced, st.as_dict())
        eng.close()


@pytest.mark.parametrize("fused", [False, True])
def test_c1_t1_k0_autoregressive(torch_cuda, c1, c1_weights, fused):
    eng, orc = make_pair(c1, c1_weights, 128, max_tree=8, max_k=3, fused=fused)
    st = lockstep_run(eng, orc, c1, np.array([-1], np.int32), si.prompt(c1, length=9), 12, k=0, l=0)
    assert st.steps == 12 and st.emitted == 13
    eng.close()


@pytest.mark.parametrize("fused", [False, True])
def test_c1_non_unit_gains(torch_cuda, c1, fused):
    """RMSNorm gains that differ between the attention norm, the MLP norm and the final norm of every layer
    (the workload configurations use gains of 1, which would hide a swapped or dropped gain)."""
    weights = si.all_weights(c1, gains=True)
    parents = si.tree_template(c1.T)
    for forced in (False, True):
        eng, orc = make_pair(c1, weights, 256, fused=fused)
        st = lockstep_run(eng, orc, c1, parents, si.prompt(c1, length=41), 6, forced=forced)
        assert st.steps == 6
        eng.close()
    # per-step insertion layers and a chain under every node take other kernel paths for the new rows' norm
    shape = si.scaled(c1, L=4)
    w4 = si.all_weights(shape, gains=True)
    eng, orc = make_pair(shape, w4, 256, max_tree=16, max_k=3, max_depth=3, max_rows=13 * 4, fused=fused)
    parents = si.random_tree(3, 13, 3, 2)
    assert lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=30), 3, k=3, l=[0, 2, 3]).steps == 3
    assert lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=30), 3, k=3, l=[1, 2, 2], chains=True).steps == 3
    eng.close()


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("Hkv", [2, 1])
def test_c1_grouped_query_attention_two_query_blocks(torch_cuda, c1, Hkv, fused):
    """4 query heads on 2 or 1 key/value heads with enough rows that rows x heads-per-group exceeds one
    64-row query block (19 x 2 = 38 and 19 x 4 = 76; 35 x 4 = 140 with the 32-node tree), gains non-unit."""
    shape = si.scaled(c1, Hkv=Hkv)
    weights = si.all_weights(shape, gains=True)
    for T, n0 in ((16, 70), (32, 9)):
        parents = si.tree_template(T)
        eng, orc = make_pair(shape, weights, 256, max_tree=32, max_k=3, max_depth=3, fused=fused)
        st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=n0), 4, k=3, l=1, forced_steps=(1, 3))
        assert st.steps == 4
        eng.close()


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("case", range(4))
def test_c1_random_trees_and_layers(torch_cuda, c1, c1_weights, case, fused):
    T = (5, 16, 33, 128)[case]
    k = (1, 3, 2, 3)[case]
    l = (0, 1, 1, 0)[case]
    parents = si.random_tree(21, T, k, case)
    eng, orc = make_pair(c1, c1_weights, 512, max_tree=128, max_k=3, max_depth=3, fused=fused)
    st = lockstep_run(eng, orc, c1, parents, si.prompt(c1, length=(3, 70, 129, 200)[case]), 4, k=k, l=l)
    assert st.steps == 4
    eng.close()


@pytest.mark.parametrize("layers", [(0, 1, 1), (0, 0, 1), (0, 1, 3), (1, 2, 3), (2, 2, 3), (3, 3, 3)])
def test_c1_one_insertion_layer_per_prediction_step(torch_cuda, c1, layers):
    """Section 3.3: prediction step i has its own layer t_i (firp_step_layers / firp_prefill_layers):
    lock-step against the oracle on the small shape, two or four layers deep, greedy and forced."""
    shape = si.scaled(c1, L=2 if max(layers) < 2 else 4, l=layers[0])
    weights = si.all_weights(shape)
    parents = si.random_tree(5, 19, 3, sum(layers))
    for forced in (False, True):
        eng, orc = make_pair(shape, weights, 256, max_tree=32, max_k=3, max_depth=3)
        st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=45), 4, forced=forced, k=3, l=list(layers))
        assert st.steps == 4
        eng.close()


def test_c1_equal_layers_are_the_single_layer_call_bit_for_bit(torch_cuda, c1, c1_weights):
    import torch
    parents = si.tree_template(8)
    tokens = torch.from_numpy(si.random_tokens(c1, 8, 3)).cuda()
    prompt = torch.from_numpy(si.prompt(c1)).cuda()
    logits = []
    for l in (1, [1, 1, 1]):
        eng, _ = make_pair(c1, c1_weights, 128)
        pout = eng.new_out(1, 1, 3, T_next=8)
        eng.prefill(0, prompt, 3, l, parents, pout)
        out = eng.new_out(1, 8, 3)
        eng.step(tokens, parents, 3, l, out)
        torch.cuda.synchronize()
        logits.append((pout.logits.cpu().numpy().copy(), out.logits.cpu().numpy().copy(), out.next_tree_tokens.cpu().numpy().copy()))
        eng.close()
    for a, b in zip(logits[0], logits[1]):
        assert np.array_equal(a, b)


def test_fused_and_per_operation_paths_agree_and_repeat_bit_for_bit(torch_cuda, c1, c1_weights):
    """The persistent kernel and the kernel-per-operation path run the same arithmetic (they may split the cached
    positions differently for the attention): logits agree to fp32 rounding.  Each path repeated on the same state
    gives bit-identical logits (fixed summation orders everywhere)."""
    import torch
    shape = si.scaled(c1, Hkv=2)
    weights = si.all_weights(shape, gains=True)
    parents = si.random_tree(4, 29, 3, 1)
    tokens = torch.from_numpy(si.random_tokens(shape, 29, 3)).cuda()
    prompt = torch.from_numpy(si.prompt(shape, length=150)).cuda()
    got = {}
    for fused in (True, False):
        eng, _ = make_pair(shape, weights, 256, max_tree=32, max_k=3, max_depth=3, fused=fused)
        pout = eng.new_out(1, 1, 3, T_next=29)
        eng.prefill(0, prompt, 3, [0, 1, 1], parents, pout)
        out = eng.new_out(1, 29, 3)
        runs = []
        for _ in range(3):
            eng.step(tokens, parents, 3, [0, 1, 1], out)
            torch.cuda.synchronize()
            runs.append(out.logits.cpu().numpy().copy())
        assert np.array_equal(runs[0], runs[1]) and np.array_equal(runs[0], runs[2]), "fused=%s: logits differ from run to run" % fused
        got[fused] = (pout.logits.cpu().numpy().copy(), runs[0])
        assert eng.launches() <= (8 if fused else 10 ** 6)
        eng.close()
    for a, b in zip(got[True], got[False]):
        assert np.abs(a - b).max() < 1e-4, np.abs(a - b).max()


def test_fused_prefill_between_steps_keeps_the_steps_launch_plan_intact(torch_cuda, c1, c1_weights):
    """Steps and prefill chunks of at most 48 rows both run as the persistent kernel, each with its own cached launch
    plan and tensor maps on the device.  Prefill, step, prefill a prompt of another length, step again on one
    engine, each time in lock-step with the oracle (a prefill that replaced the step plan's maps would show here)."""
    parents = si.tree_template(c1.T)
    eng, orc = make_pair(c1, c1_weights, 256, fused=True)
    for length in (20, 33, 7, 45):
        st = lockstep_run(eng, orc, c1, parents, si.prompt(c1, length=length), 3, forced_steps=(1,))
        assert st.steps == 3
    eng.close()


def test_a_wait_that_runs_out_is_reported_and_the_context_goes_on(torch_cuda, c1, c1_weights):
    """The time-out path: with the wait limit set to 200 us, firp_selftest_wait enqueues a kernel that waits (with
    the routine the product kernels use) on a barrier nobody arrives on; the wait runs out, the kernel returns, the
    next firp_context_len reports FIRP_ERR_DEVICE_TIMEOUT once, and the same context then steps in lock-step with
    the oracle as if nothing had happened."""
    import time
    import torch
    from paper_2410_20488_b200 import FirpError, binding
    parents = si.tree_template(c1.T)
    eng, orc = make_pair(c1, c1_weights, 256)
    eng.set_wait_limit_us(200)
    t0 = time.time()
    eng.selftest_wait()
    with pytest.raises(FirpError) as e:
        eng.context_len(0)
    assert e.value.code == binding.FIRP_ERR_DEVICE_TIMEOUT
    assert time.time() - t0 < 1.0                      # the 200 us limit was used, not the 2 s default
    assert eng.context_len(0) == 0                    # reported once, then cleared
    eng.set_wait_limit_us(0)
    st = lockstep_run(eng, orc, c1, parents, si.prompt(c1), 3)
    assert st.steps == 3
    eng.close()


def test_layers_are_validated_on_the_host(torch_cuda, c1, c1_weights):
    import torch
    from paper_2410_20488_b200 import FirpError, binding
    eng, _ = make_pair(c1, c1_weights, 128)
    tok = torch.zeros(8, dtype=torch.int32, device="cuda")
    out = eng.new_out(1, 8, 3)
    pout = eng.new_out(1, 1, 3, T_next=8)
    eng.prefill(0, torch.from_numpy(si.prompt(c1)).cuda(), 3, [0, 1, 1], si.tree_template(8), pout)
    for layers in ([1, 0, 1], [0, 1, 2], [-1, 0, 1]):
        with pytest.raises(FirpError) as e:
            eng.step(tok, si.tree_template(8), 3, layers, out)
        assert e.value.code == binding.FIRP_ERR_BAD_ARG
        with pytest.raises(FirpError) as e:
            eng.prefill(0, torch.from_numpy(si.prompt(c1)).cuda(), 3, layers, si.tree_template(8), pout)
        assert e.value.code == binding.FIRP_ERR_BAD_ARG
    eng.close()


@pytest.mark.parametrize("case", range(4))
def test_c1_a_chain_under_every_node(torch_cuda, c1, case):
    """firp_step_chains: k pseudo rows under every tree node, next tree from the end node's chain;
    lock-step against the oracle, greedy and forced, single and per-step insertion layers."""
    T = (8, 5, 19, 36)[case]
    k = (3, 1, 3, 3)[case]
    layers = (1, 0, [0, 1, 3], [1, 2, 2])[case]
    deep = not np.isscalar(layers)
    shape = si.scaled(c1, L=4 if deep else 2, l=1)
    weights = si.all_weights(shape)
    parents = si.tree_template(8) if case == 0 else si.random_tree(9, T, k, case)
    for forced in (False, True):
        eng, orc = make_pair(shape, weights, 512, max_tree=64, max_k=3, max_depth=3, max_rows=T * (1 + k))
        st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=(32, 3, 70, 131)[case]), 4, forced=forced,
                          k=k, l=layers, chains=True)
        assert st.steps == 4
        eng.close()


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("chains", [False, True])
def test_c1_masked_pseudo_rows(torch_cuda, c1, c1_weights, chains, fused):
    """The "Masked" ablation of Section 4.3 (firp_set_pseudo_masked): pseudo rows do not see one another."""
    parents = si.random_tree(3, 13, 3, 2)
    eng, orc = make_pair(c1, c1_weights, 256, masked=True, max_tree=16, max_k=3, max_depth=3, max_rows=13 * 4, fused=fused)
    st = lockstep_run(eng, orc, c1, parents, si.prompt(c1, length=40), 4, k=3, l=1 if chains else [0, 1, 1], chains=chains)
    assert st.steps == 4
    eng.close()


@pytest.mark.parametrize("fused", [False, True])
def test_c1_eq3_on_the_normalised_state(torch_cuda, c1, fused):
    """The variant of Eq. 3 that reads the anchor through the insertion layer's input RMSNorm
    (firp_set_pred_prenorm), with non-unit gains and a bias: one chain with per-step layers, and a chain under
    every node; greedy and forced."""
    shape = si.scaled(c1, L=4, Hkv=2)
    weights = si.all_weights(shape, gains=True)
    weights["pred_b"] = si.normal_bf16(shape.seed, si.stream_id("pred_w", 9), shape.k * shape.d, 0.5).reshape(shape.k, shape.d)
    parents = si.random_tree(6, 12, 3, 3)
    for chains, layers in ((False, [0, 2, 3]), (True, [1, 1, 2]), (False, 2)):
        eng, orc = make_pair(shape, weights, 256, prenorm=True, fused=fused, max_tree=16, max_k=3, max_depth=3, max_rows=12 * 4)
        st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=37), 4, k=3, l=layers, chains=chains, forced_steps=(2,))
        assert st.steps == 4
        eng.close()


@pytest.mark.parametrize("fused", [False, True])
def test_c1_paged_cache(torch_cuda, c1, fused):
    """The KV cache scattered over pages of 64 positions through a shuffled page table (firp_set_kv_pages): two
    sequences stepped together, contexts that start just below a page boundary so that the tree rows of a step
    straddle two pages and the forced-accept commits compact rows from one page into another; every step in
    lock-step with the oracle (which knows nothing of pages), committed cache rows compared through the table."""
    from lockstep import lockstep_run_batch, lockstep_steps_batch
    from paper_2410_20488_b200 import FirpError, binding
    shape = si.scaled(c1, Hkv=2)
    weights = si.all_weights(shape, gains=True)
    parents = si.tree_template(shape.T)
    eng, orc = make_pair(shape, weights, 256, max_batch=2, fused=fused)
    pages = 2 * 256 // 64
    table = si.uniform_i32(5, si.stream_id("tokens", 77), pages, 0, 1 << 20).argsort().astype(np.int32).reshape(2, -1)
    assert sorted(table.reshape(-1).tolist()) == list(range(pages)) and not np.array_equal(table.reshape(-1), np.arange(pages))
    bad = table.copy(); bad[0, 0] = bad[1, 1]
    with pytest.raises(FirpError) as e:
        eng.set_kv_pages(bad)                                    # a page used twice is refused
    assert e.value.code == binding.FIRP_ERR_BAD_ARG
    eng.set_kv_pages(table)
    prompts = [si.prompt(shape, seq=0, length=61), si.prompt(shape, seq=1, length=120)]
    st = lockstep_run_batch(eng, orc, shape, parents, prompts, 6)
    assert st.steps == 12
    # single sequence on the same paged engine: forced-accept steps (real compaction) with the cache rows compared
    st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=58), 5, forced=True, seq=1, check_cache_rows=True)
    assert st.steps == 5
    eng.set_kv_pages(None)                                       # back to contiguous rows
    st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=58), 2, seq=0, check_cache_rows=True)
    assert st.steps == 2
    eng.close()


@pytest.mark.parametrize("head_dim", [64, 128])
@pytest.mark.parametrize("fused", [False, True])
def test_c1_a_tree_of_its_own_for_every_sequence(torch_cuda, c1, fused, head_dim):
    """firp_step_trees: three sequences stepped together, each with its own tree shape and size (8, 5 and 3 of the
    T = 8 rows), its own context length; every sequence is compared with an oracle step on ITS tree (the padding
    rows dropped), both sides commit the oracle's path and take the oracle's next tree on the sequence's own shape.
    A token that would be accepted is planted in a padding row: it must not be."""
    import torch
    from lockstep import own_tree_view
    shape = si.scaled(c1, Hkv=2) if head_dim == 64 else dh128_shape(c1, 4, 2)      # 128: the tensor-core attention
    weights = si.all_weights(shape, gains=True)
    T, k, l = 8, 3, 1
    trees = [si.tree_template(8), si.random_tree(8, 5, 3, 1), si.chain_template(3)]
    sizes = np.array([len(t) for t in trees], np.int32)
    parents = np.full((3, T), 7, np.int32)                    # whatever lies beyond a tree's size is ignored
    for s_i, t in enumerate(trees):
        parents[s_i, : len(t)] = t
    eng, orc = make_pair(shape, weights, 256, max_batch=3, fused=fused)
    tokens = np.zeros((3, T), np.int32)
    for s_i, n in enumerate((40, 9, 77)):
        pout = eng.new_out(1, 1, k, T_next=len(trees[s_i]))
        eng.prefill(s_i, torch.from_numpy(si.prompt(shape, seq=s_i, length=n)).cuda(), k, l, trees[s_i], pout)
        ref = orc.prefill(si.prompt(shape, seq=s_i, length=n), k, l, trees[s_i], seq=s_i)
        tokens[s_i, : sizes[s_i]] = ref["next_tokens"]
    out = eng.new_out(3, T, k)
    st = Stats()
    for step in range(5):
        refs = [orc.step(tokens[s_i, : sizes[s_i]], trees[s_i], k, l, seq=s_i) for s_i in range(3)]
        for s_i in (1, 2):                                    # the padding rows carry the token the root would accept
            tokens[s_i, sizes[s_i]:] = refs[s_i]["best"][0]
        eng.step_trees(torch.from_numpy(tokens).cuda(), parents, sizes, k, l, out, seq_ids=[0, 1, 2])
        for s_i in range(3):
            g = own_tree_view(gpu_outputs(out, s_i, T, k), int(sizes[s_i]), T, k)
            compare_step(shape, trees[s_i], tokens[s_i, : sizes[s_i]], k, g, refs[s_i], st)
        eng.commit(3, seq_ids=[0, 1, 2], path=[r["path"] for r in refs])
        for s_i in range(3):
            orc.commit(refs[s_i]["path"], seq=s_i)
            assert eng.context_len(s_i) == orc.context_len(s_i)
            tokens[s_i, : sizes[s_i]] = refs[s_i]["next_tokens"]
    assert st.steps == 15
    eng.close()


# ---- head dimension 128: the tcgen05 attention kernel (and the mma.sync one on the same cases) ----------------
def dh128_shape(c1, H, Hkv):
    return si.scaled(c1, d=256, H=H, Hkv=Hkv, dh=128, F=512)


@pytest.mark.parametrize("tensor_core", [True, False])
@pytest.mark.parametrize("case", range(7))
def test_dh128_tree_sizes_and_contexts(torch_cuda, c1, case, tensor_core):
    """Tree sizes that select every query-block width of the tensor-core kernel (16, 32, 48, 80 columns, and two
    blocks at 131 rows), contexts that end just below, on and above a 128-position tile boundary (so that the new
    rows straddle tiles and the last tile is ragged), one to several tiles per split, and a context long enough for
    the largest cluster (8 splits of two tiles); gains non-unit."""
    T, k, n0, steps = ((1, 0, 5, 3), (8, 3, 126, 4), (24, 3, 128, 4), (40, 3, 250, 4), (64, 3, 383, 3), (128, 3, 700, 3),
                       (8, 3, 1990, 3))[case]
    shape = dh128_shape(c1, 2, 2)
    weights = si.all_weights(shape, gains=True)
    parents = si.chain_template(1) if T == 1 else si.random_tree(31, T, max(k, 1), case)
    eng, orc = make_pair(shape, weights, max(1024, n0 + 256), max_tree=128, max_k=3, max_depth=3)
    eng.set_attention_kernel(tensor_core)
    st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=n0), steps, k=k, l=1, forced_steps=(1,))
    assert st.steps == steps
    eng.close()


@pytest.mark.parametrize("tensor_core", [True, False])
@pytest.mark.parametrize("case", range(3))
def test_dh128_chains_layers_and_masked_rows(torch_cuda, c1, case, tensor_core):
    """The variants of the step at head dimension 128, on both attention kernels: a chain of pseudo rows under every
    node (firp_step_chains: 36 x 4 = 144 rows, three query blocks, per-step insertion layers), one insertion layer
    per prediction step (firp_step_layers), and the "Masked" ablation (pseudo rows do not see each other); four
    layers deep, contexts that put the new rows across a tile boundary, greedy and forced."""
    shape = si.scaled(dh128_shape(c1, 4, 2), L=4, l=1)
    weights = si.all_weights(shape, gains=True)
    for forced in (False, True):
        if case == 0:
            T, k, layers = 36, 3, [1, 2, 2]
            parents = si.random_tree(9, T, k, 3)
            eng, orc = make_pair(shape, weights, 512, max_tree=64, max_k=3, max_depth=3, max_rows=T * (1 + k))
            eng.set_attention_kernel(tensor_core)
            st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=131), 3, forced=forced, k=k, l=layers, chains=True)
        elif case == 1:
            parents = si.random_tree(5, 19, 3, 6)
            eng, orc = make_pair(shape, weights, 512, max_tree=32, max_k=3, max_depth=3)
            eng.set_attention_kernel(tensor_core)
            st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=250), 3, forced=forced, k=3, l=[0, 1, 3])
        else:
            parents = si.tree_template(32)
            eng, orc = make_pair(shape, weights, 512, masked=True, max_tree=32, max_k=3, max_depth=3)
            eng.set_attention_kernel(tensor_core)
            st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=120), 3, forced=forced, k=3, l=1)
        assert st.steps == 3
        eng.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_dh128_random_shapes_in_lockstep(torch_cuda, c1, seed):
    """Twelve seeded random cases per seed at head dimension 128: heads per kv head 1 / 2 / 4 / 8, tree sizes 1..64
    (every query-block width, one to three blocks), one to three sequences of unrelated context lengths (1..700,
    i.e. any number of tiles and a ragged last one), contiguous or paged cache, the tensor-core kernel forced or the
    library's own choice; three steps each (one forced-accept for single sequences) against the oracle."""
    from lockstep import lockstep_run_batch
    rng = np.random.default_rng(seed)
    done = 0
    while done < 12:
        H, Hkv = [(2, 2), (4, 2), (4, 1), (8, 1), (4, 4)][rng.integers(5)]
        T = int(rng.choice([1, 2, 5, 8, 13, 16, 17, 24, 29, 33, 40, 47, 64]))
        k = 0 if T == 1 else (3 if T > 40 else int(rng.integers(2 if T > 9 else 1, 4)))
        n_seq = int(rng.choice([1, 1, 2, 3]))
        if n_seq * (T + k) > 144:
            n_seq = 1
        lengths = [int(rng.integers(1, 700)) for _ in range(n_seq)]
        tensor_core = [True, None][rng.integers(2)]
        paged = bool(rng.integers(2)) and n_seq > 1
        shape = si.scaled(dh128_shape(c1, H, Hkv), seed=int(rng.integers(1000)))
        try:
            parents = si.chain_template(1) if T == 1 else si.random_tree(int(rng.integers(1000)), T, max(k, 1), done)
        except ValueError:
            continue                                           # no such tree under that depth
        weights = si.all_weights(shape, gains=True)
        eng, orc = make_pair(shape, weights, 1024, max_batch=n_seq, max_tree=T, max_k=max(k, 1), max_depth=3)
        eng.set_attention_kernel(tensor_core)
        if paged:
            eng.set_kv_pages(rng.permutation(n_seq * 1024 // 64).astype(np.int32).reshape(n_seq, -1))
        case = "H=%d Hkv=%d T=%d k=%d lengths=%s tensor_core=%s paged=%s" % (H, Hkv, T, k, lengths, tensor_core, paged)
        try:
            if n_seq == 1:
                st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=lengths[0]), 3, k=k,
                                  l=int(rng.integers(0, 2)), forced_steps=(1,))
            else:
                st = lockstep_run_batch(eng, orc, shape, parents,
                                        [si.prompt(shape, seq=s_i, length=lengths[s_i]) for s_i in range(n_seq)], 3, k=k, l=1)
        except AssertionError as e:
            raise AssertionError("%s: %s" % (case, e))
        assert st.steps == 3 * n_seq, case
        eng.close()
        done += 1


def test_dh128_free_running_decode_repeats_bit_for_bit(torch_cuda, c1):
    """400 free-running steps (device-side commits) on the tensor-core attention, twice from the same state: the
    context grows across tile boundaries and split counts, and every accepted token and every next tree must
    repeat exactly (the kernel's barriers, buffers and merge order leave nothing to timing)."""
    import hashlib
    import torch
    from paper_2410_20488_b200 import FirpEngine
    shape = dh128_shape(c1, 4, 2)
    weights = si.all_weights(shape, gains=True)
    T, k = 16, 3
    parents = si.random_tree(37, T, 3, 3)
    eng = FirpEngine(shape, weights, max_ctx=2048, max_tree=T, max_k=k, max_depth=3)
    eng.set_attention_kernel(True)
    out = eng.new_out(1, T, k, want_logits=False)
    digests = []
    for rep in range(2):
        eng.set_context_len(0, 90)
        cur = torch.from_numpy(si.random_tokens(shape, T, 3)).cuda().reshape(1, T)
        seen = []
        for _ in range(400):
            eng.step(cur, parents, k, 1, out)
            eng.commit(1)
            seen.append(out.n_accepted.clone())          # accepted_tokens holds n_accepted valid entries: compared through
            seen.append(out.best.clone())                # the verification argmax of every row and the next tree instead
            cur = out.next_tree_tokens.clone()
            seen.append(cur)
        torch.cuda.synchronize()
        h = hashlib.sha256()
        for t in seen:
            h.update(t.cpu().numpy().tobytes())
        digests.append((h.hexdigest(), eng.context_len(0)))
    assert digests[0] == digests[1] and digests[0][1] >= 490
    eng.close()


@pytest.mark.parametrize("tensor_core", [True, False])
def test_dh128_plane_counts(torch_cuda, c1, tensor_core):
    """firp_set_attention_planes / firp_set_activation_planes: plain bf16 operands (one plane) run through both
    attention kernels and every GEMM class, stay inside the bound on this two-layer shape, and deviate more from the
    oracle than the default (hi, lo) planes do; counts outside 1..2 (1..3 for the QKV projection) are refused."""
    from paper_2410_20488_b200 import FirpError, binding
    shape = dh128_shape(c1, 2, 2)
    weights = si.all_weights(shape, gains=True)
    parents = si.random_tree(35, 24, 3, 2)
    dev = {}
    for planes in (2, 1):
        eng, orc = make_pair(shape, weights, 512, max_tree=24, max_k=3, max_depth=3)
        eng.set_attention_kernel(tensor_core)
        eng.set_attention_planes(planes, planes)
        eng.set_activation_planes(planes, planes, planes, planes, planes)
        st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=300), 3, k=3, l=1, check_cache_rows=planes == 2)
        dev[planes] = st.max_abs
        for bad in ((0, 2), (2, 3)):
            with pytest.raises(FirpError) as e:
                eng.set_attention_planes(*bad)
            assert e.value.code == binding.FIRP_ERR_BAD_ARG
        with pytest.raises(FirpError) as e:
            eng.set_activation_planes(4, 2, 2, 2, 2)
        assert e.value.code == binding.FIRP_ERR_BAD_ARG
        eng.close()
    assert dev[1] > 2 * dev[2], dev


@pytest.mark.parametrize("tensor_core", [True, False, None])
def test_dh128_slot_rows_off_the_tile_grid(torch_cuda, c1, tensor_core):
    """A cache of 300 positions per sequence (no multiple of a 64- or 128-position tile) and the second slot: its rows
    start in the middle of a tile of the plane, the last tile of the context reaches into rows that are not its own,
    and the context ends 20 positions below the capacity.  None: the library chooses the kernel."""
    shape = dh128_shape(c1, 2, 2)
    weights = si.all_weights(shape, gains=True)
    parents = si.random_tree(33, 24, 3, 5)
    eng, orc = make_pair(shape, weights, 300, max_batch=2, max_tree=24, max_k=3, max_depth=3)
    eng.set_attention_kernel(tensor_core)
    st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, seq=1, length=241), 3, k=3, l=1, forced_steps=(1,), seq=1)
    assert st.steps == 3 and eng.context_len(1) <= 300 - 27
    eng.close()


@pytest.mark.parametrize("tensor_core", [True, False])
@pytest.mark.parametrize("Hkv", [2, 1])
def test_dh128_grouped_queries_batch_and_pages(torch_cuda, c1, Hkv, tensor_core):
    """4 query heads on 2 or 1 key/value heads (35 x 2 = 70 query columns in one block; 35 x 4 = 140 in two), three
    sequences of different context lengths in one step, then the same engine with the cache scattered over pages."""
    from lockstep import lockstep_run_batch
    shape = dh128_shape(c1, 4, Hkv)
    weights = si.all_weights(shape, gains=True)
    parents = si.tree_template(32)
    eng, orc = make_pair(shape, weights, 512, max_batch=3, max_tree=32, max_k=3, max_depth=3)
    from paper_2410_20488_b200 import binding
    assert binding.load_library().firp_set_attention_kernel(eng.ctx, 2) == binding.FIRP_ERR_BAD_ARG
    eng.set_attention_kernel(tensor_core)
    prompts = [si.prompt(shape, seq=0, length=300), si.prompt(shape, seq=1, length=7), si.prompt(shape, seq=2, length=129)]
    st = lockstep_run_batch(eng, orc, shape, parents, prompts, 4)
    assert st.steps == 12
    pages = 3 * 512 // 64
    table = si.uniform_i32(6, si.stream_id("tokens", 78), pages, 0, 1 << 20).argsort().astype(np.int32).reshape(3, -1)
    eng.set_kv_pages(table)
    st = lockstep_run_batch(eng, orc, shape, parents, [p[:n] for p, n in zip(prompts, (190, 60, 255))], 4)
    assert st.steps == 12
    st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=120), 4, forced=True, seq=2, check_cache_rows=True)
    assert st.steps == 4
    eng.close()


def test_chains_need_the_row_capacity(torch_cuda, c1, c1_weights):
    import torch
    from paper_2410_20488_b200 import FirpError, binding
    eng, _ = make_pair(c1, c1_weights, 128)                                   # max_rows defaults to T + k = 11
    tok = torch.zeros(8, dtype=torch.int32, device="cuda")
    out = eng.new_out(1, 8, 3, chains=True)
    pout = eng.new_out(1, 1, 3, T_next=8)
    eng.prefill(0, torch.from_numpy(si.prompt(c1)).cuda(), 3, 1, si.tree_template(8), pout)
    with pytest.raises(FirpError) as e:
        eng.step_chains(tok, si.tree_template(8), 3, 1, out)
    assert e.value.code == binding.FIRP_ERR_CAPACITY and "max_rows" in str(e.value)
    eng.close()


def test_c1_predictor_with_bias(torch_cuda, c1, c1_weights):
    """Eq. 3 with a non-zero bias b_i (the synthetic configurations use b = 0)."""
    w = dict(c1_weights)
    w["pred_b"] = si.normal_bf16(c1.seed, si.stream_id("pred_w", 7), c1.k * c1.d, 0.5).reshape(c1.k, c1.d)
    parents = si.tree_template(c1.T)
    eng, orc = make_pair(c1, w, 256)
    st = lockstep_run(eng, orc, c1, parents, si.prompt(c1, length=19), 3)
    assert st.steps == 3
    eng.close()


def test_device_side_commit_matches_explicit(torch_cuda, c1, c1_weights):
    """firp_kv_commit(path = NULL) compacts the path the device's own walk found: forced-accept steps make that a
    real depth-3 path; the committed cache rows and the logits of the following steps are compared with the oracle,
    which commits the same path explicitly."""
    import torch
    parents = si.tree_template(c1.T)
    eng, orc = make_pair(c1, c1_weights, 256)
    st = lockstep_run(eng, orc, c1, parents, si.prompt(c1), 2)
    tokens = si.random_tokens(c1, c1.T, 123)              # any tree will do: forced mode plants the principal chain
    st = lockstep_steps(eng, orc, c1, parents, tokens, 6, forced=True, device_commit=True, check_cache_rows=True)
    assert st.steps == 6 and st.emitted == 6 * 4
    # free-running with device-side commits: the committed length follows the device's own counts
    out = eng.new_out(1, c1.T, c1.k)
    total = eng.context_len(0)
    d_tokens = torch.from_numpy(np.ascontiguousarray(tokens)).cuda()
    for _ in range(4):
        eng.step(d_tokens, parents, c1.k, c1.l, out)
        eng.commit(1)
        total += int(out.n_accepted[0].item())
        assert eng.context_len(0) == total
        d_tokens = out.next_tree_tokens[0].clone()
    eng.close()


def test_device_side_commits_do_not_exhaust_the_capacity_bound(torch_cuda, c1, c1_weights):
    """A free-running loop that only ever commits on the device: the host's upper bound of the committed length
    grows by max_depth + 1 per step, the true length by about 1.  The step must keep running until the TRUE
    length reaches max_ctx (it re-reads the exact length before refusing), and refuse then."""
    import torch
    from paper_2410_20488_b200 import FirpError, binding
    parents = si.tree_template(c1.T)
    eng, _ = make_pair(c1, c1_weights, 128)
    pout = eng.new_out(1, 1, c1.k, T_next=c1.T)
    eng.prefill(0, torch.from_numpy(si.prompt(c1, length=16)).cuda(), c1.k, c1.l, parents, pout)
    out = eng.new_out(1, c1.T, c1.k)
    tokens = pout.next_tree_tokens[0].clone()
    steps, total = 0, 16
    with pytest.raises(FirpError) as e:
        for _ in range(200):
            eng.step(tokens, parents, c1.k, c1.l, out)
            eng.commit(1)
            steps += 1
            total += int(out.n_accepted[0].item())
            tokens = out.next_tree_tokens[0].clone()
    assert e.value.code == binding.FIRP_ERR_CAPACITY
    assert total + c1.T + c1.k > 128 and steps > (128 - 16 - 11) // 4, (steps, total)   # far beyond where the bound alone would stop
    assert eng.context_len(0) == total
    eng.close()


def test_host_validation_on_device(torch_cuda, c1, c1_weights):
    import torch
    from paper_2410_20488_b200 import FirpError, binding
    eng, _ = make_pair(c1, c1_weights, 64)
    tok = torch.zeros(8, dtype=torch.int32, device="cuda")
    out = eng.new_out(1, 8, 3)
    cases = [([0, 0, 1, 2, 0, 1, 4, 5], binding.FIRP_ERR_BAD_TREE),          # parents[0] != -1
             ([-1, 0, 1, 2, 3, 1, 4, 5], binding.FIRP_ERR_BAD_TREE),         # depth 4 > k
             ([-1, 0, 2, 1, 0, 1, 4, 5], binding.FIRP_ERR_BAD_TREE)]         # parents[2] >= 2
    for parents, code in cases:
        with pytest.raises(FirpError) as e:
            eng.step(tok, np.array(parents, np.int32), 3, 1, out)
        assert e.value.code == code
    with pytest.raises(FirpError) as e:                                       # k beyond the loaded maps
        eng.step(tok, si.tree_template(8), 4, 1, out)
    assert e.value.code == binding.FIRP_ERR_CAPACITY
    with pytest.raises(FirpError) as e:                                       # commit without a step
        eng.commit(1)
    assert e.value.code == binding.FIRP_ERR_STATE
    eng.set_context_len(0, 60)                                                # 60 + 11 rows > max_ctx 64
    with pytest.raises(FirpError) as e:
        eng.step(tok, si.tree_template(8), 3, 1, out)
    assert e.value.code == binding.FIRP_ERR_CAPACITY
    eng.close()


@pytest.fixture(scope="module")
def c2_weights():
    return si.all_weights(si.CONFIGS["c2"])


def test_c2_full_size_lockstep(torch_cuda, c2_weights):
    """The Llama-2-7B-shaped workload the benchmark times (T = 32, k = 3, l = 16, 512 committed
    tokens): prefill and three lock-step steps against the oracle, the last one forced-accept (a depth-3 path is
    compacted at the full 4096-wide cache rows and compared), then one more forced step committed from the
    device's own path."""
    c2 = si.CONFIGS["c2"]
    parents = si.tree_template(c2.T)
    eng, orc = make_pair(c2, c2_weights, 512 + 64)
    st = lockstep_run(eng, orc, c2, parents, si.prompt(c2), 3, forced_steps=(2,), check_cache_rows=True, sync_prefix=True)
    print("c2 greedy + forced", st.as_dict())
    assert st.steps == 3 and st.emitted == 1 + 1 + 1 + 4
    tokens = si.random_tokens(c2, c2.T, 123)
    st = lockstep_steps(eng, orc, c2, parents, tokens, 1, forced=True, device_commit=True, check_cache_rows=True)
    print("c2 forced, device-side commit", st.as_dict())
    eng.close()


@pytest.mark.parametrize("fused", [False, True])
def test_c2_layers_15_20_25_full_size(torch_cuda, c2_weights, fused):
    """The prediction layers the paper uses for its 7B models (Section 4 "Setup": 15, 20, 25) on the
    7B-shaped workload: prefill and two lock-step steps against the oracle, with the layers of a step as one
    kernel per operation and as one persistent kernel."""
    c2 = si.CONFIGS["c2"]
    parents = si.tree_template(c2.T)
    eng, orc = make_pair(c2, c2_weights, 128 + 64, fused=fused)          # a 128-token context keeps the oracle's prefill short
    st = lockstep_run(eng, orc, c2, parents, si.prompt(c2, length=128), 2, forced=False, check_cache_rows=False, l=[15, 20, 25],
                      sync_prefix=True)
    print("c2 layers 15/20/25", st.as_dict())
    assert st.steps == 2
    eng.close()


def test_c2_chain_under_every_node_full_size(torch_cuda, c2_weights):
    """T = 32 nodes each with a chain of k = 3 pseudo rows (128 rows from layer 16 on) at the 7B shape:
    prefill and one lock-step step against the oracle."""
    c2 = si.CONFIGS["c2"]
    parents = si.tree_template(c2.T)
    eng, orc = make_pair(c2, c2_weights, 128 + 160, max_rows=c2.T * (1 + c2.k))
    st = lockstep_run(eng, orc, c2, parents, si.prompt(c2, length=128), 1, forced=False, check_cache_rows=False, chains=True,
                      sync_prefix=True)
    print("c2 chains", st.as_dict())
    assert st.steps == 1
    eng.close()


def test_c4_tree_sizes_full_depth(torch_cuda, c2_weights):
    """Sweep points on the Llama-2-7B shape, all 32 layers: T = 1 (plain autoregressive, k = 0), 8, 16, 64, 128
    on a 128-token context (every row-count variant of the GEMM, 1 to 8 attention splits)."""
    c2 = si.CONFIGS["c2"]
    for T in (1, 8, 16, 64, 128):
        k = 0 if T == 1 else 3
        parents = si.tree_template(T)
        eng, orc = make_pair(c2, c2_weights, 128 + 160, max_tree=T, max_k=max(k, 1), max_depth=3)
        st = lockstep_run(eng, orc, c2, parents, si.prompt(c2, length=128), 1, k=k, l=c2.l, check_cache_rows=False, sync_prefix=True)
        print("c4 full depth T=%d" % T, st.as_dict())
        assert st.steps == 1
        eng.close()


@pytest.fixture(scope="module")
def c2_width_2_layers():
    shape = si.scaled(si.CONFIGS["c2"], L=2, l=1, name="c2-width-2-layers")
    return shape, si.all_weights(shape)


def test_c2_width_chains_with_one_layer_per_step(torch_cuda):
    """A chain under every node with the prediction steps at layers 1, 2, 3 of a 4-layer decoder of the 7B width:
    32, 64, 96 and 128 rows in successive layers, so one step runs the 40-, 80- and 144-row GEMM variants and
    the Eq. 3 GEMM on all 32 tree rows."""
    shape = si.scaled(si.CONFIGS["c2"], L=4, l=1, name="c2-width-4-layers")
    weights = si.all_weights(shape)
    parents = si.tree_template(shape.T)
    eng, orc = make_pair(shape, weights, 256 + 160, max_rows=shape.T * (1 + shape.k))
    st = lockstep_run(eng, orc, shape, parents, si.prompt(shape, length=200), 3, k=3, l=[1, 2, 3], chains=True,
                      check_cache_rows=True)
    print("c2 width, chains, layers 1/2/3", st.as_dict())
    assert st.steps == 3
    eng.close()


@pytest.mark.parametrize("n_ctx", [2048, 8192])
def test_c4_long_contexts_against_the_oracle(torch_cuda, c2_width_2_layers, n_ctx):
    """Sweep points with 2048 and 8192 committed tokens at the full Llama-2-7B width, depth cut to 2 layers, for
    T = 1 (k = 0), 32 and 128: both sides start from the same seeded prefix (bit-identical cache rows written into
    both caches, no prefill), so the oracle's cost per step is linear in the context.  The attention then runs over
    33 / 129 tiles in 8 splits, with one, one and three query blocks."""
    shape, weights = c2_width_2_layers
    for T in (1, 32, 128):
        k = 0 if T == 1 else 3
        parents = si.tree_template(T)
        eng, orc = make_pair(shape, weights, n_ctx + 2 * 160, max_tree=128, max_k=3, max_depth=3)
        seed_prefix(eng, orc, shape, 0, n_ctx)
        st = lockstep_steps(eng, orc, shape, parents, si.random_tokens(shape, T, 77 + T), 2, k=k, l=shape.l if k else 0,
                            forced_steps=(1,) if k else (), check_cache_rows=True)
        print("c4 seeded context n=%d T=%d" % (n_ctx, T), st.as_dict())
        assert st.steps == 2
        eng.close()


def test_c3_full_depth(torch_cuda):
    """Llama-2-13B shape, all 40 layers, T = 64, k = 3 at layer 20, on the configuration's 1024 committed tokens
    (seeded prefix on both sides): two lock-step steps, the second forced-accept, then the prompt path: a 128-token
    prefill through the library and one more step."""
    c3 = si.CONFIGS["c3"]
    weights = si.all_weights(c3)
    parents = si.tree_template(c3.T)
    eng, orc = make_pair(c3, weights, 1024 + 2 * 160)
    seed_prefix(eng, orc, c3, 0, 1024)
    st = lockstep_steps(eng, orc, c3, parents, si.random_tokens(c3, c3.T, 5), 2, forced_steps=(1,), check_cache_rows=True)
    print("c3 seeded context 1024", st.as_dict())
    assert st.steps == 2
    st = lockstep_run(eng, orc, c3, parents, si.prompt(c3, length=128), 1, check_cache_rows=False, sync_prefix=True)
    print("c3 after a 128-token prefill", st.as_dict())
    eng.close()


def test_c5_gqa_batch_reduced_depth(torch_cuda):
    """34B grouped-query shape (d 8192, 64 query / 8 kv heads, FFN 22016), batch of 4 sequences with their own
    32-node trees, stepped by one firp_step call; depth cut from 48 to 4 layers (the full model needs a minute of
    oracle time per step and 67 GB of weights on both sides).  First on short prompts through the library's
    prefill, then on the configuration's context lengths (drawn uniformly from [256, 4096], seeded prefixes):
    the sequences then differ in their number of kv tiles inside one attention launch."""
    from lockstep import lockstep_run_batch, lockstep_steps_batch
    shape = si.scaled(si.CONFIGS["c5"], L=4, l=2, name="c5-width-4-layers")
    weights = si.all_weights(shape)
    parents = si.tree_template(shape.T)
    lengths = (23, 64, 97, 130)
    prompts = [si.prompt(shape, seq=s, length=n) for s, n in enumerate(lengths)]
    eng, orc = make_pair(shape, weights, 4096 + 160, max_batch=4)
    st = lockstep_run_batch(eng, orc, shape, parents, prompts, 1)
    print("c5 reduced depth, short prompts", st.as_dict())
    assert st.steps == 4
    ctx = si.context_lengths(shape)
    assert ctx.min() >= 256 and ctx.max() <= 4096 and len(set(ctx.tolist())) == 4
    for s_i, n in enumerate(ctx):
        seed_prefix(eng, orc, shape, s_i, int(n))
    tokens = np.stack([si.random_tokens(shape, shape.T, 40 + s_i) for s_i in range(4)])
    st = lockstep_steps_batch(eng, orc, shape, parents, tokens, 2, check_cache_rows=True)
    print("c5 reduced depth, contexts %s" % ctx.tolist(), st.as_dict())
    assert st.steps == 8
    eng.close()
