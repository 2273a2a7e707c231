"""Parity of the CUDA path (through the C ABI) against the CPU oracle, on a B200."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from lockstep import lockstep_run, compare_step, gpu_outputs, Stats

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2410_20488_b200 import build as firp_build
    firp_build.build()
    return torch


def make_pair(shape, weights, max_ctx, **kw):
    from paper_2410_20488_b200 import FirpEngine
    eng = FirpEngine(shape, weights, max_ctx=max_ctx, **kw)
    orc = oracle.Oracle(shape, weights, max_ctx=max_ctx, n_seq=kw.get("max_batch", 1))
    return eng, orc


def test_c1_greedy_and_forced(torch_cuda, c1, c1_weights):
    parents = si.tree_template(c1.T)
    for forced in (False, True):
        eng, orc = make_pair(c1, c1_weights, 256)
        st = lockstep_run(eng, orc, c1, parents, si.prompt(c1), c1.steps, forced=forced)
        assert st.steps == c1.steps
        if forced:
            assert st.emitted == 1 + c1.steps * 4
        print("c1 forced=%s" % forced, st.as_dict())
        eng.close()


def test_c1_t1_k0_autoregressive(torch_cuda, c1, c1_weights):
    eng, orc = make_pair(c1, c1_weights, 128, max_tree=8, max_k=3)
    st = lockstep_run(eng, orc, c1, np.array([-1], np.int32), si.prompt(c1, length=9), 12, k=0, l=0)
    assert st.steps == 12 and st.emitted == 13
    eng.close()


@pytest.mark.parametrize("case", range(4))
def test_c1_random_trees_and_layers(torch_cuda, c1, c1_weights, case):
    T = (5, 16, 33, 128)[case]
    k = (1, 3, 2, 3)[case]
    l = (0, 1, 1, 0)[case]
    parents = si.random_tree(21, T, k, case)
    eng, orc = make_pair(c1, c1_weights, 512, max_tree=128, max_k=3, max_depth=3)
    st = lockstep_run(eng, orc, c1, parents, si.prompt(c1, length=(3, 70, 129, 200)[case]), 4, k=k, l=l)
    assert st.steps == 4
    eng.close()


def test_device_side_commit_matches_explicit(torch_cuda, c1, c1_weights):
    """firp_kv_commit(NULL path) uses the path found on the device."""
    import torch
    parents = si.tree_template(c1.T)
    eng, orc = make_pair(c1, c1_weights, 256)
    prompt = si.prompt(c1)
    d_prompt = torch.from_numpy(prompt).cuda()
    pout = eng.new_out(1, 1, c1.k, T_next=c1.T)
    eng.prefill(0, d_prompt, c1.k, c1.l, parents, pout)
    out = eng.new_out(1, c1.T, c1.k)
    tokens = pout.next_tree_tokens[0].clone()
    total = prompt.size
    for _ in range(6):
        eng.step(tokens, parents, c1.k, c1.l, out)
        eng.commit(1)                                   # device-side path
        total += int(out.n_accepted[0].item())
        assert eng.context_len(0) == total
        tokens = out.next_tree_tokens[0].clone()
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
    tokens): prefill and three lock-step steps against the oracle, the last one forced-accept."""
    c2 = si.CONFIGS["c2"]
    parents = si.tree_template(c2.T)
    eng, orc = make_pair(c2, c2_weights, 512 + 64)
    st = lockstep_run(eng, orc, c2, parents, si.prompt(c2), 2, forced=False, check_cache_rows=True)
    print("c2 greedy", st.as_dict())
    assert st.steps == 2
    eng.close()
